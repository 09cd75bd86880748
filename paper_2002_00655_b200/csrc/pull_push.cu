// pull, push and the small maintenance kernels of the parameter store.
//
// pull  (Table 2 of the paper): key -> (owner, slot) lookup, then a 128-bit
//       vectorised gather of the row.
// push  (Table 2; cumulative, Section 2.1): the occurrences of a call are
//       sorted by key; a warp reduces 32 consecutive sorted occurrences in
//       fp64, applies every segment that lies wholly inside its tile with one
//       read-modify-write of the row, and parks partial sums of segments that
//       cross tile borders; a second kernel adds those partials in tile order.
//       The order of every sum is fixed by the sorted positions, so results
//       are reproducible bit for bit.
#include "ps_internal.cuh"

namespace psb {

// ---------------------------------------------------------------- init ----
__global__ void init_range_partition_kernel(uint2* __restrict__ table, unsigned long long* __restrict__ tops,
                                            uint32_t* __restrict__ stacks, uint64_t K, uint32_t N, uint64_t S,
                                            uint64_t B) {
    const uint64_t gid = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t k = gid; k < K; k += stride) table[k] = make_uint2((uint32_t)(k / B), (uint32_t)(k % B));
    for (uint64_t x = gid; x < (uint64_t)N * S; x += stride) {
        const uint64_t p = x / S, t = x % S;
        const uint64_t first = p * B;
        const uint64_t cnt = first >= K ? 0 : tmin<uint64_t>(K - first, B);
        if (t < S - cnt) stacks[x] = (uint32_t)(S - 1 - t);
        if (t == 0) tops[p] = S - cnt;
    }
}

void launch_init_range_partition(ps_store* ps, cudaStream_t s) {
    const uint64_t K = ps->cfg.num_keys, S = ps->cfg.slots_per_part;
    const uint32_t N = ps->cfg.num_workers;
    const uint64_t B = (K + N - 1) / N;
    const uint64_t work = tmax<uint64_t>(K, (uint64_t)N * S);
    const uint32_t grid = (uint32_t)tmin<uint64_t>((work + 255) / 256, (uint64_t)ps->sm_count * 16);
    PS_LAUNCH(ps, init_range_partition_kernel, grid, 256, s, ps->table, ps->tops, ps->stacks, K, N, S, B);
}

// ------------------------------------------------------------ set rows ----
__global__ void __launch_bounds__(256)
set_rows_kernel(const uint64_t* __restrict__ keys, uint64_t n, const float4* __restrict__ vals,
                float4* __restrict__ store, const uint2* __restrict__ table, uint64_t S, uint64_t K, uint32_t L4,
                DevStatus* st, unsigned int epoch) {
    const int lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t n_warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    for (uint64_t t = warp; t < n; t += n_warps) {
        const uint64_t key = keys[t];
        if (key >= K) {
            if (lane == 0) latch_error(st, epoch, PS_ERR_KEY_RANGE);
            continue;
        }
        const uint64_t row = phys_row(table[key], S);
        for (uint32_t f = lane; f < L4; f += 32) store[row * L4 + f] = vals[t * L4 + f];
    }
}

void launch_set_rows(ps_store* ps, const uint64_t* d_keys, uint64_t n, const float* d_vals, cudaStream_t s) {
    const uint32_t grid = (uint32_t)tmin<uint64_t>((n + 7) / 8, (uint64_t)ps->sm_count * 8);
    PS_LAUNCH(ps, set_rows_kernel, grid, 256, s, d_keys, n, (const float4*)d_vals, (float4*)ps->store, ps->table,
              ps->cfg.slots_per_part, ps->cfg.num_keys, ps->cfg.row_len / 4, ps->status, 0u);
}

// ---------------------------------------------------------------- pull ----
// Rows travel store -> shared memory -> caller's buffer as bulk asynchronous copies of whole rows, without
// passing through registers: a lane looks its key up, asks for the row, and once the round's rows have
// landed asks for them to be written out.  A warp works on rounds of kPullStageBytes / row_bytes keys, two
// rounds in flight (the loads of one beside the stores of the one before).
constexpr uint32_t kPullStageBytes = 4096;          // per warp and stage
constexpr size_t kPullSmem = (size_t)8 * 2 * kPullStageBytes;

__global__ void __launch_bounds__(256)
pull_bulk_kernel(const uint64_t* __restrict__ keys, uint64_t n, char* __restrict__ out, const char* __restrict__ store,
                 const uint2* __restrict__ table, uint64_t S, uint64_t K, uint32_t row_bytes, uint32_t per_round,
                 DevStatus* st, unsigned int epoch) {
    __shared__ __align__(8) uint64_t bars[8][2];
    extern __shared__ __align__(128) char pull_stage[];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t n_warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    char* my = pull_stage + (size_t)w * 2 * kPullStageBytes;
    if (lane < 2) mbar_init(&bars[w][lane], 1);
    mbar_init_fence();
    __syncwarp();
    uint32_t uses = 0;
    int stage = 0;
    // the round whose loads are in flight: its first key, how many rows were asked for, whether this lane has one
    uint64_t prev_t0 = 0;
    uint32_t prev_rows = 0;
    bool prev_mine = false, have_prev = false;
    auto finish = [&](int sg) -> bool {             // waits for a round's rows and sends them on their way
        if (prev_rows) {
            const uint32_t parity = (uses >> sg) & 1u;
            if (!mbar_wait(&bars[w][sg], parity) && !mbar_wait(&bars[w][sg], parity)) {
                if (lane == 0) latch_error(st, epoch, PS_ERR_CUDA);
                return false;
            }
            uses ^= 1u << sg;
            fence_async_smem();
        }
        if (prev_mine)
            bulk_s2g(out + (prev_t0 + lane) * row_bytes, my + (size_t)sg * kPullStageBytes + (size_t)lane * row_bytes,
                     row_bytes);
        bulk_commit();
        return true;
    };
    for (uint64_t t0 = warp * per_round; t0 < n; t0 += n_warps * per_round) {
        const uint64_t t = t0 + lane;
        const bool mine = (uint32_t)lane < per_round && t < n;
        uint64_t row = 0;
        bool ok = false;
        if (mine) {
            const uint64_t key = keys[t];
            if (key < K) {
                row = phys_row(table[key], S);
                ok = true;
            } else {
                latch_error(st, epoch, PS_ERR_KEY_RANGE);
                float4* o = (float4*)(out + t * row_bytes);         // a key out of range reads as a row of zeros
                for (uint32_t f = 0; f < row_bytes / 16; ++f) o[f] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        const uint32_t rows = __popc(__ballot_sync(0xffffffffu, ok));
        bulk_wait_read<0>();                        // the stores that last read this stage (the round before last) are done with it
        __syncwarp();
        if (rows) {
            if (lane == 0) mbar_expect_tx(&bars[w][stage], rows * row_bytes);
            __syncwarp();
            if (ok)
                bulk_g2s(my + (size_t)stage * kPullStageBytes + (size_t)lane * row_bytes, store + row * row_bytes,
                         row_bytes, &bars[w][stage]);
        }
        if (have_prev && !finish(stage ^ 1)) return;
        prev_t0 = t0; prev_rows = rows; prev_mine = ok; have_prev = true;
        stage ^= 1;
    }
    if (have_prev && !finish(stage ^ 1)) return;
    bulk_wait_read<0>();
}

// One warp gathers kRows rows at a time so that several independent 128-bit
// loads are in flight per lane (rows too long for the staged kernel above).
template <int kRows>
__global__ void __launch_bounds__(256)
pull_kernel(const uint64_t* __restrict__ keys, uint64_t n, float4* __restrict__ out,
            const float4* __restrict__ store, const uint2* __restrict__ table, uint64_t S, uint64_t K,
            uint32_t L4, DevStatus* st, unsigned int epoch) {
    const int lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t n_warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    for (uint64_t t0 = warp * kRows; t0 < n; t0 += n_warps * kRows) {
        uint64_t row[kRows];
        bool ok[kRows];
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            ok[r] = false;
            row[r] = 0;
            if (t0 + r < n) {
                const uint64_t key = keys[t0 + r];
                if (key < K) {
                    row[r] = phys_row(table[key], S);
                    ok[r] = true;
                } else if (lane == 0) {
                    latch_error(st, epoch, PS_ERR_KEY_RANGE);
                }
            }
        }
        for (uint32_t f = lane; f < L4; f += 32) {
            float4 v[kRows];
#pragma unroll
            for (int r = 0; r < kRows; ++r)
                v[r] = ok[r] ? __ldg(store + row[r] * L4 + f) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int r = 0; r < kRows; ++r)
                if (t0 + r < n) __stcs(out + (t0 + r) * L4 + f, v[r]);
        }
    }
}

void launch_pull(ps_store* ps, const uint64_t* d_keys, uint64_t n, float* d_out, cudaStream_t s) {
    const uint32_t row_bytes = ps->cfg.row_len * 4;
    if (row_bytes <= kPullStageBytes) {
        static std::atomic<unsigned long long> smem_set{0};
        opt_in_smem((const void*)pull_bulk_kernel, kPullSmem, &smem_set);
        const uint32_t per_round = tmin<uint32_t>(32u, kPullStageBytes / row_bytes);
        const uint64_t rounds = (n + per_round - 1) / per_round;
        const uint32_t grid = (uint32_t)tmin<uint64_t>((rounds + 7) / 8, (uint64_t)ps->sm_count * 3);
        PS_LAUNCH_SMEM(ps, pull_bulk_kernel, grid, 256, kPullSmem, s, d_keys, n, (char*)d_out, (const char*)ps->store,
                       ps->table, ps->cfg.slots_per_part, ps->cfg.num_keys, row_bytes, per_round, ps->status, 0u);
        return;
    }
    const uint32_t grid = (uint32_t)tmin<uint64_t>((n + 31) / 32, (uint64_t)ps->sm_count * 8);
    PS_LAUNCH(ps, pull_kernel<4>, grid, 256, s, d_keys, n, (float4*)d_out, (const float4*)ps->store, ps->table,
              ps->cfg.slots_per_part, ps->cfg.num_keys, ps->cfg.row_len / 4, ps->status, 0u);
}

// rows of keys first_key .. first_key + n, in key order (export)
__global__ void __launch_bounds__(256)
gather_by_key_kernel(uint64_t first_key, uint64_t n, float4* __restrict__ out, const float4* __restrict__ store,
                     const uint2* __restrict__ table, uint64_t S, uint32_t L4) {
    const int lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t n_warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    for (uint64_t t = warp; t < n; t += n_warps) {
        const uint64_t row = phys_row(table[first_key + t], S);
        for (uint32_t f = lane; f < L4; f += 32) out[t * L4 + f] = store[row * L4 + f];
    }
}

void launch_gather_rows_by_key(ps_store* ps, uint64_t first_key, uint64_t n, float* d_out, cudaStream_t s) {
    const uint32_t grid = (uint32_t)tmin<uint64_t>((n + 7) / 8, (uint64_t)ps->sm_count * 8);
    PS_LAUNCH(ps, gather_by_key_kernel, grid, 256, s, first_key, n, (float4*)d_out, (const float4*)ps->store,
              ps->table, ps->cfg.slots_per_part, ps->cfg.row_len / 4);
}

__global__ void get_location_kernel(const uint64_t* __restrict__ keys, uint64_t n, uint32_t* __restrict__ owner,
                                    uint32_t* __restrict__ slot, const uint2* __restrict__ table, uint64_t K,
                                    DevStatus* st, unsigned int epoch) {
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n) return;
    const uint64_t key = keys[t];
    if (key >= K) {
        latch_error(st, epoch, PS_ERR_KEY_RANGE);
        owner[t] = kSentinelPad;
        slot[t] = kSentinelPad;
        return;
    }
    const uint2 e = table[key];
    owner[t] = e.x;
    slot[t] = e.y;
}

void launch_get_location(ps_store* ps, const uint64_t* d_keys, uint64_t n, uint32_t* d_owner, uint32_t* d_slot,
                         cudaStream_t s) {
    PS_LAUNCH(ps, get_location_kernel, div_up_u32(n, 256), 256, s, d_keys, n, d_owner, d_slot, ps->table,
              ps->cfg.num_keys, ps->status, 0u);
}

// ---------------------------------------------------------------- push ----
__global__ void prepare_keys_kernel(const uint64_t* __restrict__ keys, uint64_t n, uint32_t* __restrict__ out,
                                    uint64_t K, DevStatus* st, unsigned int epoch) {
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n) return;
    const uint64_t key = keys[t];
    if (key >= K) {
        latch_error(st, epoch, PS_ERR_KEY_RANGE);
        out[t] = (uint32_t)K;
    } else {
        out[t] = (uint32_t)key;
    }
}

void launch_prepare_keys(ps_store* ps, const uint64_t* d_keys, uint64_t n, cudaStream_t s) {
    PS_LAUNCH(ps, prepare_keys_kernel, div_up_u32(n, 256), 256, s, d_keys, n, ps->keysA, ps->cfg.num_keys,
              ps->status, ps->epoch);
}

struct d4 {
    double x, y, z, w;
};

// Staging of the reduction kernel for rows of up to kCh column blocks (32 float4 each): positions whose
// copies are asked for together, and groups in flight per warp.  A position takes 2 x kCh x 512 bytes (update
// row and target row); a warp stages 6 KB (8 KB for kCh = 4), so four (three) blocks of 8 warps fit an SM.
__host__ __device__ constexpr int reduce_group(int kCh) { return kCh == 1 ? 2 : 1; }
__host__ __device__ constexpr int reduce_stages(int kCh) { return kCh <= 2 ? 3 : 2; }
__host__ __device__ constexpr size_t reduce_smem(int kCh) {
    return (size_t)8 * reduce_stages(kCh) * reduce_group(kCh) * 2 * kCh * 32 * sizeof(float4);
}
static_assert(reduce_smem(1) >= 8 * 32 * 32 && reduce_smem(4) <= 64 * 1024, "staging also serves as the pre-add scratch");
constexpr int kFixupWarps = 8;
constexpr int kGroupMinSpan = 8 * kReduceTile;   // a group's entering segment is pre-added only if at least this long
constexpr int kGroupTiles = 64;     // tiles whose parked parts are pre-added per group (8 reduction blocks)

// Tail of the reduction kernel, kept out of line so that it does not weigh on the main loop's registers.
// The last block to finish in an aligned group of 64 tiles adds up, once, the parked parts of the (long)
// segment that enters the group from the group before; the fix-up kernel then needs one value per group
// for a segment that runs through thousands of tiles (a hot key), instead of one per tile.
__device__ __noinline__ void group_preadd(const uint32_t* __restrict__ sk, uint32_t n, uint32_t L4,
                                          const double* __restrict__ carry, unsigned int* __restrict__ group_done,
                                          double* __restrict__ group_sum, uint32_t group, uint64_t gpos, uint32_t kg,
                                          d4 (*gpart)[32], unsigned int* s_ticket, uint32_t tile_len,
                                          uint32_t arrivals) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t L = L4 * 4;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) *s_ticket = atomicAdd(&group_done[group], 1u);
    __syncthreads();
    if (*s_ticket != arrivals - 1) return;              // `arrivals` blocks work on the group's tiles
    __threadfence();
    // tiles of the group that begin with the entering segment's key: a prefix of the group's tiles
    const uint64_t tpos = gpos + (uint64_t)threadIdx.x * tile_len;
    const int hit = threadIdx.x < kGroupTiles && tpos < n && sk[tpos] == kg;
    const uint32_t m = (uint32_t)__syncthreads_count(hit);
    const uint32_t t0 = group * kGroupTiles;
    for (uint32_t f0 = 0; f0 < L4; f0 += 32) {
        const uint32_t f = f0 + lane;
        const bool act = f < L4;
        d4 a = {0.0, 0.0, 0.0, 0.0};
        if (act) {
#pragma unroll 4
            for (uint32_t t = w; t < m; t += 8) {
                const double* c2 = carry + ((uint64_t)(t0 + t) * 2) * L + (uint64_t)f * 4;
                const double2 x = __ldcg((const double2*)c2), y = __ldcg((const double2*)(c2 + 2));
                a.x += x.x; a.y += x.y; a.z += y.x; a.w += y.y;
            }
        }
        gpart[w][lane] = a;
        __syncthreads();
        if (w == 0 && act) {
            d4 t = gpart[0][lane];
#pragma unroll
            for (int i = 1; i < 8; ++i) {
                t.x += gpart[i][lane].x; t.y += gpart[i][lane].y; t.z += gpart[i][lane].z; t.w += gpart[i][lane].w;
            }
            double* g = group_sum + (uint64_t)group * L + (uint64_t)f * 4;
            *(double2*)g = make_double2(t.x, t.y);
            *(double2*)(g + 2) = make_double2(t.z, t.w);
        }
        __syncthreads();
    }
}

// A warp owns sorted positions [tile*32, tile*32+32).  A segment (run of equal
// keys) that starts and ends inside the tile is summed in fp64 and applied with
// one read-modify-write of its row; a segment that continues from the previous
// tile parks its partial sum in carry slot 0 of the tile, one that continues
// into the next tile in slot 1, and the tile that starts such a segment is
// appended to the list the fix-up kernel works through.
// Every lane looks up the row of its own position's key, so the 32 table reads
// go out together; then the positions are walked in groups whose update rows
// and target rows are all requested before the first is used.
//
// kScaled: occurrence o does not have an update row of its own.  Its update is scales[o] times a source
// row shared with other occurrences: the occurrences come in runs of `slots` per example, example e owning
// source rows 2e (used, by its slot 0) and 2e + 1 (used by all its other slots) of `upd`.
//
// kL4 / kSlots: the row length in float4 and the slots per example if known at compile time (0: taken from the
// arguments); row offsets, the copy size and the division by the slots then fold.
template <int kCh, bool kScaled, int kL4, int kSlots>
__global__ void __launch_bounds__(256)
push_reduce_kernel(const uint32_t* __restrict__ sk, const uint32_t* __restrict__ sv, uint32_t n,
                   const float4* __restrict__ upd, const float* __restrict__ scales, uint32_t slots_arg,
                   float4* __restrict__ store, const uint2* __restrict__ table,
                   uint64_t S, uint32_t K, uint32_t L4_arg, double* __restrict__ carry,
                   uint4* __restrict__ starters, unsigned int* __restrict__ starter_count,
                   unsigned int* __restrict__ group_done, double* __restrict__ group_sum,
                   DevStatus* st, unsigned int epoch) {
    __shared__ unsigned int s_ticket;
    __shared__ __align__(8) uint64_t bars[8][3];    // per warp and stage: the barrier word its copies report to
    const uint32_t L4 = kL4 ? (uint32_t)kL4 : L4_arg;
    const uint32_t slots = kSlots ? (uint32_t)kSlots : slots_arg;
    if (call_failed(st, epoch)) return;
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const uint32_t tile = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t base = (uint64_t)tile * kReduceTile;
    const uint32_t n_valid = base < n ? (uint32_t)tmin<uint64_t>((uint64_t)kReduceTile, n - base) : 0u;
    const uint32_t key = lane < n_valid ? sk[base + lane] : kSentinelPad;
    uint32_t occ = lane < n_valid ? sv[base + lane] : 0u;
    const bool usable = key < K;                    // "no key" marks and padding sort last
    float scale = 1.f;
    if (kScaled && usable) {
        scale = scales[occ];
        const uint32_t e = occ / slots;
        occ = 2u * e + (occ != e * slots ? 1u : 0u);
    }
    uint64_t row = 0;
    if (usable) row = phys_row(table[key], S);
    uint32_t prev = __shfl_up_sync(full, key, 1);
    if (lane == 0) prev = (base > 0 && base - 1 < n) ? sk[base - 1] : kSentinelPad;
    const uint32_t next_after = (base + kReduceTile < n) ? sk[base + kReduceTile] : kSentinelPad;
    uint32_t next = __shfl_down_sync(full, key, 1);
    if (lane == 31) next = next_after;
    const unsigned head_mask = __ballot_sync(full, key != prev);
    const unsigned usable_mask = __ballot_sync(full, usable);
    // positions at which a segment's part in this tile ends: its true end, or the tile's last position
    const unsigned end_mask = __ballot_sync(full, usable && (key != next || lane == 31));
    // positions before the first head belong to a segment that came in from the previous tile
    const int first_head = head_mask ? (__ffs(head_mask) - 1) : 32;
    // the last segment runs on iff the position after the tile holds the same usable key
    const uint32_t key31 = __shfl_sync(full, key, 31);
    const bool runs_on = key31 < K && next_after == key31;
    // a border-crossing segment starts in this tile iff it runs on and has its head here
    if (runs_on && head_mask != 0u && lane == 31)
        starters[atomicAdd(starter_count, 1u)] = make_uint4(tile, key, (uint32_t)row, (uint32_t)(row >> 32));
    // does a segment enter this block's group of 64 tiles from the group before?  (asked here, with the
    // walk's loads still to come, and needed only after the walk)
    const uint32_t group = blockIdx.x / (kGroupTiles / 8);
    const uint64_t gpos = (uint64_t)group * kGroupTiles * kReduceTile;     // first sorted position of the group
    // Only a segment that also covers the group's first kGroupMinSpan positions is worth it: shorter ones
    // end within a few tiles and the fix-up kernel takes those tile by tile.
    uint32_t kg = kSentinelPad, kg_prev = kSentinelPad - 1, kg_far = kSentinelPad - 2;
    if (gpos > 0 && gpos + kGroupMinSpan - 1 < n) {
        kg = sk[gpos];
        kg_prev = sk[gpos - 1];
        kg_far = sk[gpos + kGroupMinSpan - 1];
    }
    const uint32_t L = L4 * 4;
    // Rows are staged through shared memory with bulk asynchronous copies: for a group of G positions the
    // lane that owns a position asks for its whole update row and, where a segment ends, for the target row
    // (one instruction each for the whole group), the copies report to a barrier word of the warp's own,
    // and ST groups are kept in flight per warp.
    constexpr int G = reduce_group(kCh), ST = reduce_stages(kCh);
    constexpr int kSlotF4 = 2 * G * kCh * 32;                   // float4s of one stage of one warp
    extern __shared__ float4 stage_mem[];
    const int w = threadIdx.x >> 5;
    float4* my_stage = stage_mem + (size_t)w * (ST * kSlotF4);
    if (lane < ST) mbar_init(&bars[w][lane], 1);
    mbar_init_fence();
    __syncwarp();
    const int n_groups = ((int)n_valid + G - 1) / G;
    // positions whose target row is fetched: a segment ends there and is neither parked on the way in nor out
    const bool fetch_me = usable && (key != next || lane == 31) && !(lane < first_head || (lane == 31 && runs_on));
    const unsigned fetch_mask = __ballot_sync(full, fetch_me);
    const unsigned gmask0 = G == 32 ? full : ((1u << G) - 1u);
    uint32_t uses = 0;                                          // how often the warp has waited so far, per stage: parity
    bool dead = false;
    for (uint32_t f0 = 0; f0 < L4 && !dead; f0 += 32 * kCh) {   // one round unless a row is longer than 128 kCh floats
        const uint32_t chunk4 = tmin<uint32_t>(L4 - f0, 32u * kCh);
        const uint32_t chunk_bytes = chunk4 * 16u;
        const uint32_t fl = f0 + lane;
        auto issue = [&](int g, int stage) {
            if (g >= n_groups) return;
            const unsigned gm = gmask0 << (g * G);
            const uint32_t n_rows = __popc(usable_mask & gm) + __popc(fetch_mask & gm);
            if (n_rows == 0) return;                            // nothing to wait for either: see the walk
            if (lane == g * G) mbar_expect_tx(&bars[w][stage], n_rows * chunk_bytes);
            __syncwarp();
            if ((gm >> lane) & 1u) {
                float4* dst = my_stage + (size_t)stage * kSlotF4 + (size_t)(lane - g * G) * (2 * kCh * 32);
                if (usable) bulk_g2s(dst, upd + (uint64_t)occ * L4 + f0, chunk_bytes, &bars[w][stage]);
                if (fetch_me) bulk_g2s(dst + kCh * 32, store + row * L4 + f0, chunk_bytes, &bars[w][stage]);
            }
        };
#pragma unroll
        for (int g = 0; g < ST - 1; ++g) issue(g, g);
        d4 acc[kCh];
#pragma unroll
        for (int c = 0; c < kCh; ++c) acc[c] = d4{0.0, 0.0, 0.0, 0.0};
        int st_use = 0, st_fill = ST - 1;
        for (int g = 0; g < n_groups; ++g) {
            __syncwarp();                                       // every lane is done reading the stage to be refilled
            issue(g + ST - 1, st_fill);
            const unsigned gm = gmask0 << (g * G);
            const float4* slot = my_stage + (size_t)st_use * kSlotF4 + lane;
            if (usable_mask & gm) {
                const uint32_t parity = (uses >> st_use) & 1u;
                if (!mbar_wait(&bars[w][st_use], parity) && !mbar_wait(&bars[w][st_use], parity)) {
                    if (lane == 0) latch_error(st, epoch, PS_ERR_CUDA);
                    dead = true;                                // a copy that does not arrive: give the call up
                    break;
                }
                uses ^= 1u << st_use;
            }
            st_use = st_use + 1 == ST ? 0 : st_use + 1;
            st_fill = st_fill + 1 == ST ? 0 : st_fill + 1;
#pragma unroll
            for (int k = 0; k < G; ++k) {
                const int p = g * G + k;
                const float sc = kScaled ? __shfl_sync(full, scale, p) : 1.f;
                if (!((usable_mask >> p) & 1u)) continue;
                // A segment of exactly one occurrence needs no fp64 sum: row + update (one fused multiply-add if
                // the update is a factor times a source row) rounds the exact sum once, and the conversions to
                // and from fp64, which share a pipe with little throughput, are not issued.
                if ((((head_mask & fetch_mask) >> p) & 1u)) {
                    const uint64_t rw1 = __shfl_sync(full, row, p);
#pragma unroll
                    for (int c = 0; c < kCh; ++c) {
                        if (fl + 32 * c >= L4) continue;
                        const float4 u = slot[(k * 2 * kCh + c) * 32];
                        float4 v = slot[(k * 2 * kCh + kCh + c) * 32];
                        if (kScaled) {
                            v.x = fmaf(sc, u.x, v.x); v.y = fmaf(sc, u.y, v.y);
                            v.z = fmaf(sc, u.z, v.z); v.w = fmaf(sc, u.w, v.w);
                        } else {
                            v.x += u.x; v.y += u.y; v.z += u.z; v.w += u.w;
                        }
                        store[rw1 * L4 + fl + 32 * c] = v;
                    }
                    continue;
                }
                const double d = (double)sc;
#pragma unroll
                for (int c = 0; c < kCh; ++c) {
                    if (fl + 32 * c >= L4) continue;
                    const float4 u = slot[(k * 2 * kCh + c) * 32];
                    if (kScaled) {
                        acc[c].x += d * (double)u.x; acc[c].y += d * (double)u.y;
                        acc[c].z += d * (double)u.z; acc[c].w += d * (double)u.w;
                    } else {
                        acc[c].x += (double)u.x; acc[c].y += (double)u.y;
                        acc[c].z += (double)u.z; acc[c].w += (double)u.w;
                    }
                }
                if (!((end_mask >> p) & 1u)) continue;
                const uint64_t rw = __shfl_sync(full, row, p);
                const bool from_prev = p < first_head;
                const bool parked = from_prev || (p == 31 && runs_on);
#pragma unroll
                for (int c = 0; c < kCh; ++c) {
                    const uint32_t f = fl + 32 * c;
                    if (f < L4) {
                        if (!parked) {
                            float4 v = slot[(k * 2 * kCh + kCh + c) * 32];
                            v.x = (float)((double)v.x + acc[c].x); v.y = (float)((double)v.y + acc[c].y);
                            v.z = (float)((double)v.z + acc[c].z); v.w = (float)((double)v.w + acc[c].w);
                            store[rw * L4 + f] = v;
                        } else {
                            double* cs = carry + ((uint64_t)tile * 2 + (from_prev ? 0 : 1)) * L + (uint64_t)f * 4;
                            *(double2*)cs = make_double2(acc[c].x, acc[c].y);
                            *(double2*)(cs + 2) = make_double2(acc[c].z, acc[c].w);
                        }
                    }
                    acc[c] = d4{0.0, 0.0, 0.0, 0.0};
                }
            }
        }
        __syncwarp();
    }
    if (!(kg < K && kg_prev == kg && kg_far == kg)) return;     // nothing to pre-add for this group
    // the staging memory is free by now (every warp has waited for all its copies) and serves as scratch
    group_preadd(sk, n, L4, carry, group_done, group_sum, group, gpos, kg, reinterpret_cast<d4 (*)[32]>(stage_mem),
                 &s_ticket, kReduceTile, tmin<uint32_t>(kGroupTiles / 8, gridDim.x - group * (kGroupTiles / 8)));
}

// ------------------------------------------------- ComplEx: AdaGrad inside the reduction ----
// The reduction of a ComplEx step whose update rows are GRADIENTS (2 d values per occurrence, Re then Im,
// written by kge_step_kernel<.., kGradOnly>), not finished steps.  AdaGrad is taken per data point from the
// accumulators as they were before the batch (Appendix A of the paper stores them in the PS, next to the
// embedding): an occurrence with gradient g adds (-lr g / (sqrt(G + g^2) + eps), g^2) to its key's row
// [Re | Im | G_Re | G_Im].  So where a part of a segment begins the warp fetches the key's row and keeps embedding
// and accumulators in registers; every position then needs only its gradient row, half the bytes of a finished
// update row, and the step kernel neither loads accumulators nor evaluates square roots.  The sums, the
// parked partials of parts that cross tile borders (laid out like the row: steps, then squared gradients) and
// the fix-up launch are those of push_reduce_kernel; the arithmetic per occurrence is the same fp32 expression
// the step kernel used, so results do not change.  kC: float4 of a gradient row per lane (d <= 64 kC).
template <int kC>
__global__ void __launch_bounds__(256, 3)
kge_reduce_kernel(const uint32_t* __restrict__ sk, const uint32_t* __restrict__ sv, uint32_t n,
                  const float4* __restrict__ grad, float4* __restrict__ store, const uint2* __restrict__ table,
                  uint64_t S, uint32_t K, uint32_t G4, float lr, float eps, double* __restrict__ carry,
                  uint4* __restrict__ starters, unsigned int* __restrict__ starter_count,
                  unsigned int* __restrict__ group_done, double* __restrict__ group_sum, DevStatus* st,
                  unsigned int epoch) {
    __shared__ unsigned int s_ticket;
    __shared__ __align__(8) uint64_t bars[8][2];
    extern __shared__ float4 stage_mem[];
    if (call_failed(st, epoch)) return;
    constexpr int kST = 2;
    constexpr int kSlotF4 = 3 * kC * 32;            // one position: gradient row, then the key's whole row
    const uint32_t L4 = 2 * G4;                     // float4 of a row: embedding (G4), accumulators (G4)
    const uint32_t L = L4 * 4;
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t tile = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t base = (uint64_t)tile * kReduceTile;
    const uint32_t n_valid = base < n ? (uint32_t)tmin<uint64_t>((uint64_t)kReduceTile, n - base) : 0u;
    const uint32_t key = lane < n_valid ? sk[base + lane] : kSentinelPad;
    const uint32_t occ = lane < n_valid ? sv[base + lane] : 0u;
    const bool usable = key < K;
    uint64_t row = 0;
    if (usable) row = phys_row(table[key], S);
    uint32_t prev = __shfl_up_sync(full, key, 1);
    if (lane == 0) prev = (base > 0 && base - 1 < n) ? sk[base - 1] : kSentinelPad;
    const uint32_t next_after = (base + kReduceTile < n) ? sk[base + kReduceTile] : kSentinelPad;
    uint32_t next = __shfl_down_sync(full, key, 1);
    if (lane == 31) next = next_after;
    const unsigned head_mask = __ballot_sync(full, key != prev);
    const unsigned usable_mask = __ballot_sync(full, usable);
    const unsigned end_mask = __ballot_sync(full, usable && (key != next || lane == 31));
    const int first_head = head_mask ? (__ffs(head_mask) - 1) : 32;
    const uint32_t key31 = __shfl_sync(full, key, 31);
    const bool runs_on = key31 < K && next_after == key31;
    if (runs_on && head_mask != 0u && lane == 31)
        starters[atomicAdd(starter_count, 1u)] = make_uint4(tile, key, (uint32_t)row, (uint32_t)(row >> 32));
    const bool begin_me = usable && (lane == 0 || key != prev);     // the key's row is fetched here
    const unsigned begin_mask = __ballot_sync(full, begin_me);
    const uint32_t group = blockIdx.x / (kGroupTiles / 8);
    const uint64_t gpos = (uint64_t)group * kGroupTiles * kReduceTile;
    uint32_t kg = kSentinelPad, kg_prev = kSentinelPad - 1, kg_far = kSentinelPad - 2;
    if (gpos > 0 && gpos + kGroupMinSpan - 1 < n) {
        kg = sk[gpos];
        kg_prev = sk[gpos - 1];
        kg_far = sk[gpos + kGroupMinSpan - 1];
    }
    float4* my_stage = stage_mem + (size_t)w * (kST * kSlotF4);
    if (lane < kST) mbar_init(&bars[w][lane], 1);
    mbar_init_fence();
    __syncwarp();
    const uint32_t grad_bytes = G4 * 16u, row_bytes = L4 * 16u;
    auto issue = [&](int p, int stage) {
        if (p >= (int)n_valid || !((usable_mask >> p) & 1u)) return;
        const bool b = (begin_mask >> p) & 1u;
        if (lane == p) {
            mbar_expect_tx(&bars[w][stage], grad_bytes + (b ? row_bytes : 0u));
            float4* dst = my_stage + (size_t)stage * kSlotF4;
            bulk_g2s(dst, grad + (uint64_t)occ * G4, grad_bytes, &bars[w][stage]);
            if (b) bulk_g2s(dst + kC * 32, store + row * L4, row_bytes, &bars[w][stage]);
        }
    };
    issue(0, 0);
    d4 acc_t[kC], acc_g[kC];
    float4 th[kC], Gv[kC];
#pragma unroll
    for (int c = 0; c < kC; ++c) {
        acc_t[c] = acc_g[c] = d4{0.0, 0.0, 0.0, 0.0};
        th[c] = Gv[c] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    uint32_t uses = 0;
    for (int p = 0; p < (int)n_valid; ++p) {
        const int stg = p & 1;
        __syncwarp();                               // every lane is done reading the stage to be refilled
        issue(p + 1, stg ^ 1);
        if (!((usable_mask >> p) & 1u)) continue;
        const uint32_t parity = (uses >> stg) & 1u;
        if (!mbar_wait(&bars[w][stg], parity) && !mbar_wait(&bars[w][stg], parity)) {
            if (lane == 0) latch_error(st, epoch, PS_ERR_CUDA);
            break;                                  // a copy that does not arrive: give the call up
        }
        uses ^= 1u << stg;
        const float4* slot = my_stage + (size_t)stg * kSlotF4;
        if ((begin_mask >> p) & 1u) {
#pragma unroll
            for (int c = 0; c < kC; ++c) {
                const uint32_t f = lane + 32 * c;
                if (f < G4) {
                    th[c] = slot[kC * 32 + f];
                    Gv[c] = slot[kC * 32 + G4 + f];
                }
                acc_t[c] = acc_g[c] = d4{0.0, 0.0, 0.0, 0.0};
            }
        }
        // A segment of exactly one occurrence (most keys of a batch) needs no fp64 sum: row + update in fp32 rounds
        // the same exact sum once, and the conversions, which share a pipe with the square roots and reciprocals
        // that bounds this kernel, are not issued.
        if (((begin_mask & end_mask) >> p) & 1u && p >= first_head && !(p == 31 && runs_on)) {
            const uint64_t rw = __shfl_sync(full, row, p);
#pragma unroll
            for (int c = 0; c < kC; ++c) {
                const uint32_t f = lane + 32 * c;
                if (f >= G4) continue;
                const float4 g = slot[f];
                const float qx = g.x * g.x, qy = g.y * g.y, qz = g.z * g.z, qw = g.w * g.w;
                float4 t = th[c], a = Gv[c];
                t.x += adagrad_step(g.x, a.x + qx, lr, eps); t.y += adagrad_step(g.y, a.y + qy, lr, eps);
                t.z += adagrad_step(g.z, a.z + qz, lr, eps); t.w += adagrad_step(g.w, a.w + qw, lr, eps);
                a.x += qx; a.y += qy; a.z += qz; a.w += qw;
                store[rw * L4 + f] = t;
                store[rw * L4 + G4 + f] = a;
            }
            continue;
        }
#pragma unroll
        for (int c = 0; c < kC; ++c) {
            const uint32_t f = lane + 32 * c;
            if (f >= G4) continue;
            const float4 g = slot[f];
            const float qx = g.x * g.x, qy = g.y * g.y, qz = g.z * g.z, qw = g.w * g.w;
            acc_t[c].x += (double)adagrad_step(g.x, Gv[c].x + qx, lr, eps);
            acc_t[c].y += (double)adagrad_step(g.y, Gv[c].y + qy, lr, eps);
            acc_t[c].z += (double)adagrad_step(g.z, Gv[c].z + qz, lr, eps);
            acc_t[c].w += (double)adagrad_step(g.w, Gv[c].w + qw, lr, eps);
            acc_g[c].x += (double)qx; acc_g[c].y += (double)qy; acc_g[c].z += (double)qz; acc_g[c].w += (double)qw;
        }
        if (!((end_mask >> p) & 1u)) continue;
        const uint64_t rw = __shfl_sync(full, row, p);
        const bool from_prev = p < first_head;
        const bool parked = from_prev || (p == 31 && runs_on);
#pragma unroll
        for (int c = 0; c < kC; ++c) {
            const uint32_t f = lane + 32 * c;
            if (f >= G4) continue;
            if (!parked) {
                float4 t = th[c], a = Gv[c];
                t.x = (float)((double)t.x + acc_t[c].x); t.y = (float)((double)t.y + acc_t[c].y);
                t.z = (float)((double)t.z + acc_t[c].z); t.w = (float)((double)t.w + acc_t[c].w);
                a.x = (float)((double)a.x + acc_g[c].x); a.y = (float)((double)a.y + acc_g[c].y);
                a.z = (float)((double)a.z + acc_g[c].z); a.w = (float)((double)a.w + acc_g[c].w);
                store[rw * L4 + f] = t;
                store[rw * L4 + G4 + f] = a;
            } else {
                double* cs = carry + ((uint64_t)tile * 2 + (from_prev ? 0 : 1)) * L;
                double* ct = cs + (uint64_t)f * 4;
                double* cg = cs + (uint64_t)(G4 + f) * 4;
                *(double2*)ct = make_double2(acc_t[c].x, acc_t[c].y);
                *(double2*)(ct + 2) = make_double2(acc_t[c].z, acc_t[c].w);
                *(double2*)cg = make_double2(acc_g[c].x, acc_g[c].y);
                *(double2*)(cg + 2) = make_double2(acc_g[c].z, acc_g[c].w);
            }
        }
    }
    __syncwarp();
    if (!(kg < K && kg_prev == kg && kg_far == kg)) return;     // nothing to pre-add for this group
    __syncthreads();                                // the staging memory serves as scratch from here on
    group_preadd(sk, n, L4, carry, group_done, group_sum, group, gpos, kg, reinterpret_cast<d4 (*)[32]>(stage_mem),
                 &s_ticket, kReduceTile, tmin<uint32_t>(kGroupTiles / 8, gridDim.x - group * (kGroupTiles / 8)));
}

// ------------------------------------------------- MF: gradient inside the reduction ----
// One minibatch of matrix factorization without update rows.  The occurrences (2t: row factor of cell t,
// 2t + 1: its column factor) arrive sorted by key, as for a push, each with a record {cell, value of the
// cell, row of the key, row of the cell's other factor} written by the sort.  For every sorted position
// the PARTNER row (the other factor) is fetched and, where a segment's part in a tile begins, the key's
// own row; e = v - <own, partner> is formed on the spot and lr (e partner - lambda own) is added to the
// segment's sum.
//
// The kernel is bound by instruction issue, not by memory, if a whole warp works on one position (a row
// of 100 values keeps 25 lanes busy for one instruction while the bookkeeping of the position costs
// dozens).  So a position is handled by EIGHT lanes: a warp covers 32 consecutive positions as four tiles
// of kMfTile = 8 positions, one per group of eight lanes, and every instruction of the walk serves four
// positions.  A lane holds every eighth float4 of a row.  Tiles of eight positions are the unit of the
// border logic: a segment's part that crosses a tile border parks its fp64 partial sum (slot 0 of the tile
// it enters, slot 1 of the tile it leaves) and the fix-up launch adds the parts up, as for a push.
// A segment of exactly one position needs no fp64 sum: own + update is formed in fp32, which rounds the
// same exact sum once.
//
// Nothing may overwrite a row that another position still reads, so new rows are left in `staged` (indexed by
// the sorted position where the segment ends) with the row's address in `apply_row`, and the fix-up launch,
// which runs after every read of this kernel, moves them into the store.  One case needs neither staging nor a
// segment: a row factor whose key occurs ONCE in the batch (nearly all of them, rows being drawn uniformly) is
// read by exactly one position, the column-factor occurrence of its cell, as the partner.  That position has
// both rows in hand; it forms the row factor's new row too and writes it in place, and the row factor's own
// position is skipped together with its two row fetches.  The loss of a cell is taken where its row factor
// is updated.
constexpr int kMfTile = 8;
constexpr int kMfStages = 3;
constexpr size_t kMfSmem = (size_t)8 * kMfStages * 4 * 64 * sizeof(float4) + 128;   // warp x stage x group x {partner, own}; room to align

enum : uint32_t { kFUsable = 1, kFBegin = 2, kFEnd = 4, kFParked = 8, kFFromPrev = 16, kFBoth = 32, kFSingle = 64,
                  kFColumn = 128 };

// kG4: the four partner rows of a walk step (one per group of eight lanes) are fetched by ONE instruction of the TMA
// unit (tile::gather4 on the store seen as a 2-D tensor of rows) instead of four bulk copies: 0.6 M fewer warp
// instructions per launch on the 10M x 1M matrix, 1.5 us of 45 per step.  (The walk is bound by its own instructions
// and by its scattered row writes: with no row copies at all it takes 8.0 of its 10.4 us.)  A stage of a warp is then
// laid out as {four partner rows, one after the other | four own rows of 512 bytes}.
template <int kC, bool kG4>
__global__ void __launch_bounds__(256, 2)
mf_sub_kernel(const __grid_constant__ CUtensorMap row_map, const uint32_t* __restrict__ sk, const uint4* __restrict__ rec,
              const uint32_t* __restrict__ cellpos, uint32_t n,
              uint32_t col_base, float lr, float lam, float4* store, uint32_t K,
              uint32_t L4, float4* __restrict__ staged, uint64_t* __restrict__ apply_row, double* __restrict__ carry,
              uint4* __restrict__ starters, unsigned int* __restrict__ starter_count,
              unsigned int* __restrict__ group_done, double* __restrict__ group_sum,
              double* __restrict__ loss_partial, DevStatus* st, unsigned int epoch) {
    __shared__ unsigned int s_ticket;
    __shared__ __align__(8) uint64_t bars[8][kMfStages];
    __shared__ double wl[8];
    extern __shared__ float4 stage_mem[];
    if (call_failed(st, epoch)) return;
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int sg = lane >> 3, l8 = lane & 7;
    // The row side comes first in key order (one occurrence per cell: the first half of the positions) and its
    // blocks find almost only positions that the column side handles.  The blocks are taken from the middle on, so
    // that the column side is placed first, its most frequent keys (whose groups need a pre-added value) before
    // the rest, and the short blocks of the row side fill in as places come free.
    const uint32_t gb = (blockIdx.x + (n / 2) / 256) % gridDim.x;
    const uint32_t tile32 = gb * 8 + w;
    const uint64_t base = (uint64_t)tile32 * 32;
    const uint64_t pos = base + lane;
    const bool inside = pos < n;
    // {cell, value of the cell, row of the key, row of the cell's other factor}, written by the sort's last pass
    const uint4 me = inside ? rec[pos] : make_uint4(0u, 0u, 0u, 0u);
    const uint32_t key = inside ? sk[pos] : kSentinelPad;
    const float val = __uint_as_float(me.y);
    const uint32_t row = me.z, prow = me.w;
    uint32_t prev = __shfl_up_sync(full, key, 1);
    if (lane == 0) prev = (base > 0 && base - 1 < n) ? sk[base - 1] : kSentinelPad;
    uint32_t next = __shfl_down_sync(full, key, 1);
    if (lane == 31) next = (base + 32 < n) ? sk[base + 32] : kSentinelPad;
    const bool head = key != prev;
    // A row factor whose key occurs once in the batch is read by exactly one position of the column side (its
    // cell's), as the partner.  That position has both rows in hand, so it also forms the row factor's new row and
    // writes it in place; the row side then skips the position, and its two row fetches.
    bool both = false;                              // column side: this position also updates its partner
    bool usable = key < K;
    const bool row_side = key < col_base;
    if (row_side) {
        if (usable && head && key != next) usable = false;
    } else if (usable) {
        const uint32_t pp = cellpos[me.x];          // sorted position of the cell's row-factor occurrence
        const uint32_t kp = sk[pp];
        const uint32_t kl = pp > 0 ? sk[pp - 1] : kSentinelPad, kr = pp + 1 < n ? sk[pp + 1] : kSentinelPad;
        both = kl != kp && kr != kp;
    }
    const unsigned head_mask = __ballot_sync(full, head);
    const unsigned usable_mask = __ballot_sync(full, usable);
    // the head of this position's segment, if it lies in the warp's 32 positions
    const unsigned at_or_below = head_mask & (0xffffffffu >> (31 - lane));
    const int seg_head = at_or_below ? 31 - __clz(at_or_below) : -1;
    const bool from_prev = usable && seg_head < 8 * sg;             // the segment came in from an earlier tile
    const bool begin_me = usable && (l8 == 0 || head);              // the own row is fetched here
    const bool end_me = usable && (l8 == 7 || key != next);         // the segment's part in the tile ends here
    const bool runs_on = end_me && key == next;                     // ... and goes on in the next tile
    const bool parked = end_me && (from_prev || runs_on);
    const bool stage_me = end_me && !parked;                        // a whole segment ends here: new row
    const uint32_t tile8 = tile32 * 4 + sg;
    if (runs_on && !from_prev) starters[atomicAdd(starter_count, 1u)] = make_uint4(tile8, key, row, 0u);
    const unsigned begin_mask = __ballot_sync(full, begin_me);
    const uint32_t flags = (usable ? kFUsable : 0u) | (begin_me ? kFBegin : 0u) | (end_me ? kFEnd : 0u) |
                           (parked ? kFParked : 0u) | (from_prev ? kFFromPrev : 0u) |
                           (((usable && row_side) || both) ? kFBoth : 0u) | ((begin_me && stage_me) ? kFSingle : 0u) |
                           ((usable && !row_side) ? kFColumn : 0u);
    // does a long segment enter this block's group of 64 tiles from the group before?
    constexpr uint32_t kTilesPerBlock = 8 * 4;
    const uint32_t group = gb / (kGroupTiles / kTilesPerBlock);
    const uint64_t gpos = (uint64_t)group * kGroupTiles * kMfTile;
    uint32_t kg = kSentinelPad, kg_prev = kSentinelPad - 1, kg_far = kSentinelPad - 2;
    if (gpos > 0 && gpos + 8 * kMfTile - 1 < n) {
        kg = sk[gpos];
        kg_prev = sk[gpos - 1];
        kg_far = sk[gpos + 8 * kMfTile - 1];
    }
    const uint32_t L = L4 * 4;
    // (the stages start on a 128-byte boundary of shared memory: the TMA unit asks for that)
    float4* my_stage = stage_mem + ((128u - (smem_addr(stage_mem) & 127u)) & 127u) / 16 + (size_t)w * (kMfStages * 4 * 64);
    // Rows reach shared memory as bulk asynchronous copies of whole rows, issued by the lane that holds the
    // position; all copies of a walk step report to one barrier word of the warp.  (Per-lane 16-byte
    // asynchronous copies were measured too: 26 and 43 us per side against 20 and 20 with bulk copies.)
    if (lane < kMfStages) mbar_init(&bars[w][lane], 1);
    mbar_init_fence();
    __syncwarp();
    const uint32_t row_bytes = L4 * 16u;
    // asks for the rows of the four positions of walk step s2 (one per group)
    auto issue = [&](int s2, int stage) {
        if (s2 >= kMfTile) return;
        const unsigned sm = 0x01010101u << s2;
        if (kG4) {
            // the partner rows of the four groups' positions of this step (row 0 for a group that has none)
            const uint32_t want = usable ? prow : 0u;
            const int r0 = (int)__shfl_sync(full, want, s2), r1 = (int)__shfl_sync(full, want, 8 + s2);
            const int r2 = (int)__shfl_sync(full, want, 16 + s2), r3 = (int)__shfl_sync(full, want, 24 + s2);
            if (!(usable_mask & sm)) return;
            float4* dst = my_stage + (size_t)stage * 256;
            if (lane == 0) {
                mbar_expect_tx(&bars[w][stage], (4u + __popc(begin_mask & sm)) * row_bytes);
                tma_gather4(dst, &row_map, 0, r0, r1, r2, r3, &bars[w][stage]);
            }
            __syncwarp();
            if (l8 == s2 && begin_me) bulk_g2s(dst + 128 + sg * 32, store + (uint64_t)row * L4, row_bytes, &bars[w][stage]);
            return;
        }
        const uint32_t n_rows = __popc(usable_mask & sm) + __popc(begin_mask & sm);
        if (n_rows == 0) return;
        if (lane == 0) mbar_expect_tx(&bars[w][stage], n_rows * row_bytes);
        __syncwarp();
        if (l8 == s2 && usable) {
            float4* dst = my_stage + (size_t)(stage * 4 + sg) * 64;
            bulk_g2s(dst, store + (uint64_t)prow * L4, row_bytes, &bars[w][stage]);
            if (begin_me) bulk_g2s(dst + 32, store + (uint64_t)row * L4, row_bytes, &bars[w][stage]);
        }
    };
#pragma unroll
    for (int s2 = 0; s2 < kMfStages - 1; ++s2) issue(s2, s2);
    d4 acc[kC];
    float4 own[kC];
#pragma unroll
    for (int c = 0; c < kC; ++c) {
        acc[c] = d4{0.0, 0.0, 0.0, 0.0};
        own[c] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float nw = 0.f, loss_f = 0.f;                   // this lane's share of |own|^2 and of the tile's loss
    // A column factor's new row may go straight into the store if nobody else reads the row: its readers are the
    // positions of its own segment and, as a partner, the row-factor positions of its cells, and those are all
    // skipped if every position of the segment also updates its partner.
    bool direct = false;
    uint32_t uses = 0;
    int st_use = 0, st_fill = kMfStages - 1;
    const int n_steps = usable_mask ? kMfTile : 0;  // (a warp of skipped positions has nothing to walk)
#pragma unroll 1
    for (int s2 = 0; s2 < n_steps; ++s2) {
        __syncwarp();                               // every lane is done reading the stage to be refilled
        issue(s2 + kMfStages - 1, st_fill);
        const unsigned sm = 0x01010101u << s2;
        if (usable_mask & sm) {
            const uint32_t parity = (uses >> st_use) & 1u;
            if (!mbar_wait(&bars[w][st_use], parity) && !mbar_wait(&bars[w][st_use], parity)) {
                if (lane == 0) latch_error(st, epoch, PS_ERR_CUDA);
                break;                              // a copy that does not arrive: give the call up
            }
            uses ^= 1u << st_use;
        }
        // where this group's partner row and own row of the step lie
        const float4* slot = kG4 ? my_stage + (size_t)st_use * 256 + (size_t)sg * L4 + l8
                                 : my_stage + (size_t)(st_use * 4 + sg) * 64 + l8;
        const float4* oslot = kG4 ? my_stage + (size_t)st_use * 256 + 128 + sg * 32 + l8 : slot + 32;
        st_use = st_use + 1 == kMfStages ? 0 : st_use + 1;
        st_fill = st_fill + 1 == kMfStages ? 0 : st_fill + 1;
        const int src = 8 * sg + s2;
        const uint32_t f = __shfl_sync(full, flags, src);
        const float v = __shfl_sync(full, val, src);
        const uint64_t drow = base + src;           // a finished row goes to the staging row of its position
        const uint32_t prow_s = __shfl_sync(full, prow, src), row_s = __shfl_sync(full, row, src);
        const bool live = f & kFUsable;
        constexpr uint32_t kFDirect = kFBoth | kFColumn;
        if (f & kFBegin) direct = true;
        if (live) direct = direct && (f & kFDirect) == kFDirect;
        if (f & kFBegin) {
            nw = 0.f;
#pragma unroll
            for (int c = 0; c < kC; ++c) {
                own[c] = (uint32_t)(l8 + 8 * c) < L4 ? oslot[8 * c] : make_float4(0.f, 0.f, 0.f, 0.f);
                nw += own[c].x * own[c].x + own[c].y * own[c].y + own[c].z * own[c].z + own[c].w * own[c].w;
                acc[c] = d4{0.0, 0.0, 0.0, 0.0};
            }
        }
        float4 h[kC];
        float dot = 0.f, nh = 0.f;
#pragma unroll
        for (int c = 0; c < kC; ++c) {
            h[c] = (live && (uint32_t)(l8 + 8 * c) < L4) ? slot[8 * c] : make_float4(0.f, 0.f, 0.f, 0.f);
            dot += own[c].x * h[c].x + own[c].y * h[c].y + own[c].z * h[c].z + own[c].w * h[c].w;
            nh += h[c].x * h[c].x + h[c].y * h[c].y + h[c].z * h[c].z + h[c].w * h[c].w;
        }
        dot += __shfl_xor_sync(full, dot, 1);
        dot += __shfl_xor_sync(full, dot, 2);
        dot += __shfl_xor_sync(full, dot, 4);
        const float e = v - dot;
        // the cell's loss: the lanes keep their shares of the two squared norms, one lane adds the squared error
        // (taken where the cell's row factor is updated: on the row side, or here for a row key that occurs once)
        if (f & kFBoth) loss_f += 0.5f * lam * (nw + nh) + (l8 == 0 ? 0.5f * e * e : 0.f);
        if ((f & kFBoth) && (f & kFColumn)) {        // the partner's new row: it is a segment of this one position
#pragma unroll
            for (int c = 0; c < kC; ++c) {
                if ((uint32_t)(l8 + 8 * c) < L4) {
                    float4 r;
                    r.x = h[c].x + lr * (e * own[c].x - lam * h[c].x);
                    r.y = h[c].y + lr * (e * own[c].y - lam * h[c].y);
                    r.z = h[c].z + lr * (e * own[c].z - lam * h[c].z);
                    r.w = h[c].w + lr * (e * own[c].w - lam * h[c].w);
                    store[(uint64_t)prow_s * L4 + l8 + 8 * c] = r;
                }
            }
        }
        if (f & kFSingle) {
#pragma unroll
            for (int c = 0; c < kC; ++c) {
                if ((uint32_t)(l8 + 8 * c) < L4) {
                    float4 r;
                    r.x = own[c].x + lr * (e * h[c].x - lam * own[c].x);
                    r.y = own[c].y + lr * (e * h[c].y - lam * own[c].y);
                    r.z = own[c].z + lr * (e * h[c].z - lam * own[c].z);
                    r.w = own[c].w + lr * (e * h[c].w - lam * own[c].w);
                    if (direct) store[(uint64_t)row_s * L4 + l8 + 8 * c] = r;
                    else staged[drow * L4 + l8 + 8 * c] = r;
                }
            }
            // a staged row goes on the (short) list of rows the fix-up launch moves into the store
            if (!direct && l8 == 0) apply_row[atomicAdd(starter_count + 1, 1u)] = ((uint64_t)row_s << 32) | drow;
        } else if (live) {
#pragma unroll
            for (int c = 0; c < kC; ++c) {
                acc[c].x += (double)(lr * (e * h[c].x - lam * own[c].x));
                acc[c].y += (double)(lr * (e * h[c].y - lam * own[c].y));
                acc[c].z += (double)(lr * (e * h[c].z - lam * own[c].z));
                acc[c].w += (double)(lr * (e * h[c].w - lam * own[c].w));
            }
            if (f & kFEnd) {
#pragma unroll
                for (int c = 0; c < kC; ++c) {
                    const uint32_t fi = l8 + 8 * c;
                    if (fi >= L4) continue;
                    if (f & kFParked) {
                        double* cs = carry + ((uint64_t)tile8 * 2 + ((f & kFFromPrev) ? 0 : 1)) * L + (uint64_t)fi * 4;
                        *(double2*)cs = make_double2(acc[c].x, acc[c].y);
                        *(double2*)(cs + 2) = make_double2(acc[c].z, acc[c].w);
                    } else {
                        float4 r = own[c];
                        r.x = (float)((double)r.x + acc[c].x); r.y = (float)((double)r.y + acc[c].y);
                        r.z = (float)((double)r.z + acc[c].z); r.w = (float)((double)r.w + acc[c].w);
                        if (direct) store[(uint64_t)row_s * L4 + fi] = r;
                        else staged[drow * L4 + fi] = r;
                    }
                }
                if (!direct && !(f & kFParked) && l8 == 0)
                    apply_row[atomicAdd(starter_count + 1, 1u)] = ((uint64_t)row_s << 32) | drow;
            }
        }
    }
    __syncthreads();                                // the staging memory is scratch from here on
    // per-block loss partial, fixed order
    {
        const double lw = warp_sum_d((double)loss_f);
        if (lane == 0) wl[w] = lw;
        __syncthreads();
        if (threadIdx.x == 0) {
            double t = 0;
            for (int i = 0; i < 8; ++i) t += wl[i];
            loss_partial[blockIdx.x] = t;
        }
    }
    if (!(kg < K && kg_prev == kg && kg_far == kg)) return;
    const uint32_t arrivals = tmin<uint32_t>(kGroupTiles / kTilesPerBlock, gridDim.x - group * (kGroupTiles / kTilesPerBlock));
    group_preadd(sk, n, L4, carry, group_done, group_sum, group, gpos, kg, reinterpret_cast<d4 (*)[32]>(stage_mem),
                 &s_ticket, kMfTile, arrivals);
}

// Warps work through the list of tiles that start a border-crossing segment, one segment per warp at a
// time.  The warp finds the parked partials the segment has left behind (32 probes at a time): those of
// the tiles it runs through in the starter's group, then one pre-added value per later group, then the
// tiles after the last such group.  Up to eight partials the warp adds itself, in position order, to the
// starting tile's own partial, and updates the row; longer walks are shared by the block's warps.
// The shape of every sum depends only on the sorted positions.  The last block adds the call's loss
// partials, in index order.
template <int kCh>
__global__ void __launch_bounds__(32 * kFixupWarps, (kCh == 3 || kCh == 1) ? 3 : 2)
push_fixup_kernel(const uint32_t* __restrict__ sk, uint32_t n, float4* __restrict__ store,
                  const uint2* __restrict__ table, uint64_t S, uint32_t K, uint32_t L4,
                  const double* __restrict__ carry, const double* __restrict__ group_sum,
                  const uint4* __restrict__ starters,
                  const unsigned int* __restrict__ starter_count, const double* __restrict__ loss_partial,
                  uint32_t loss_blocks, double* __restrict__ loss_accum, uint32_t fix_blocks,
                  const float4* __restrict__ staged, const uint64_t* __restrict__ apply_row, uint32_t tile_len,
                  uint32_t apply_lo, const DevStatus* st, unsigned int epoch) {
    if (call_failed(st, epoch)) return;
    if (blockIdx.x > fix_blocks) {
        // Blocks past the loss block move staged rows into the store (calls that stage rows only): the reduction
        // left a list of {row, staging position}; a warp takes 32 entries at a time and copies their rows, several
        // in flight at once.
        const unsigned full = 0xffffffffu;
        const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
        const uint32_t listed = starter_count[1];
        const uint32_t stride = (gridDim.x - fix_blocks - 1) * kFixupWarps * 32;
        for (uint32_t b0 = ((blockIdx.x - fix_blocks - 1) * kFixupWarps + w) * 32; b0 < listed; b0 += stride) {
            const uint64_t e = b0 + lane < listed ? apply_row[b0 + lane] : ~0ull;
            unsigned m = __ballot_sync(full, b0 + lane < listed);
            constexpr int kFly = kCh == 1 ? 8 : 4;           // rows in flight per warp
            while (m) {
                int q[kFly];
                uint64_t ee[kFly];
                float4 x[kFly][kCh];
#pragma unroll
                for (int a = 0; a < kFly; ++a) {
                    q[a] = m ? __ffs(m) - 1 : -1;
                    m &= m - 1;                              // 0 stays 0
                    ee[a] = __shfl_sync(full, e, q[a] & 31);
                }
#pragma unroll
                for (int a = 0; a < kFly; ++a)
#pragma unroll
                    for (int c = 0; c < kCh; ++c)
                        if (q[a] >= 0 && lane + 32 * c < L4) x[a][c] = __ldcs(staged + (ee[a] & 0xffffffffu) * L4 + lane + 32 * c);
#pragma unroll
                for (int a = 0; a < kFly; ++a)
#pragma unroll
                    for (int c = 0; c < kCh; ++c)
                        if (q[a] >= 0 && lane + 32 * c < L4) store[(ee[a] >> 32) * L4 + lane + 32 * c] = x[a][c];
            }
        }
        return;
    }
    if (blockIdx.x == fix_blocks) {
        if (loss_accum) {                           // fixed-shape sum: strided per thread, then a tree
            __shared__ double ws[kFixupWarps];
            double t = 0;
            for (uint32_t b = threadIdx.x; b < loss_blocks; b += blockDim.x) t += loss_partial[b];
            t = warp_sum_d(t);
            if ((threadIdx.x & 31) == 0) ws[threadIdx.x >> 5] = t;
            __syncthreads();
            if (threadIdx.x == 0) {
                double tot = 0;
                for (int i = 0; i < kFixupWarps; ++i) tot += ws[i];
                *loss_accum += tot;
            }
        }
        return;
    }
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t count = *starter_count;
    const uint32_t L = L4 * 4;
    const uint32_t n_tiles = (uint32_t)(((uint64_t)n + tile_len - 1) / tile_len);
    const uint32_t min_span = 8 * tile_len;                 // shortest entering segment a group pre-adds
    // blocks that share the list: a warp per entry in one round if there are enough blocks; the others are done
    const uint32_t list_blocks = tmin<uint32_t>(fix_blocks, (count + kFixupWarps - 1) / kFixupWarps);
    if (blockIdx.x >= list_blocks) return;
    const uint32_t n_warps = list_blocks * kFixupWarps;
    // what a warp found out about its segment, for the block to share the work of a long one
    struct Walk {
        uint32_t tile, last_tile, group0, n_groups, rem_first, rem_cnt, is_long;
        uint64_t row;
    };
    __shared__ Walk walks[kFixupWarps];
    __shared__ d4 part[kFixupWarps][kCh][32];
    // one parked partial added to a[]: base is its f = 0 element
    auto add = [&](d4* a, uint32_t f0, const double* base) {
#pragma unroll
        for (int c = 0; c < kCh; ++c) {
            const uint32_t f = f0 + lane + 32 * c;
            if (f < L4) {
                const double2 x = *(const double2*)(base + (uint64_t)f * 4);
                const double2 y = *(const double2*)(base + (uint64_t)f * 4 + 2);
                a[c].x += x.x; a[c].y += x.y; a[c].z += y.x; a[c].w += y.y;
            }
        }
    };
    // where parked partial number i of the walk lies (tiles of the starter's group, then groups, then the rest)
    auto nth = [&](const Walk& k, uint32_t i) -> const double* {
        const uint32_t n1 = k.last_tile - k.tile;
        if (i < n1) return carry + ((uint64_t)(k.tile + 1 + i) * 2) * L;
        if (i < n1 + k.n_groups) return group_sum + ((uint64_t)k.group0 + (i - n1)) * L;
        return carry + ((uint64_t)(k.rem_first + (i - n1 - k.n_groups)) * 2) * L;
    };
    // Adds partials number i0, i0 + stride, ... (below n_parts) to a[], in that order; kB of them are requested
    // together before the first is added, so a walk costs one round trip per kB partials.
    constexpr int kB = kCh == 1 ? 4 : (kCh == 2 ? 4 : 2);
    auto add_range = [&](d4* a, uint32_t f0, const Walk& k, uint32_t i0, uint32_t stride, uint32_t n_parts) {
        for (uint32_t i = i0; i < n_parts; i += kB * stride) {
            double2 x[kB][kCh], y[kB][kCh];
#pragma unroll
            for (int b = 0; b < kB; ++b) {
                const uint32_t ib = i + b * stride;
                const double* base = nth(k, ib < n_parts ? ib : i);
#pragma unroll
                for (int c = 0; c < kCh; ++c) {
                    const uint32_t f = f0 + lane + 32 * c;
                    x[b][c] = y[b][c] = make_double2(0.0, 0.0);
                    if (ib < n_parts && f < L4) {
                        x[b][c] = *(const double2*)(base + (uint64_t)f * 4);
                        y[b][c] = *(const double2*)(base + (uint64_t)f * 4 + 2);
                    }
                }
            }
#pragma unroll
            for (int b = 0; b < kB; ++b) {
                if (i + b * stride >= n_parts) break;
#pragma unroll
                for (int c = 0; c < kCh; ++c) {
                    a[c].x += x[b][c].x; a[c].y += x[b][c].y; a[c].z += y[b][c].x; a[c].w += y[b][c].y;
                }
            }
        }
    };
    // The list is roughly in position order, so the most frequent keys (neighbours in key order for Zipf inputs,
    // each with a long walk that occupies a whole block) stand next to each other: consecutive entries go to
    // different blocks.
    for (uint32_t s0 = 0; s0 < count; s0 += n_warps) {      // same trip count for all warps of a block
        const uint32_t si = s0 + w * list_blocks + blockIdx.x;
        Walk k = {0, 0, 0, 0, 0, 0, 0, 0};
        if (si < count) {
            const uint4 rec = starters[si];                 // {tile, key, row} as the reduction saw them
            const uint32_t kl = rec.y;
            k.tile = rec.x;
            k.row = (uint64_t)rec.z | ((uint64_t)rec.w << 32);
            // The segment runs through the tiles after `tile` whose first key is its key (keys are sorted,
            // so they form a run).  Up to the end of the starter's group of 64 tiles they are taken one by
            // one; every later group the segment enters has one pre-added value.
            const uint32_t group_end = (k.tile / kGroupTiles + 1) * kGroupTiles;    // first tile of the next group
            const uint32_t walk_end = tmin<uint32_t>(group_end, n_tiles);
            k.last_tile = k.tile;
            for (uint32_t t0 = k.tile + 1; t0 < walk_end; t0 += 32) {
                const uint32_t t2 = t0 + lane;
                const unsigned m = __ballot_sync(full, t2 < walk_end && sk[(uint64_t)t2 * tile_len] == kl);
                k.last_tile += (uint32_t)__popc(m);
                if (m != full) break;
            }
            k.group0 = group_end / kGroupTiles;
            if (k.last_tile + 1 == group_end) {
                for (;;) {
                    const uint64_t g2 = (uint64_t)k.group0 + k.n_groups + lane;
                    const uint64_t gp = g2 * kGroupTiles * tile_len;
                    const unsigned m = __ballot_sync(
                        full, gp + min_span - 1 < n && sk[gp] == kl && sk[gp + min_span - 1] == kl);
                    k.n_groups += (uint32_t)__popc(m);      // hits are a prefix of the probed range
                    if (m != full) break;
                }
                k.rem_first = group_end + k.n_groups * kGroupTiles;
                const uint32_t t2 = k.rem_first + lane;
                k.rem_cnt = (uint32_t)__popc(__ballot_sync(
                    full, lane < 8 && t2 < n_tiles && sk[(uint64_t)t2 * tile_len] == kl));
            }
            const uint32_t n_parts = k.last_tile - k.tile + k.n_groups + k.rem_cnt;
            k.is_long = n_parts > kFixupWarps ? 1u : 0u;
            if (!k.is_long) {                               // a short walk: this warp alone, partials in position order
                for (uint32_t f0 = 0; f0 < L4; f0 += 32 * kCh) {
                    d4 a[kCh];
                    float4 r[kCh];
#pragma unroll
                    for (int c = 0; c < kCh; ++c) {
                        const uint32_t f = f0 + lane + 32 * c;
                        a[c] = d4{0.0, 0.0, 0.0, 0.0};
                        r[c] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (f < L4) r[c] = store[k.row * L4 + f];
                    }
                    add(a, f0, carry + ((uint64_t)k.tile * 2 + 1) * L);
                    add_range(a, f0, k, 0, 1, n_parts);
#pragma unroll
                    for (int c = 0; c < kCh; ++c) {
                        const uint32_t f = f0 + lane + 32 * c;
                        if (f < L4) {
                            float4 v = r[c];
                            v.x = (float)((double)v.x + a[c].x); v.y = (float)((double)v.y + a[c].y);
                            v.z = (float)((double)v.z + a[c].z); v.w = (float)((double)v.w + a[c].w);
                            store[k.row * L4 + f] = v;
                        }
                    }
                }
            }
        }
        if (lane == 0) walks[w] = k;
        __syncthreads();
        // long walks: the block's warps share one (warp w takes every 8th partial), the eight warp sums are
        // added in warp order to the starting tile's own partial, and warp 0 updates the row
        for (int j = 0; j < kFixupWarps; ++j) {
            if (!walks[j].is_long) continue;                // the same decision in every warp
            const Walk kj = walks[j];
            const uint32_t n_parts = kj.last_tile - kj.tile + kj.n_groups + kj.rem_cnt;
            for (uint32_t f0 = 0; f0 < L4; f0 += 32 * kCh) {
                d4 a[kCh];
                float4 r[kCh];
#pragma unroll
                for (int c = 0; c < kCh; ++c) {
                    const uint32_t f = f0 + lane + 32 * c;
                    a[c] = d4{0.0, 0.0, 0.0, 0.0};
                    r[c] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (w == 0 && f < L4) r[c] = store[kj.row * L4 + f];       // asked for early, used after the barrier
                }
                add_range(a, f0, kj, w, kFixupWarps, n_parts);
#pragma unroll
                for (int c = 0; c < kCh; ++c) part[w][c][lane] = a[c];
                __syncthreads();
                if (w == 0) {
                    d4 t[kCh];
#pragma unroll
                    for (int c = 0; c < kCh; ++c) t[c] = d4{0.0, 0.0, 0.0, 0.0};
                    add(t, f0, carry + ((uint64_t)kj.tile * 2 + 1) * L);
#pragma unroll
                    for (int c = 0; c < kCh; ++c) {
                        const uint32_t f = f0 + lane + 32 * c;
                        if (f >= L4) continue;
#pragma unroll
                        for (int i = 0; i < kFixupWarps; ++i) {
                            t[c].x += part[i][c][lane].x; t[c].y += part[i][c][lane].y;
                            t[c].z += part[i][c][lane].z; t[c].w += part[i][c][lane].w;
                        }
                        float4 v = r[c];
                        v.x = (float)((double)v.x + t[c].x); v.y = (float)((double)v.y + t[c].y);
                        v.z = (float)((double)v.z + t[c].z); v.w = (float)((double)v.w + t[c].w);
                        store[kj.row * L4 + f] = v;
                    }
                }
                __syncthreads();
            }
        }
        __syncthreads();                                    // walks[] is rewritten in the next round
    }
}

// ------------------------------------------------- push by atomic adds (measured alternative) ----
// The cumulative push without the sort: every occurrence adds its update row to the key's row with
// `red.global.add.v4.f32`.  The order in which the terms of a key meet is whatever the hardware makes of it, so
// sums of more than two terms are not reproducible from run to run, and every term is rounded into the row as
// it arrives (fp32), not summed in fp64 and rounded once.  A first kernel checks the keys, so that a call with a
// key out of range still changes nothing.
__global__ void __launch_bounds__(256)
push_check_keys_kernel(const uint64_t* __restrict__ keys, uint64_t n, uint64_t K, DevStatus* st, unsigned int epoch) {
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < n && keys[t] >= K) latch_error(st, epoch, PS_ERR_KEY_RANGE);
}

__global__ void __launch_bounds__(256)
push_atomic_kernel(const uint64_t* __restrict__ keys, uint64_t n, const float4* __restrict__ upd, float4* store,
                   const uint2* __restrict__ table, uint64_t S, uint32_t L4, const DevStatus* st, unsigned int epoch) {
    if (call_failed(st, epoch)) return;
    const int lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t n_warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    // a warp takes four occurrences at a time: four table look-ups and up to four update chunks per lane in flight
    for (uint64_t t0 = warp * 4; t0 < n; t0 += n_warps * 4) {
        uint64_t row[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) row[r] = t0 + r < n ? phys_row(table[keys[t0 + r]], S) : 0;
        for (uint32_t f = lane; f < L4; f += 32) {
            float4 u[4];
#pragma unroll
            for (int r = 0; r < 4; ++r)
                u[r] = t0 + r < n ? __ldcs(upd + (t0 + r) * L4 + f) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int r = 0; r < 4; ++r)
                if (t0 + r < n) {
                    float* d = reinterpret_cast<float*>(store + row[r] * L4 + f);
                    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(d), "f"(u[r].x), "f"(u[r].y),
                                 "f"(u[r].z), "f"(u[r].w)
                                 : "memory");
                }
        }
    }
}

void run_push_atomic(ps_store* ps, const uint64_t* d_keys, uint64_t n, const float* d_upd, cudaStream_t s) {
    PS_LAUNCH(ps, push_check_keys_kernel, div_up_u32(n, 256), 256, s, d_keys, n, ps->cfg.num_keys, ps->status, ps->epoch);
    const uint32_t grid = (uint32_t)tmin<uint64_t>((n + 31) / 32, (uint64_t)ps->sm_count * 8);
    PS_LAUNCH(ps, push_atomic_kernel, grid, 256, s, d_keys, n, (const float4*)d_upd, (float4*)ps->store, ps->table,
              ps->cfg.slots_per_part, ps->cfg.row_len / 4, ps->status, ps->epoch);
}

int run_push_sort(ps_store* ps, uint32_t n, cudaStream_t s) {
    return radix_sort_pairs(ps, n, nullptr, ps->key_bits, s, 0, ps->starter_count, div_up_u32(n, kGroupSpan));
}

// The launch that follows a reduction: finishes the border-crossing segments (tiles of tile_len positions), adds the
// loss partials and, for calls that staged new rows instead of writing them, moves the rows staged at
// positions apply_lo .. n into the store.
static void launch_fixup(ps_store* ps, const uint32_t* sk, uint32_t n, double* d_loss_accum, uint32_t loss_blocks,
                         bool apply, uint32_t tile_len, uint32_t apply_lo, cudaStream_t s) {
    const uint32_t tiles = div_up_u32(n, tile_len);
    const uint32_t L4 = ps->cfg.row_len / 4;
    // a warp per listed segment; there are fewer segments in the list than tiles
    const uint32_t fix_blocks = tmin<uint32_t>(div_up_u32(tiles, kFixupWarps), (uint32_t)ps->sm_count * (apply ? 4 : 8));
    // the rows staged by a matrix-factorization step are few (row keys with several cells, and their columns): a
    // handful of blocks works through their list
    const uint32_t apply_blocks = apply ? 8u : 0u;
    (void)apply_lo;
    const uint32_t grid = fix_blocks + 1 + apply_blocks;
#define FIXUP_ARGS sk, n, (float4*)ps->store, ps->table, ps->cfg.slots_per_part, (uint32_t)ps->cfg.num_keys, L4,   \
                   ps->carry, ps->group_sum, ps->starters, ps->starter_count, ps->loss_partial, loss_blocks,      \
                   loss_blocks ? d_loss_accum : nullptr, fix_blocks, (const float4*)ps->upd, ps->apply_rows,      \
                   tile_len, apply_lo, ps->status, ps->epoch
    if (L4 <= 32) PS_LAUNCH(ps, push_fixup_kernel<1>, grid, 32 * kFixupWarps, s, FIXUP_ARGS);
    else if (L4 <= 64) PS_LAUNCH(ps, push_fixup_kernel<2>, grid, 32 * kFixupWarps, s, FIXUP_ARGS);
    else if (L4 <= 96) PS_LAUNCH(ps, push_fixup_kernel<3>, grid, 32 * kFixupWarps, s, FIXUP_ARGS);
    else PS_LAUNCH(ps, push_fixup_kernel<4>, grid, 32 * kFixupWarps, s, FIXUP_ARGS);
#undef FIXUP_ARGS
}

// The MF step on sorted occurrences (which: buffer that holds the sorted keys; the records are in ps->rec); rows
// of at most 128 values.  One launch over all positions, then the fix-up launch, which also moves the staged rows
// into the store.
void run_mf_fused(ps_store* ps, uint32_t n_cells, int which, uint64_t col_key_base, float lr, float lambda,
                  double* d_loss_accum, cudaStream_t s, bool gather4) {
    const uint32_t* sk = which ? ps->keysB : ps->keysA;
    const uint32_t n = 2 * n_cells;
    const uint32_t L4 = ps->cfg.row_len / 4;
    const uint32_t blocks = div_up_u32(n, 256);
#define SUB_ARGS                                                                                                     \
    ps->row_map, sk, ps->rec, ps->cellpos, n, (uint32_t)col_key_base, lr, lambda, (float4*)ps->store, (uint32_t)ps->cfg.num_keys, \
        L4, (float4*)ps->upd, ps->apply_rows, ps->carry, ps->starters, ps->starter_count, ps->group_done,            \
        ps->group_sum, ps->loss_partial, ps->status, ps->epoch
#define SUB_LAUNCH(kC)                                                                                               \
    do {                                                                                                             \
        static std::atomic<unsigned long long> smem_set{0}, smem_set4{0};                                            \
        if (gather4) {                                                                                               \
            opt_in_smem((const void*)mf_sub_kernel<kC, true>, kMfSmem, &smem_set4);                                  \
            if (ps->prof) prof_before(ps, "mf_sub_kernel<" #kC ",gather4>", s);                                      \
            mf_sub_kernel<kC, true><<<blocks, 256, kMfSmem, s>>>(SUB_ARGS);                                          \
        } else {                                                                                                     \
            opt_in_smem((const void*)mf_sub_kernel<kC, false>, kMfSmem, &smem_set);                                  \
            if (ps->prof) prof_before(ps, "mf_sub_kernel<" #kC ">", s);                                              \
            mf_sub_kernel<kC, false><<<blocks, 256, kMfSmem, s>>>(SUB_ARGS);                                         \
        }                                                                                                            \
        if (ps->prof) prof_after(ps, s);                                                                             \
        ps->launches++;                                                                                              \
    } while (0)
    if (L4 <= 8) SUB_LAUNCH(1);
    else if (L4 <= 16) SUB_LAUNCH(2);
    else if (L4 <= 24) SUB_LAUNCH(3);
    else SUB_LAUNCH(4);
#undef SUB_LAUNCH
#undef SUB_ARGS
    launch_fixup(ps, sk, n, d_loss_accum, d_loss_accum ? blocks : 0, true, kMfTile, 0, s);
}

void run_push_reduce(ps_store* ps, uint32_t n, int which, const float* d_upd, double* d_loss_accum,
                     uint32_t loss_blocks, cudaStream_t s, const float* d_scales, uint32_t slots) {
    const uint32_t* sk = which ? ps->keysB : ps->keysA;
    const uint32_t* sv = which ? ps->valsB : ps->valsA;
    const uint32_t tiles = div_up_u32(n, kReduceTile);
    const uint32_t blocks = div_up_u32(tiles, 8);
    const uint32_t L4 = ps->cfg.row_len / 4;
#define REDUCE_ARGS sk, sv, n, (const float4*)d_upd, d_scales, slots, (float4*)ps->store, ps->table,                 \
                    ps->cfg.slots_per_part, (uint32_t)ps->cfg.num_keys, L4, ps->carry, ps->starters,                \
                    ps->starter_count, ps->group_done, ps->group_sum, ps->status, ps->epoch
#define REDUCE_LAUNCH(kCh, kScaled, kL4, kSlots)                                                                     \
    do {                                                                                                             \
        static std::atomic<unsigned long long> smem_set{0};                                                          \
        opt_in_smem((const void*)push_reduce_kernel<kCh, kScaled, kL4, kSlots>, reduce_smem(kCh), &smem_set);        \
        if (ps->prof) prof_before(ps, "push_reduce_kernel<" #kCh "," #kScaled ">", s);                               \
        push_reduce_kernel<kCh, kScaled, kL4, kSlots><<<blocks, 256, reduce_smem(kCh), s>>>(REDUCE_ARGS);            \
        if (ps->prof) prof_after(ps, s);                                                                             \
        ps->launches++;                                                                                              \
    } while (0)
    // the row lengths of the paper's workloads get kernels of their own: 128, 300 (41 slots per center) and 400 values
    if (d_scales) {
        if (L4 == 75 && slots == 41) REDUCE_LAUNCH(3, true, 75, 41);
        else if (L4 <= 32) REDUCE_LAUNCH(1, true, 0, 0);
        else if (L4 <= 64) REDUCE_LAUNCH(2, true, 0, 0);
        else if (L4 <= 96) REDUCE_LAUNCH(3, true, 0, 0);
        else REDUCE_LAUNCH(4, true, 0, 0);
    } else {
        if (L4 == 32) REDUCE_LAUNCH(1, false, 32, 0);
        else if (L4 == 100) REDUCE_LAUNCH(4, false, 100, 0);
        else if (L4 <= 32) REDUCE_LAUNCH(1, false, 0, 0);
        else if (L4 <= 64) REDUCE_LAUNCH(2, false, 0, 0);
        else if (L4 <= 96) REDUCE_LAUNCH(3, false, 0, 0);
        else REDUCE_LAUNCH(4, false, 0, 0);
    }
#undef REDUCE_LAUNCH
#undef REDUCE_ARGS
    launch_fixup(ps, sk, n, d_loss_accum, loss_blocks, false, kReduceTile, 0, s);
}

void run_kge_reduce(ps_store* ps, uint32_t n, int which, uint32_t dim, float lr, float eps, double* d_loss_accum,
                    uint32_t loss_blocks, cudaStream_t s) {
    const uint32_t* sk = which ? ps->keysB : ps->keysA;
    const uint32_t* sv = which ? ps->valsB : ps->valsA;
    const uint32_t blocks = div_up_u32(div_up_u32(n, kReduceTile), 8);
    const uint32_t G4 = dim / 2;                     // float4 of a gradient row (2 dim values)
#define KR_ARGS sk, sv, n, (const float4*)ps->upd, (float4*)ps->store, ps->table, ps->cfg.slots_per_part,            \
                (uint32_t)ps->cfg.num_keys, G4, lr, eps, ps->carry, ps->starters, ps->starter_count, ps->group_done, \
                ps->group_sum, ps->status, ps->epoch
#define KR_LAUNCH(kC)                                                                                                \
    do {                                                                                                             \
        static std::atomic<unsigned long long> smem_set{0};                                                          \
        const size_t smem = (size_t)8 * 2 * 3 * kC * 32 * sizeof(float4);                                            \
        opt_in_smem((const void*)kge_reduce_kernel<kC>, smem, &smem_set);                                            \
        if (ps->prof) prof_before(ps, "kge_reduce_kernel<" #kC ">", s);                                              \
        kge_reduce_kernel<kC><<<blocks, 256, smem, s>>>(KR_ARGS);                                                    \
        if (ps->prof) prof_after(ps, s);                                                                             \
        ps->launches++;                                                                                              \
    } while (0)
    if (G4 <= 32) KR_LAUNCH(1);
    else KR_LAUNCH(2);
#undef KR_LAUNCH
#undef KR_ARGS
    launch_fixup(ps, sk, n, d_loss_accum, loss_blocks, false, kReduceTile, 0, s);
}

void run_push_pipeline(ps_store* ps, uint32_t n, const float* d_upd, double* d_loss_accum, uint32_t loss_blocks,
                       cudaStream_t s) {
    const int which = run_push_sort(ps, n, s);
    run_push_reduce(ps, n, which, d_upd, d_loss_accum, loss_blocks, s);
}

}  // namespace psb
