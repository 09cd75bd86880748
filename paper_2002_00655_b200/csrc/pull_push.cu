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
              ps->cfg.slots_per_part, ps->cfg.num_keys, ps->cfg.row_len / 4, ps->status, ps->epoch);
}

// ---------------------------------------------------------------- pull ----
// One warp gathers kRows rows at a time so that several independent 128-bit
// loads are in flight per lane.
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
    const uint32_t grid = (uint32_t)tmin<uint64_t>((n + 31) / 32, (uint64_t)ps->sm_count * 8);
    PS_LAUNCH(ps, pull_kernel<4>, grid, 256, s, d_keys, n, (float4*)d_out, (const float4*)ps->store, ps->table,
              ps->cfg.slots_per_part, ps->cfg.num_keys, ps->cfg.row_len / 4, ps->status, ps->epoch);
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
              ps->cfg.num_keys, ps->status, ps->epoch);
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

// A warp owns sorted positions [tile*32, tile*32+32).  A segment (run of equal
// keys) that starts and ends inside the tile is summed and applied here; a
// segment that continues from the previous tile parks its partial sum in carry
// slot 0 of the tile, one that continues into the next tile in slot 1.
__global__ void __launch_bounds__(256)
push_reduce_kernel(const uint32_t* __restrict__ sk, const uint32_t* __restrict__ sv, uint32_t n,
                   const float4* __restrict__ upd, float4* __restrict__ store, const uint2* __restrict__ table,
                   uint64_t S, uint32_t K, uint32_t L4, double* __restrict__ carry, const DevStatus* st,
                   unsigned int epoch) {
    if (call_failed(st, epoch)) return;
    const int lane = threadIdx.x & 31;
    const uint32_t tile = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t base = (uint64_t)tile * kReduceTile;
    if (base >= n) return;
    const uint32_t n_valid = (uint32_t)tmin<uint64_t>((uint64_t)kReduceTile, n - base);
    const uint32_t key = lane < n_valid ? sk[base + lane] : kSentinelPad;
    const uint32_t occ = lane < n_valid ? sv[base + lane] : 0u;
    uint32_t prev = __shfl_up_sync(0xffffffffu, key, 1);
    if (lane == 0) prev = base > 0 ? sk[base - 1] : kSentinelPad;
    const bool head = key != prev;
    const uint32_t next_after = (base + kReduceTile < n) ? sk[base + kReduceTile] : kSentinelPad;
    const bool head0 = __shfl_sync(0xffffffffu, (int)head, 0) != 0;
    unsigned heads = __ballot_sync(0xffffffffu, head) | 1u;
    const uint32_t L = L4 * 4;
    while (heads) {
        const int start = __ffs(heads) - 1;
        heads &= heads - 1;
        int end = heads ? (__ffs(heads) - 1) : kReduceTile;
        const uint32_t rkey = __shfl_sync(0xffffffffu, key, start);
        if (rkey >= K) break;                       // "no key" marks sort last
        const bool to_tile_end = end >= (int)n_valid;
        if (to_tile_end) end = (int)n_valid;
        const bool cont_start = (start == 0) && !head0;
        const bool cont_end = to_tile_end && n_valid == kReduceTile && next_after == rkey;
        const uint64_t row = phys_row(table[rkey], S);
        for (uint32_t f0 = 0; f0 < L4; f0 += 32) {
            const uint32_t f = f0 + lane;
            const bool act = f < L4;
            d4 acc = {0.0, 0.0, 0.0, 0.0};
#pragma unroll 4
            for (int p = start; p < end; ++p) {
                const uint32_t o = __shfl_sync(0xffffffffu, occ, p);
                if (act) {
                    const float4 u = __ldcs(upd + (uint64_t)o * L4 + f);
                    acc.x += (double)u.x; acc.y += (double)u.y; acc.z += (double)u.z; acc.w += (double)u.w;
                }
            }
            if (!act) continue;
            if (!cont_start && !cont_end) {
                float4 r = store[row * L4 + f];
                r.x = (float)((double)r.x + acc.x); r.y = (float)((double)r.y + acc.y);
                r.z = (float)((double)r.z + acc.z); r.w = (float)((double)r.w + acc.w);
                store[row * L4 + f] = r;
            } else {
                double* c = carry + ((uint64_t)tile * 2 + (cont_start ? 0 : 1)) * L + (uint64_t)f * 4;
                *(double2*)c = make_double2(acc.x, acc.y);
                *(double2*)(c + 2) = make_double2(acc.z, acc.w);
            }
        }
    }
}

// first index in [lo, n) whose key is greater than `key`
__device__ __forceinline__ uint64_t upper_bound_u32(const uint32_t* __restrict__ a, uint64_t lo, uint64_t n,
                                                    uint32_t key) {
    uint64_t hi = n;
    while (lo < hi) {
        const uint64_t mid = (lo + hi) >> 1;
        if (a[mid] <= key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// One warp per tile whose last segment starts in the tile and runs on into the
// next: it adds the parked partials tile by tile and applies the sum.  The
// block after the last tile block adds the call's loss partials, in index order.
__global__ void __launch_bounds__(256)
push_fixup_kernel(const uint32_t* __restrict__ sk, uint32_t n, float4* __restrict__ store,
                  const uint2* __restrict__ table, uint64_t S, uint32_t K, uint32_t L4,
                  const double* __restrict__ carry, const double* __restrict__ loss_partial,
                  uint32_t loss_blocks, double* __restrict__ loss_accum, uint32_t tile_blocks,
                  const DevStatus* st, unsigned int epoch) {
    if (call_failed(st, epoch)) return;
    if (blockIdx.x >= tile_blocks) {
        if (loss_accum && threadIdx.x == 0) {
            double tot = 0;
            for (uint32_t b = 0; b < loss_blocks; ++b) tot += loss_partial[b];
            *loss_accum += tot;
        }
        return;
    }
    const int lane = threadIdx.x & 31;
    const uint32_t tile = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t base = (uint64_t)tile * kReduceTile;
    if (base + kReduceTile >= n) return;             // the last tile cannot run on
    const uint32_t kl = sk[base + kReduceTile - 1];
    if (kl >= K || sk[base + kReduceTile] != kl) return;
    if (sk[base] == kl && base > 0 && sk[base - 1] == kl) return;   // continues a segment from before
    const uint64_t end_pos = upper_bound_u32(sk, base + kReduceTile, n, kl);
    const uint32_t last_tile = (uint32_t)((end_pos - 1) / kReduceTile);
    const uint32_t L = L4 * 4;
    const uint64_t row = phys_row(table[kl], S);
    for (uint32_t f = lane; f < L4; f += 32) {
        const double* c = carry + ((uint64_t)tile * 2 + 1) * L + (uint64_t)f * 4;
        double2 a = *(const double2*)c, b = *(const double2*)(c + 2);
#pragma unroll 4
        for (uint32_t t2 = tile + 1; t2 <= last_tile; ++t2) {
            const double* c2 = carry + ((uint64_t)t2 * 2) * L + (uint64_t)f * 4;
            const double2 a2 = *(const double2*)c2, b2 = *(const double2*)(c2 + 2);
            a.x += a2.x; a.y += a2.y; b.x += b2.x; b.y += b2.y;
        }
        float4 r = store[row * L4 + f];
        r.x = (float)((double)r.x + a.x); r.y = (float)((double)r.y + a.y);
        r.z = (float)((double)r.z + b.x); r.w = (float)((double)r.w + b.y);
        store[row * L4 + f] = r;
    }
}

void run_push_pipeline(ps_store* ps, uint32_t n, const float* d_upd, double* d_loss_accum, uint32_t loss_blocks,
                       cudaStream_t s) {
    const int which = radix_sort_pairs(ps, n, nullptr, ps->key_bits, true, s, 0);
    const uint32_t* sk = which ? ps->keysB : ps->keysA;
    const uint32_t* sv = which ? ps->valsB : ps->valsA;
    const uint32_t tiles = div_up_u32(n, kReduceTile);
    const uint32_t blocks = div_up_u32(tiles, 8);
    const uint32_t L4 = ps->cfg.row_len / 4;
    PS_LAUNCH(ps, push_reduce_kernel, blocks, 256, s, sk, sv, n, (const float4*)d_upd, (float4*)ps->store, ps->table,
              ps->cfg.slots_per_part, (uint32_t)ps->cfg.num_keys, L4, ps->carry, ps->status, ps->epoch);
    PS_LAUNCH(ps, push_fixup_kernel, blocks + 1, 256, s, sk, n, (float4*)ps->store, ps->table,
              ps->cfg.slots_per_part, (uint32_t)ps->cfg.num_keys, L4, ps->carry, ps->loss_partial, loss_blocks,
              loss_blocks ? d_loss_accum : nullptr, blocks, ps->status, ps->epoch);
}

}  // namespace psb
