// localize (Sections 3.1 and 3.2 of the paper) as one batched relocation.
//
// The paper relocates a parameter with three messages (requester -> home node,
// home node -> old owner, old owner -> requester; Figure 4).  With the whole
// store and the location table in one GPU's memory the same end state is
// reached by kernels: the requested keys are sorted and de-duplicated, keys the
// requester already owns are dropped, each remaining key gets a slot popped
// from the requester's free stack, its row is copied there, its old slot is
// pushed onto the old owner's free stack, and its table entry is rewritten.
// Every choice is a function of the sorted key order, so a sequential program
// reproduces tables and free lists bit for bit.
#include "ps_internal.cuh"

namespace psb {

struct LocScratch {
    uint32_t *flag, *mkey, *mowner, *mslot, *mnew;
};

// (a region of its own, not the update-row scratch: a relocation may run beside a step that is using that)
static LocScratch loc_scratch(ps_store* ps) {
    uint32_t* base = ps->loc_scratch;
    LocScratch s;
    s.flag = base;
    s.mkey = base + ps->max_keys;
    s.mowner = base + 2 * ps->max_keys;
    s.mslot = base + 3 * ps->max_keys;
    s.mnew = base + 4 * ps->max_keys;
    return s;
}

constexpr int kLocMaxChunks = 4096;     // chunks of 256 sorted positions whose sums one block can scan in shared memory

// First half of a localize call, one cooperative launch (the blocks meet at one grid barrier):
//   1. flag[pos] = 1 iff sorted position pos holds the first occurrence of a key that must move; sum per chunk of 256
//   2. every block scans the chunk sums (the same values in every block); the total is the number of keys that
//      move; if the requester has fewer free slots the call fails as a whole and nothing has been changed
//   3. the m-th moving key (ascending) takes the m-th slot from the top of the requester's stack; its old location
//      is recorded and its table entry rewritten.
__global__ void __launch_bounds__(256)
loc_plan_kernel(const uint32_t* __restrict__ sk, uint32_t n, uint2* table, uint32_t worker, uint64_t S, uint32_t K,
                const unsigned long long* __restrict__ tops, const uint32_t* __restrict__ stacks,
                uint32_t* __restrict__ flag, uint32_t* chunk_sums, LocScratch sc, uint32_t* __restrict__ owner_keys,
                unsigned int* bar, DevStatus* st, unsigned int epoch) {
    __shared__ uint32_t prefix[kLocMaxChunks];
    __shared__ uint32_t sm[8];
    __shared__ int s_ok;
    if (call_failed(st, epoch)) return;
    const uint32_t n_chunks = (n + 255) / 256;
    for (uint32_t c = blockIdx.x; c < n_chunks; c += gridDim.x) {
        const uint32_t pos = c * 256 + threadIdx.x;
        int f = 0;
        if (pos < n) {
            const uint32_t key = sk[pos];
            const bool first = pos == 0 || sk[pos - 1] != key;
            if (first && key < K) f = table[key].x != worker;
            flag[pos] = f;
        }
        const int total = __syncthreads_count(f);
        if (threadIdx.x == 0) chunk_sums[c] = total;
    }
    if (!grid_barrier(bar, gridDim.x, &s_ok)) {
        if (threadIdx.x == 0) atomicCAS(&st->sticky, 0u, (unsigned int)PS_ERR_CUDA);
        return;
    }
    uint32_t running = 0;
    for (uint32_t c0 = 0; c0 < n_chunks; c0 += 256) {
        const uint32_t i = c0 + threadIdx.x;
        const uint32_t v = i < n_chunks ? __ldcg(chunk_sums + i) : 0;
        uint32_t tot;
        const uint32_t ex = block_exclusive_scan_256(v, sm, &tot);
        if (i < n_chunks) prefix[i] = running + ex;
        running += tot;
    }
    __syncthreads();
    const unsigned long long top_w = tops[worker];
    if (blockIdx.x == 0 && threadIdx.x == 0) st->moved_total = running;
    if ((unsigned long long)running > top_w) {              // the same decision in every block
        if (blockIdx.x == 0 && threadIdx.x == 0) latch_error(st, epoch, PS_ERR_CAPACITY);
        grid_leave(bar, gridDim.x);
        return;
    }
    for (uint32_t c = blockIdx.x; c < n_chunks; c += gridDim.x) {
        const uint32_t pos = c * 256 + threadIdx.x;
        const uint32_t f = pos < n ? flag[pos] : 0;
        uint32_t tot;
        const uint32_t m = prefix[c] + block_exclusive_scan_256(f, sm, &tot);
        if (f) {
            const uint32_t key = sk[pos];
            const uint2 e = table[key];
            const uint32_t new_slot = stacks[(uint64_t)worker * S + (top_w - 1 - m)];
            sc.mkey[m] = key;
            sc.mowner[m] = e.x;
            sc.mslot[m] = e.y;
            sc.mnew[m] = new_slot;
            owner_keys[m] = e.x;
            table[key] = make_uint2(worker, new_slot);
        }
    }
    grid_leave(bar, gridDim.x);
}

__device__ __forceinline__ uint32_t lower_bound_u32(const uint32_t* __restrict__ a, uint32_t n, uint32_t key) {
    uint32_t lo = 0, hi = n;
    while (lo < hi) {
        const uint32_t mid = (lo + hi) >> 1;
        if (a[mid] < key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// Second half, one cooperative launch.  so = old owners of the moving keys, stably sorted (so ascending key inside
// an owner); sv = index m of the key.  Vacated slots go onto the old owners' stacks and the rows are moved; after a
// grid barrier (the stack heights are read by every push above) the heights are updated.
__global__ void __launch_bounds__(256)
loc_apply_kernel(const uint32_t* __restrict__ so, const uint32_t* __restrict__ sv, LocScratch sc,
                 unsigned long long* tops, uint32_t* __restrict__ stacks, float4* __restrict__ store, uint32_t worker,
                 uint64_t S, uint32_t L4, unsigned int* bar, DevStatus* st, unsigned int epoch) {
    __shared__ int s_ok;
    if (call_failed(st, epoch)) return;
    const uint32_t total = st->moved_total;
    const uint32_t gid = blockIdx.x * blockDim.x + threadIdx.x, n_threads = gridDim.x * blockDim.x;
    for (uint32_t q = gid; q < total; q += n_threads) {
        const uint32_t p = so[q];
        const uint32_t rank = q - lower_bound_u32(so, total, p);
        stacks[(uint64_t)p * S + tops[p] + rank] = sc.mslot[sv[q]];
    }
    const int lane = threadIdx.x & 31;
    for (uint32_t m = gid >> 5; m < total; m += n_threads >> 5) {
        const uint64_t src = (uint64_t)sc.mowner[m] * S + sc.mslot[m];
        const uint64_t dst = (uint64_t)worker * S + sc.mnew[m];
        for (uint32_t f = lane; f < L4; f += 32) store[dst * L4 + f] = store[src * L4 + f];
    }
    if (!grid_barrier(bar, gridDim.x, &s_ok)) {
        if (threadIdx.x == 0) atomicCAS(&st->sticky, 0u, (unsigned int)PS_ERR_CUDA);
        return;
    }
    for (uint32_t q = gid; q < total; q += n_threads) {
        const uint32_t p = so[q];
        if (q == total - 1 || so[q + 1] != p) tops[p] += (q - lower_bound_u32(so, total, p) + 1);   // one thread per owner
        if (q == 0) {
            tops[worker] -= total;                          // the requester is never an old owner
            st->rows_moved += total;
        }
    }
    grid_leave(bar, gridDim.x);
}

// ------------------------------------------------------------------------------------------------
// The whole call after the key sort as ONE cooperative launch, for stores of at most kLocFastWorkers
// partitions.  A block owns a contiguous span of the sorted positions.
//   phase 1   count the span's first occurrences that must move                          -> grid barrier 1
//   phase 2a  every block adds up the block counts (its own offset m0 among the moving keys, and the call's
//             total: the capacity check, the same decision in every block); the m-th moving key takes the m-th
//             slot from the top of the requester's stack, its old location is noted, its table entry rewritten;
//             old owners are counted per block                                           -> grid barrier 2
//   phase 3   per old owner: keys that leave it in earlier blocks = where this block's vacated slots go on that
//             owner's stack; one warp ranks the block's keys per owner in key order (warp match, running
//             counters in shared memory: stable) and pushes the vacated slots; the last block writes the new
//             stack heights (every block read the old ones before barrier 2)
//   rows      every block moves an equal share of ALL moving keys (the spans hold very different numbers of
//             them): old slot -> shared memory -> new slot as bulk asynchronous copies of whole rows, several
//             rounds in flight per warp.
// No second sort, no flag array, two grid barriers instead of four launches with four.
constexpr uint32_t kLocFastWorkers = 1024;          // partitions the per-block owner counters have room for
constexpr uint32_t kLocMaxGrid = 512;
constexpr uint32_t kLocStageBytes = 4096;           // row staging per warp and stage
constexpr int kLocStages = 3;
constexpr size_t kLocSmem = (size_t)8 * kLocStages * kLocStageBytes;

__global__ void __launch_bounds__(256, 2)
loc_fused_kernel(const uint32_t* __restrict__ sk, uint32_t n, uint32_t span, uint2* table, uint32_t worker,
                 uint32_t N, uint64_t S, uint32_t K, unsigned long long* tops, uint32_t* stacks, char* store,
                 uint32_t row_bytes, uint32_t* block_counts, uint32_t* owner_counts, LocScratch sc,
                 const uint32_t* __restrict__ busy_keys, uint32_t n_busy, uint32_t part_size, unsigned int* bar,
                 DevStatus* st, unsigned int epoch) {
    __shared__ uint32_t s_hist[kLocFastWorkers];    // phase 2a: keys leaving each owner from this block; phase 3: next stack position
    __shared__ uint32_t s_top[kLocFastWorkers];     // stack heights before the call (S < 2^32)
    __shared__ uint32_t s_part[2][256];
    __shared__ uint32_t sm[8];
    __shared__ uint32_t s_stat[2];
    __shared__ int s_ok;
    __shared__ __align__(8) uint64_t bars[8][kLocStages];
    extern __shared__ __align__(128) char loc_stage[];
    if (call_failed(st, epoch)) return;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const uint32_t b = blockIdx.x, G = gridDim.x;
    const uint32_t lo = (uint32_t)tmin<uint64_t>((uint64_t)b * span, n), hi = (uint32_t)tmin<uint64_t>((uint64_t)lo + span, n);
    // does sorted position pos hold the first occurrence of a key that must move?
    auto must_move = [&](uint32_t pos) -> bool {
        if (pos >= hi) return false;
        const uint32_t key = sk[pos];
        if (key >= K || (pos > 0 && sk[pos - 1] == key)) return false;
        return table[key].x != worker;
    };
    // ---- phase 1 ----
    // The first kKeep tiles of the span (all of it unless the call is very large) are looked at with every load of
    // a kind in flight at once, and what was read (key, table entry) stays in registers for phase 2a.
    constexpr int kKeep = 2;
    uint32_t k_key[kKeep];
    uint2 k_ent[kKeep];
    bool k_first[kKeep];
#pragma unroll
    for (int q = 0; q < kKeep; ++q) {
        const uint32_t pos = lo + q * 256 + tid;
        k_key[q] = pos < hi ? sk[pos] : kSentinelPad;
        const uint32_t before_it = (pos < hi && pos > 0) ? sk[pos - 1] : kSentinelPad;
        k_first[q] = pos < hi && k_key[q] < K && (pos == 0 || before_it != k_key[q]);
    }
#pragma unroll
    for (int q = 0; q < kKeep; ++q) k_ent[q] = k_first[q] ? table[k_key[q]] : make_uint2(worker, 0u);
    uint32_t cnt = 0, n_local = 0;
#pragma unroll
    for (int q = 0; q < kKeep; ++q) {
        if (lo + q * 256 >= hi) break;
        const bool mv = k_first[q] && k_ent[q].x != worker;
        cnt += (uint32_t)__syncthreads_count(mv);
        n_local += (uint32_t)__syncthreads_count(k_first[q] && !mv);
    }
    for (uint32_t t0 = lo + kKeep * 256; t0 < hi; t0 += 256) {
        const uint32_t pos = t0 + tid;
        const bool mv = must_move(pos);
        const bool first = pos < hi && sk[pos] < K && (pos == 0 || sk[pos - 1] != sk[pos]);
        cnt += (uint32_t)__syncthreads_count(mv);
        n_local += (uint32_t)__syncthreads_count(first && !mv);
    }
    if (tid == 0) {
        block_counts[b] = cnt;
        if (b == 0) st->deferred_now = 0u;                      // (added to after the barrier)
    }
    if (!grid_barrier(bar, G, &s_ok)) {
        if (tid == 0) atomicCAS(&st->sticky, 0u, (unsigned int)PS_ERR_CUDA);
        return;
    }
    // ---- phase 2a ----
    uint32_t before = 0, all = 0;
    for (uint32_t i = tid; i < G; i += 256) {
        const uint32_t v = __ldcg(block_counts + i);
        all += v;
        if (i < b) before += v;
    }
    uint32_t m0, total;
    block_exclusive_scan_256(before, sm, &m0);
    block_exclusive_scan_256(all, sm, &total);
    const unsigned long long top_w = tops[worker];
    if (b == 0 && tid == 0) {
        st->moved_total = total;
        st->loc_requested += n;
    }
    if ((unsigned long long)total > top_w) {                    // the same decision in every block: nothing has changed yet
        if (b == 0 && tid == 0) latch_error(st, epoch, PS_ERR_CAPACITY);
        grid_leave(bar, G);
        return;
    }
    for (uint32_t i = tid; i < N; i += 256) {
        s_hist[i] = 0u;
        s_top[i] = (uint32_t)tops[i];
    }
    if (tid < 2) s_stat[tid] = 0u;
    __syncthreads();
    uint32_t running = 0;
    for (uint32_t t0 = lo; t0 < hi; t0 += 256) {
        const uint32_t q = (t0 - lo) >> 8;
        bool f;
        uint32_t key = 0;
        uint2 e = make_uint2(0u, 0u);
        if (q == 0) { f = k_first[0] && k_ent[0].x != worker; key = k_key[0]; e = k_ent[0]; }
        else if (q == 1) { f = k_first[1] && k_ent[1].x != worker; key = k_key[1]; e = k_ent[1]; }
        else {
            f = must_move(t0 + tid);
            if (f) {
                key = sk[t0 + tid];
                e = table[key];
            }
        }
        uint32_t tot;
        const uint32_t ex = block_exclusive_scan_256(f ? 1u : 0u, sm, &tot);
        if (f) {
            const uint32_t m = m0 + running + ex;
            const uint32_t new_slot = stacks[(uint64_t)worker * S + (top_w - 1 - m)];
            // A key that the call running beside this one also touches keeps its table entry and its row until
            // that call is through (loc_deferred_kernel); its slot and its old owner's stack are settled now.
            bool wait_for_it = false;
            if (busy_keys) {
                uint32_t lo2 = 0, hi2 = n_busy;
                while (lo2 < hi2) {
                    const uint32_t mid = (lo2 + hi2) >> 1;
                    if (busy_keys[mid] < key) lo2 = mid + 1; else hi2 = mid;
                }
                wait_for_it = lo2 < n_busy && busy_keys[lo2] == key;
            }
            sc.mkey[m] = key;
            sc.flag[m] = wait_for_it ? 1u : 0u;
            sc.mowner[m] = e.x;
            sc.mslot[m] = e.y;
            sc.mnew[m] = new_slot;
            if (!wait_for_it) table[key] = make_uint2(worker, new_slot);
            atomicAdd(&s_hist[e.x], 1u);
            if (wait_for_it) atomicAdd(&s_stat[0], 1u);
            if (e.x != key / part_size) atomicAdd(&s_stat[1], 1u);      // it had left its initial partition before
        }
        running += tot;
    }
    __syncthreads();
    if (tid == 0) {
        if (s_stat[0]) atomicAdd(&st->loc_deferred, (unsigned long long)s_stat[0]);
        if (s_stat[1]) atomicAdd(&st->loc_moved_again, (unsigned long long)s_stat[1]);
        if (n_local) atomicAdd(&st->loc_already_local, (unsigned long long)n_local);
        if (s_stat[0]) atomicAdd(&st->deferred_now, s_stat[0]);
    }
    for (uint32_t i = tid; i < N; i += 256) owner_counts[(size_t)b * N + i] = s_hist[i];
    // ---- phase 3 ----
    __threadfence();
    if (!grid_barrier(bar, 2 * G, &s_ok)) {
        if (tid == 0) atomicCAS(&st->sticky, 0u, (unsigned int)PS_ERR_CUDA);
        return;
    }
    {
        // owner p's column of the per-block counts, added up by 256 / Np threads (Np = N rounded up to a power of two)
        uint32_t Np = 1;
        while (Np < N && Np < 256) Np <<= 1;
        const uint32_t nq = 256 / Np, q = tid / Np;
        for (uint32_t p0 = 0; p0 < N; p0 += Np) {
            const uint32_t p = p0 + (tid % Np);
            uint32_t base = 0, tot = 0;
            if (p < N) {
                for (uint32_t r0 = q; r0 < G; r0 += 16 * nq) {        // sixteen of the column's values asked for at a time
                    uint32_t c[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k)
                        c[k] = r0 + k * nq < G ? __ldcg(owner_counts + (size_t)(r0 + k * nq) * N + p) : 0u;
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        tot += c[k];
                        if (r0 + k * nq < b) base += c[k];
                    }
                }
            }
            s_part[0][tid] = base;
            s_part[1][tid] = tot;
            __syncthreads();
            if (q == 0 && p < N) {
                for (uint32_t i = 1; i < nq; ++i) {
                    base += s_part[0][tid + i * Np];
                    tot += s_part[1][tid + i * Np];
                }
                s_hist[p] = s_top[p] + base;
                if (b == G - 1 && tot) tops[p] = (unsigned long long)s_top[p] + tot;    // never the requester's stack
            }
            __syncthreads();
        }
        if (b == G - 1 && tid == 0) {
            tops[worker] = top_w - total;
            st->rows_moved += total;
        }
    }
    if (w == 0) {
        const unsigned lt = (1u << lane) - 1u;
        // the block's keys in rounds of 32; the old places of the first rounds are asked for all at once, so that
        // the walk below (one round after the other: the counters run on) does not wait for memory in every round
        constexpr int kAhead = 16;
        uint32_t own_r[kAhead], slot_r[kAhead];
#pragma unroll
        for (int k = 0; k < kAhead; ++k) {
            const uint32_t i = k * 32 + lane;
            own_r[k] = i < cnt ? sc.mowner[m0 + i] : 0u;
            slot_r[k] = i < cnt ? sc.mslot[m0 + i] : 0u;
        }
        auto place = [&](bool valid, uint32_t owner, uint32_t slot) {
            const unsigned peers = __match_any_sync(0xffffffffu, valid ? owner : (0x80000000u + lane));
            const int leader = __ffs(peers) - 1;
            uint32_t old = 0;
            if (valid && lane == leader) {
                old = s_hist[owner];
                s_hist[owner] = old + __popc(peers);
            }
            old = __shfl_sync(0xffffffffu, old, leader);
            if (valid) stacks[(uint64_t)owner * S + old + __popc(peers & lt)] = slot;
            __syncwarp();
        };
#pragma unroll
        for (int k = 0; k < kAhead; ++k)
            if ((uint32_t)k * 32 < cnt) place((uint32_t)k * 32 + lane < cnt, own_r[k], slot_r[k]);
        for (uint32_t i0 = kAhead * 32; i0 < cnt; i0 += 32) {
            const bool valid = i0 + lane < cnt;
            place(valid, valid ? sc.mowner[m0 + i0 + lane] : 0u, valid ? sc.mslot[m0 + i0 + lane] : 0u);
        }
    }
    // ---- the rows: every block moves an equal share of the call's moving keys (their old and new places are
    // in memory since barrier 2), whatever its own span of positions held ----
    const uint32_t mlo = (uint32_t)((uint64_t)b * total / G), mcnt = (uint32_t)((uint64_t)(b + 1) * total / G) - mlo;
    if (row_bytes <= kLocStageBytes) {
        char* my = loc_stage + (size_t)w * kLocStages * kLocStageBytes;
        if (lane < kLocStages) mbar_init(&bars[w][lane], 1);
        mbar_init_fence();
        __syncwarp();
        const uint32_t per_round = tmin<uint32_t>(32u, kLocStageBytes / row_bytes);
        const uint32_t n_rounds = (mcnt + per_round - 1) / per_round;
        uint32_t uses = 0;
        // rounds w, w + 8, ...; the loads of up to kLocStages - 1 later rounds are in flight while one is written out
        uint64_t dst_of[kLocStages];
        bool mine_of[kLocStages];
        uint32_t rows_of[kLocStages];
        auto issue = [&](uint32_t r, int stage) {
            mine_of[stage] = false;
            rows_of[stage] = 0;
            if (r >= n_rounds) return;
            const uint32_t i = r * per_round + lane;
            bool mine = (uint32_t)lane < per_round && i < mcnt;
            uint64_t src = 0;
            if (mine) {
                const uint32_t m = mlo + i;
                mine = __ldcg(sc.flag + m) == 0u;               // (rows that wait for the call beside this one move later)
                src = (uint64_t)__ldcg(sc.mowner + m) * S + __ldcg(sc.mslot + m);
                dst_of[stage] = (uint64_t)worker * S + __ldcg(sc.mnew + m);
            }
            const uint32_t rows = (uint32_t)__popc(__ballot_sync(0xffffffffu, mine));
            mine_of[stage] = mine;
            rows_of[stage] = rows;
            bulk_wait_read<kLocStages - 2>();                   // the stores that last read this stage have let go of it
            __syncwarp();
            if (lane == 0) mbar_expect_tx(&bars[w][stage], rows * row_bytes);   // (rows may be 0: the phase completes at once)
            __syncwarp();
            if (mine) bulk_g2s(my + (size_t)stage * kLocStageBytes + (size_t)lane * row_bytes, store + src * row_bytes,
                               row_bytes, &bars[w][stage]);
        };
        bool dead = false;
        int st_fill = 0;
        uint32_t r_next = w;
        for (int k = 0; k < kLocStages - 1; ++k) {
            issue(r_next, st_fill);
            bulk_commit();                                      // keeps one bulk group per issued round (empty here)
            r_next += 8;
            st_fill = st_fill + 1 == kLocStages ? 0 : st_fill + 1;
        }
        int st_use = 0;
        for (uint32_t r = w; r < n_rounds && !dead; r += 8) {
            const uint32_t parity = (uses >> st_use) & 1u;
            if (!mbar_wait(&bars[w][st_use], parity) && !mbar_wait(&bars[w][st_use], parity)) {
                if (lane == 0) latch_error(st, epoch, PS_ERR_CUDA);
                dead = true;
                break;
            }
            uses ^= 1u << st_use;
            fence_async_smem();
            if (mine_of[st_use])
                bulk_s2g(store + dst_of[st_use] * row_bytes, my + (size_t)st_use * kLocStageBytes + (size_t)lane * row_bytes,
                         row_bytes);
            bulk_commit();
            st_use = st_use + 1 == kLocStages ? 0 : st_use + 1;
            issue(r_next, st_fill);
            r_next += 8;
            st_fill = st_fill + 1 == kLocStages ? 0 : st_fill + 1;
        }
        bulk_wait_read<0>();
    } else {
        // rows too long for the staging: a warp per row, 128-bit loads and stores
        const uint32_t L4 = row_bytes / 16;
        float4* st4 = reinterpret_cast<float4*>(store);
        for (uint32_t i = w; i < mcnt; i += 8) {
            const uint32_t m = mlo + i;
            if (__ldcg(sc.flag + m)) continue;
            const uint64_t src = (uint64_t)__ldcg(sc.mowner + m) * S + __ldcg(sc.mslot + m), dst = (uint64_t)worker * S + __ldcg(sc.mnew + m);
            for (uint32_t f = lane; f < L4; f += 32) st4[dst * L4 + f] = st4[src * L4 + f];
        }
    }
    grid_leave(bar, G);
}

// Second half of a relocation that ran beside another call: the moving keys that call touched (flag[m] = 1) get
// their rows moved and their table entries rewritten now that it is through.
__global__ void __launch_bounds__(256)
loc_deferred_kernel(LocScratch sc, uint2* table, float4* store, uint32_t worker, uint64_t S, uint32_t L4,
                    const DevStatus* st, unsigned int epoch) {
    if (call_failed(st, epoch) || st->deferred_now == 0u) return;
    const uint32_t total = st->moved_total;
    const int lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, n_warps = (gridDim.x * blockDim.x) >> 5;
    for (uint32_t m0 = warp * 32; m0 < total; m0 += n_warps * 32) {
        const uint32_t m = m0 + lane;
        const bool mine = m < total && sc.flag[m] != 0u;
        unsigned todo = __ballot_sync(0xffffffffu, mine);
        if (mine) table[sc.mkey[m]] = make_uint2(worker, sc.mnew[m]);
        const uint64_t my_src = mine ? (uint64_t)sc.mowner[m] * S + sc.mslot[m] : 0;
        const uint64_t my_dst = mine ? (uint64_t)worker * S + sc.mnew[m] : 0;
        while (todo) {                                          // the warp moves the rows, four in flight at a time
            int q[4];
            uint64_t src[4], dst[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                q[a] = todo ? __ffs(todo) - 1 : -1;
                todo &= todo - 1;                               // 0 stays 0
                src[a] = __shfl_sync(0xffffffffu, my_src, q[a] & 31);
                dst[a] = __shfl_sync(0xffffffffu, my_dst, q[a] & 31);
            }
            for (uint32_t f = lane; f < L4; f += 32) {
                float4 x[4];
#pragma unroll
                for (int a = 0; a < 4; ++a)
                    if (q[a] >= 0) x[a] = store[src[a] * L4 + f];
#pragma unroll
                for (int a = 0; a < 4; ++a)
                    if (q[a] >= 0) store[dst[a] * L4 + f] = x[a];
            }
        }
    }
}

void run_localize_deferred(ps_store* ps, uint32_t worker, uint32_t n, cudaStream_t s) {
    LocScratch sc = loc_scratch(ps);
    const uint32_t grid = tmin<uint32_t>(div_up_u32(n, 256), (uint32_t)ps->sm_count * 8);
    PS_LAUNCH(ps, loc_deferred_kernel, grid, 256, s, sc, ps->table, (float4*)ps->store, worker, ps->cfg.slots_per_part,
              ps->cfg.row_len / 4, ps->status, ps->epoch);
}

// The call's keys (range-checked) have been sorted already; `which` says into which buffers.
void run_localize(ps_store* ps, uint32_t worker, uint32_t n, int which, cudaStream_t s, const uint32_t* busy_keys,
                  uint32_t n_busy) {
    LocScratch sc = loc_scratch(ps);
    const uint32_t* sk = which ? ps->keysB : ps->keysA;
    uint32_t* owner_keys = which ? ps->keysA : ps->keysB;    // the buffer the sorted keys are not in
    const uint32_t chunks = div_up_u32(n, 256);
    const uint64_t S = ps->cfg.slots_per_part;
    const uint32_t K = (uint32_t)ps->cfg.num_keys;
    const uint32_t L4 = ps->cfg.row_len / 4;
    if (ps->cfg.num_workers <= kLocFastWorkers) {
        static std::atomic<unsigned long long> smem_set{0};
        opt_in_smem((const void*)loc_fused_kernel, kLocSmem, &smem_set);
        // two blocks per SM at most (all of them resident: they meet at grid barriers)
        const uint32_t max_grid = tmin<uint32_t>((uint32_t)ps->sm_count * 2, kLocMaxGrid);
        uint32_t span = tmax<uint32_t>(div_up_u32(n, max_grid), 32u);
        const uint32_t grid_f = div_up_u32(n, span);
        uint2* table = ps->table;
        unsigned long long* tops = ps->tops;
        uint32_t* stacks = ps->stacks;
        char* store = (char*)ps->store;
        uint32_t row_bytes = ps->cfg.row_len * 4, N = ps->cfg.num_workers;
        uint32_t* block_counts = ps->loc_counts;
        uint32_t* owner_counts = ps->loc_counts + kLocMaxGrid;
        unsigned int* bar = ps->sort_ctl + 2;                   // words 0 and 1 belong to the sort
        DevStatus* st = ps->status;
        unsigned int epoch = ps->epoch;
        uint32_t part_size = div_up_u32(ps->cfg.num_keys, ps->cfg.num_workers);
        void* args[] = {(void*)&sk, (void*)&n, (void*)&span, (void*)&table, (void*)&worker, (void*)&N, (void*)&S, (void*)&K,
                        (void*)&tops, (void*)&stacks, (void*)&store, (void*)&row_bytes, (void*)&block_counts,
                        (void*)&owner_counts, (void*)&sc, (void*)&busy_keys, (void*)&n_busy, (void*)&part_size,
                        (void*)&bar, (void*)&st, (void*)&epoch};
        if (ps->prof) prof_before(ps, "loc_fused_kernel", s);
        cudaLaunchCooperativeKernel((const void*)loc_fused_kernel, dim3(grid_f), dim3(256), args, kLocSmem, s);
        if (ps->prof) prof_after(ps, s);
        ps->launches++;
        return;
    }
    // more partitions than the fused kernel keeps counters for: plan, sort the moving keys by old owner, apply.
    // cooperative launches (the blocks meet at a grid barrier): as many blocks as are resident at once, at most
    uint32_t grid = tmin<uint32_t>(chunks, (uint32_t)ps->sm_count * 4);
    unsigned int* bar_plan = ps->sort_ctl + 2;               // words 0 and 1 belong to the sort
    unsigned int* bar_apply = ps->sort_ctl + 4;
    uint2* table = ps->table;
    const unsigned long long* tops_c = ps->tops;
    unsigned long long* tops = ps->tops;
    uint32_t* stacks = ps->stacks;
    uint32_t* flag = sc.flag;
    uint32_t* sums = ps->scan_sums;
    DevStatus* st = ps->status;
    unsigned int epoch = ps->epoch;
    {
        void* args[] = {(void*)&sk, (void*)&n, (void*)&table, (void*)&worker, (void*)&S, (void*)&K, (void*)&tops_c,
                        (void*)&stacks, (void*)&flag, (void*)&sums, (void*)&sc, (void*)&owner_keys, (void*)&bar_plan,
                        (void*)&st, (void*)&epoch};
        if (ps->prof) prof_before(ps, "loc_plan_kernel", s);
        cudaLaunchCooperativeKernel((const void*)loc_plan_kernel, dim3(grid), dim3(256), args, 0, s);
        if (ps->prof) prof_after(ps, s);
        ps->launches++;
    }
    const int w2 = radix_sort_pairs(ps, n, &ps->status->moved_total, ps->owner_bits, s, which ^ 1, nullptr, 0);
    const uint32_t* so = w2 ? ps->keysB : ps->keysA;
    const uint32_t* sv = w2 ? ps->valsB : ps->valsA;
    {
        float4* store = (float4*)ps->store;
        void* args[] = {(void*)&so, (void*)&sv, (void*)&sc, (void*)&tops, (void*)&stacks, (void*)&store, (void*)&worker,
                        (void*)&S, (void*)&L4, (void*)&bar_apply, (void*)&st, (void*)&epoch};
        grid = tmin<uint32_t>(tmax<uint32_t>(div_up_u32(n, 8), 1u), (uint32_t)ps->sm_count * 4);
        if (ps->prof) prof_before(ps, "loc_apply_kernel", s);
        cudaLaunchCooperativeKernel((const void*)loc_apply_kernel, dim3(grid), dim3(256), args, 0, s);
        if (ps->prof) prof_after(ps, s);
        ps->launches++;
    }
}

}  // namespace psb
