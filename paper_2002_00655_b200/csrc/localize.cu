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

static LocScratch loc_scratch(ps_store* ps) {
    uint32_t* base = (uint32_t*)ps->upd;
    LocScratch s;
    s.flag = base;
    s.mkey = base + ps->max_keys;
    s.mowner = base + 2 * ps->max_keys;
    s.mslot = base + 3 * ps->max_keys;
    s.mnew = base + 4 * ps->max_keys;
    return s;
}

// flag[pos] = 1 iff sorted position pos holds the first occurrence of a key that must move
__global__ void __launch_bounds__(256)
loc_flag_kernel(const uint32_t* __restrict__ sk, uint32_t n, const uint2* __restrict__ table, uint32_t worker,
                uint32_t K, uint32_t* __restrict__ flag, uint32_t* __restrict__ block_sums, const DevStatus* st,
                unsigned int epoch) {
    if (call_failed(st, epoch)) return;
    const uint32_t pos = blockIdx.x * 256 + threadIdx.x;
    int f = 0;
    if (pos < n) {
        const uint32_t key = sk[pos];
        const bool first = pos == 0 || sk[pos - 1] != key;
        if (first && key < K) f = table[key].x != worker;
        flag[pos] = f;
    }
    const int total = __syncthreads_count(f);
    if (threadIdx.x == 0) block_sums[blockIdx.x] = total;
}

__global__ void __launch_bounds__(256)
loc_scan_sums_kernel(uint32_t* __restrict__ block_sums, uint32_t n_blocks, DevStatus* st, unsigned int epoch) {
    __shared__ uint32_t sm[8];
    if (call_failed(st, epoch)) return;
    uint32_t running = 0;
    for (uint32_t c0 = 0; c0 < n_blocks; c0 += 256) {
        const uint32_t i = c0 + threadIdx.x;
        const uint32_t v = i < n_blocks ? block_sums[i] : 0;
        uint32_t tot;
        const uint32_t ex = block_exclusive_scan_256(v, sm, &tot);
        if (i < n_blocks) block_sums[i] = running + ex;
        running += tot;
    }
    if (threadIdx.x == 0) st->moved_total = running;
}

// The m-th moving key (ascending) takes the m-th slot from the top of the
// requester's stack; its old location is recorded and its table entry rewritten.
__global__ void __launch_bounds__(256)
loc_assign_kernel(const uint32_t* __restrict__ sk, uint32_t n, uint2* __restrict__ table, uint32_t worker, uint64_t S,
                  const unsigned long long* __restrict__ tops, const uint32_t* __restrict__ stacks,
                  const uint32_t* __restrict__ flag, const uint32_t* __restrict__ block_sums, LocScratch sc,
                  uint32_t* __restrict__ owner_keys, DevStatus* st, unsigned int epoch) {
    __shared__ uint32_t sm[8];
    if (call_failed(st, epoch)) return;
    const unsigned long long top_w = tops[worker];
    if ((unsigned long long)st->moved_total > top_w) {      // same decision in every thread of the grid
        if (blockIdx.x == 0 && threadIdx.x == 0) latch_error(st, epoch, PS_ERR_CAPACITY);
        return;
    }
    const uint32_t pos = blockIdx.x * 256 + threadIdx.x;
    const uint32_t f = pos < n ? flag[pos] : 0;
    uint32_t tot;
    const uint32_t m = block_sums[blockIdx.x] + block_exclusive_scan_256(f, sm, &tot);
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

__device__ __forceinline__ uint32_t lower_bound_u32(const uint32_t* __restrict__ a, uint32_t n, uint32_t key) {
    uint32_t lo = 0, hi = n;
    while (lo < hi) {
        const uint32_t mid = (lo + hi) >> 1;
        if (a[mid] < key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// so = old owners of the moving keys, stably sorted (so ascending key inside an
// owner); sv = index m of the key.  Vacated slots go onto the old owner's stack.
__global__ void __launch_bounds__(256)
loc_free_kernel(const uint32_t* __restrict__ so, const uint32_t* __restrict__ sv, const uint32_t* __restrict__ mslot,
                const unsigned long long* __restrict__ tops, uint32_t* __restrict__ stacks, uint64_t S,
                const DevStatus* st, unsigned int epoch) {
    if (call_failed(st, epoch)) return;
    const uint32_t total = st->moved_total;
    const uint32_t q = blockIdx.x * 256 + threadIdx.x;
    if (q >= total) return;
    const uint32_t p = so[q];
    const uint32_t rank = q - lower_bound_u32(so, total, p);
    stacks[(uint64_t)p * S + tops[p] + rank] = mslot[sv[q]];
}

__global__ void __launch_bounds__(256)
loc_commit_kernel(const uint32_t* __restrict__ so, unsigned long long* __restrict__ tops, uint32_t worker,
                  DevStatus* st, unsigned int epoch) {
    if (call_failed(st, epoch)) return;
    const uint32_t total = st->moved_total;
    const uint32_t q = blockIdx.x * 256 + threadIdx.x;
    if (q >= total) return;
    const uint32_t p = so[q];
    if (q == total - 1 || so[q + 1] != p) tops[p] += (q - lower_bound_u32(so, total, p) + 1);   // one thread per owner
    if (q == 0) {
        tops[worker] -= total;                              // the requester is never an old owner
        st->rows_moved += total;
    }
}

__global__ void __launch_bounds__(256)
loc_move_kernel(LocScratch sc, float4* __restrict__ store, uint32_t worker, uint64_t S, uint32_t L4,
                const DevStatus* st, unsigned int epoch) {
    if (call_failed(st, epoch)) return;
    const uint32_t total = st->moved_total;
    const int lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t n_warps = (gridDim.x * blockDim.x) >> 5;
    for (uint32_t m = warp; m < total; m += n_warps) {
        const uint64_t src = (uint64_t)sc.mowner[m] * S + sc.mslot[m];
        const uint64_t dst = (uint64_t)worker * S + sc.mnew[m];
        for (uint32_t f = lane; f < L4; f += 32) store[dst * L4 + f] = store[src * L4 + f];
    }
}

// The call's keys (range-checked) have been sorted already; `which` says into which buffers.
void run_localize(ps_store* ps, uint32_t worker, uint32_t n, int which, cudaStream_t s) {
    LocScratch sc = loc_scratch(ps);
    const uint32_t* sk = which ? ps->keysB : ps->keysA;
    uint32_t* owner_keys = which ? ps->keysA : ps->keysB;    // the buffer the sorted keys are not in
    const uint32_t blocks = div_up_u32(n, 256);
    const uint64_t S = ps->cfg.slots_per_part;
    const uint32_t K = (uint32_t)ps->cfg.num_keys;
    PS_LAUNCH(ps, loc_flag_kernel, blocks, 256, s, sk, n, ps->table, worker, K, sc.flag, ps->scan_sums, ps->status,
              ps->epoch);
    PS_LAUNCH(ps, loc_scan_sums_kernel, 1, 256, s, ps->scan_sums, blocks, ps->status, ps->epoch);
    PS_LAUNCH(ps, loc_assign_kernel, blocks, 256, s, sk, n, ps->table, worker, S, ps->tops, ps->stacks, sc.flag,
              ps->scan_sums, sc, owner_keys, ps->status, ps->epoch);
    const int w2 = radix_sort_pairs(ps, n, &ps->status->moved_total, ps->owner_bits, s, which ^ 1, nullptr, 0);
    const uint32_t* so = w2 ? ps->keysB : ps->keysA;
    const uint32_t* sv = w2 ? ps->valsB : ps->valsA;
    PS_LAUNCH(ps, loc_free_kernel, blocks, 256, s, so, sv, sc.mslot, ps->tops, ps->stacks, S, ps->status, ps->epoch);
    PS_LAUNCH(ps, loc_commit_kernel, blocks, 256, s, so, ps->tops, worker, ps->status, ps->epoch);
    uint32_t move_blocks = div_up_u32(n, 8);
    if (move_blocks > (uint32_t)ps->sm_count * 8) move_blocks = (uint32_t)ps->sm_count * 8;
    PS_LAUNCH(ps, loc_move_kernel, move_blocks, 256, s, sc, (float4*)ps->store, worker, S, ps->cfg.row_len / 4,
              ps->status, ps->epoch);
}

}  // namespace psb
