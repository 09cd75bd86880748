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

// The call's keys (range-checked) have been sorted already; `which` says into which buffers.
void run_localize(ps_store* ps, uint32_t worker, uint32_t n, int which, cudaStream_t s) {
    LocScratch sc = loc_scratch(ps);
    const uint32_t* sk = which ? ps->keysB : ps->keysA;
    uint32_t* owner_keys = which ? ps->keysA : ps->keysB;    // the buffer the sorted keys are not in
    const uint32_t chunks = div_up_u32(n, 256);
    const uint64_t S = ps->cfg.slots_per_part;
    const uint32_t K = (uint32_t)ps->cfg.num_keys;
    const uint32_t L4 = ps->cfg.row_len / 4;
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
