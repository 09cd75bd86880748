// Internal declarations shared by the translation units of the library.
// Nothing here is part of the public interface (see include/ps.h).
#pragma once

#include <atomic>
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ps.h"

namespace psb {

constexpr uint32_t kSentinelPad = 0xFFFFFFFFu;   // never a key: num_keys < 2^32 - 1
constexpr int kSortThreads = 256;
constexpr int kSortItems = 8;
constexpr int kSortTile = kSortThreads * kSortItems;   // keys per sort block
constexpr int kRadixBits = 8;
constexpr int kRadix = 1 << kRadixBits;
constexpr int kMaxSortPasses = 4;                // 32-bit keys
constexpr int kSortCtlWords = kMaxSortPasses * kRadix + kMaxSortPasses;   // digit histograms of every pass, then tickets
constexpr int kReduceTile = 32;                  // sorted occurrences per warp in the segmented reduction
constexpr int kGroupSpan = 64 * kReduceTile;      // sorted positions whose parked parts are pre-added together
constexpr int kMaxLossBlocks = 4096;
constexpr int kHostStages = 3;                   // staging areas for batches that arrive from host memory
constexpr int kSortSets = 4;                     // calls whose key sort may be in flight at once (see SortSet)
constexpr int kSideStreams = 3;                  // internal streams that calls with a long sort take in turn

// Device-resident status words.  An error is latched per call with the call's
// epoch, so no kernel has to clear anything before a call starts.
struct DevStatus {
    unsigned int sticky;            // first error code since the last ps_sync
    unsigned int call_err_epoch[4]; // number of the last sorting call with that number mod 4 that failed on the device
                                    // (up to kSortSets such calls of one handle are in flight: later ones' sorts
                                    // beside the current one's kernels; only calls that take a buffer set are numbered)
    unsigned int moved_total;       // localize: number of keys that move in the current call
    unsigned int deferred_now;      // ... of which wait for the call that runs beside the relocation (ps_localize_beside)
    unsigned long long rows_moved;  // rows relocated by all successful localize calls so far
    unsigned long long loc_requested;       // keys handed to localize calls, repeats included
    unsigned long long loc_already_local;   // distinct keys per call that the requester owned already
    unsigned long long loc_moved_again;     // moved keys that had left their initial partition before (taken from a
                                            // worker that had localized them: localization conflicts, Section 3.2)
    unsigned long long loc_deferred;        // moved keys that had to wait for the call running beside the relocation
};

static_assert(kSortSets <= 4, "one error-epoch word per call in flight");

struct Profile;

// One of the kSortSets sets of buffers the key sort and the segment bookkeeping work in.  Calls rotate
// through the sets so that the sorts of the next steps can run while earlier steps are still reducing.
struct SortSet {
    uint32_t *keysA, *keysB, *valsA, *valsB;
    uint32_t* tile_state;
    uint32_t* sort_ctl;
    unsigned int* group_done;
    uint4* rec;
    uint32_t* cellpos;
    uint4* starters;
    unsigned int* starter_count;
    uint4* mf_dup;
    unsigned int* mf_tickets;
    cudaEvent_t ev_free;            // recorded after the last kernel that used the set
    bool used;
    bool loc_reader;                // a relocation on another stream reads this set's sorted keys (ps_localize_beside)
    int sorted_which;               // which key buffer holds the call's sorted keys (-1: the call sorted none)
    uint32_t sorted_n;
};

}  // namespace psb

struct ps_store {
    ps_config_t cfg;
    uint64_t max_keys;
    int key_bits;                   // bits needed for keys 0..K inclusive (K is the "no key" mark)
    uint32_t sort_blocks_cap;       // blocks the sort's digit counters (tile_state) have room for
    int owner_bits;
    // caller-owned device buffers
    float* store;
    uint2* table;                   // (owner, slot) per key
    unsigned long long* tops;       // N stack heights
    uint32_t* stacks;               // N x S
    char* ws;
    size_t ws_bytes;
    // carved out of the workspace
    psb::DevStatus* status;
    uint32_t *keysA, *keysB, *valsA, *valsB;
    uint32_t* tile_state;           // kMaxSortPasses x sort blocks x kRadix digit counters
    uint32_t* sort_ctl;             // the sort's grid barrier (two words) in kSortCtlWords, followed by group_done
    uint4* rec;                     // MF: {cell, cell value, row of the key, row of the other factor} per sorted position
    uint32_t* cellpos;              // MF: sorted position of each cell's row-factor occurrence
    uint4* mf_dup;                  // MF by column: per column position {first position, count, rank} of its cell's row key
    unsigned int* mf_tickets;       // MF by column: a ticket counter per row-side position, then one per block, then one
    unsigned int* group_done;       // per group of 64 reduction tiles: reduction blocks that have finished
    double* group_sum;              // per group: pre-added parked parts of the segment entering it (row_len)
    uint32_t* scan_sums;            // block sums of the device-wide scan
    uint32_t* loc_counts;           // localize: moving keys per block (512 words), then per block and old owner
    uint32_t* loc_scratch;          // localize: five words per key of the call (old and new places of the moving keys)
    float* upd;                     // max_keys x row_len update rows (also localize scratch)
    double* carry;                  // nReduceTiles x 2 x row_len partial sums of segments that span tiles
    uint4* starters;                // {tile, key, row} of the tiles that start a border-crossing segment
    unsigned int* starter_count;
    double* loss_partial;           // max(kMaxLossBlocks, one per 256 key occurrences)
    uint64_t* apply_rows;           // per sorted position: address of the row staged there, or all ones
    char* staging;                  // host-batch staging, max_keys x 8 bytes (the first of `stagings`)
    char* stagings[psb::kHostStages];
    // host state
    uint32_t epoch;
    uint64_t launches;
    int sm_count;
    psb::Profile* prof;             // per-kernel event timing, off unless ps_profile_start was called
    cudaStream_t side;              // key extraction and sort of the current call run here, beside the gradient kernel:
    cudaStream_t sides[psb::kSideStreams];  // one of these; calls whose sort is longer than the rest of the step take them
    int side_idx, side_alt;         // in turn, so that the sorts of several later steps run beside each other
    unsigned long long side_capture_id[psb::kSideStreams];  // graph capture each of them was last forked into (0 = none)
    cudaEvent_t ev_fork, ev_join;
    psb::SortSet sets[psb::kSortSets];           // keysA .. starter_count above always point into sets[cur_set]
    int cur_set;
    cudaStream_t copy;              // host batches are copied here in overlapped mode (ps_set_host_overlap)
    cudaEvent_t ev_copied[psb::kHostStages], ev_consumed[psb::kHostStages];
    bool consumed_valid[psb::kHostStages];
    int host_slot;
    bool host_overlap;
    cudaEvent_t batch_ready;        // set while a call's batch is still on its way: the side stream waits for it
    bool pipelined;                 // see ps_set_pipelining
    CUtensorMap row_map;            // the store as a 2-D tensor (row_len x rows, one row per box) for row gathers by the TMA unit
    bool row_map_ok;
    int mf_path;                    // see ps_set_mf_path
    psb::SortSet* last_set;         // the most recent call's buffer set if that call sorted its keys (else null)
    cudaStream_t last_stream;       // the stream of the most recent call
    cudaEvent_t ev_before, ev_sorted;       // most recent sorting call: the caller's stream before its first kernel; after its sort
    cudaEvent_t ev_loc;             // end of the most recent ps_localize_beside
    bool loc_pending;               // ... which later calls still have to be ordered after
    int push_mode;                  // see ps_set_push_mode
    bool table_dirty[psb::kSideStreams];   // per side stream: the location table was rewritten since that stream last waited
                                    // for the caller's (a sort that reads the table must not start before the rewrite)
    unsigned long long capture_id;  // graph capture the caller's stream was in at the last step call (0 = none)
};

namespace psb {

struct WsLayout {
    size_t status, keysA[kSortSets], keysB[kSortSets], valsA[kSortSets], valsB[kSortSets], tile_state[kSortSets],
        sort_ctl[kSortSets], rec[kSortSets], cellpos[kSortSets], mf_dup[kSortSets], mf_tickets[kSortSets], scan_sums, loc_counts, loc_scratch, upd, carry, group_sum, starters[kSortSets], starter_count[kSortSets],
        loss_partial, apply_rows, staging[kHostStages], total;
};
WsLayout ws_layout(const ps_config_t& cfg, uint64_t max_keys);

inline uint32_t div_up_u32(uint64_t a, uint64_t b) { return (uint32_t)((a + b - 1) / b); }

// The opt-in to more than 48 KB of dynamic shared memory is a per-DEVICE attribute of a kernel: `done` keeps one
// bit per device ordinal (a static of the launch site), so every GPU the process uses gets the attribute once.
inline void opt_in_smem(const void* fn, size_t bytes, std::atomic<unsigned long long>* done) {
    int d = -1;
    const bool known = cudaGetDevice(&d) == cudaSuccess && d >= 0 && d < 64;
    if (known && ((done->load(std::memory_order_relaxed) >> d) & 1ull)) return;
    cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (known) done->fetch_or(1ull << d, std::memory_order_relaxed);
}
template <class T> __host__ __device__ inline T tmin(T a, T b) { return a < b ? a : b; }
template <class T> __host__ __device__ inline T tmax(T a, T b) { return a > b ? a : b; }

// ---- ps_api.cu: optional per-kernel timing ----
void prof_before(ps_store* ps, const char* name, cudaStream_t s);
void prof_after(ps_store* ps, cudaStream_t s);

#define PS_LAUNCH(ps, kernel, grid, block, stream, ...)                       \
    do {                                                                     \
        if ((ps)->prof) psb::prof_before((ps), #kernel, (stream));           \
        kernel<<<(grid), (block), 0, (stream)>>>(__VA_ARGS__);               \
        if ((ps)->prof) psb::prof_after((ps), (stream));                     \
        (ps)->launches++;                                                    \
    } while (0)

#define PS_LAUNCH_SMEM(ps, kernel, grid, block, smem, stream, ...)            \
    do {                                                                     \
        if ((ps)->prof) psb::prof_before((ps), #kernel, (stream));           \
        kernel<<<(grid), (block), (smem), (stream)>>>(__VA_ARGS__);          \
        if ((ps)->prof) psb::prof_after((ps), (stream));                     \
        (ps)->launches++;                                                    \
    } while (0)

// ---- sort.cu ----
// Stable LSD radix sort of (key, value) pairs on the low `bits` bits of the key, one cooperative launch.
// Values are the positions 0..n-1 of the input.  Input in the A buffers (start = 0) or the B buffers
// (start = 1).  If n_dev is not null the element count is read from device memory (n is then an upper
// bound used for the launch shape).  Returns 0 if the result is in the A buffers, 1 if in the B buffers.
// Before its first grid barrier the kernel clears *zero_me (if not null) and the first `zero_groups`
// words of group_done.
int radix_sort_pairs(ps_store* ps, uint32_t n, const unsigned int* n_dev, int bits, cudaStream_t stream, int start,
                     unsigned int* zero_me, uint32_t zero_groups);
// the same on range-checked 64-bit caller keys (no separate key kernel); key_bits bits
int radix_sort_keys64(ps_store* ps, const uint64_t* d_keys, uint32_t n, cudaStream_t stream, unsigned int* zero_me,
                      uint32_t zero_groups);
// the 2 n_cells occurrences of a batch of matrix cells (2t: row factor, 2t + 1: column factor), keys taken
// from the batch arrays inside the sort; with `records` the last pass writes ps->rec beside the sorted keys
int radix_sort_mf(ps_store* ps, const uint32_t* d_i, const uint32_t* d_j, const float* d_v, uint32_t n_cells,
                  uint64_t col_key_base, bool records, cudaStream_t stream, unsigned int* zero_me,
                  uint32_t zero_groups);

// ---- pull_push.cu ----
void launch_init_range_partition(ps_store* ps, cudaStream_t s);
void launch_set_rows(ps_store* ps, const uint64_t* d_keys, uint64_t n, const float* d_vals, cudaStream_t s);
void launch_pull(ps_store* ps, const uint64_t* d_keys, uint64_t n, float* d_out, cudaStream_t s);
void launch_get_location(ps_store* ps, const uint64_t* d_keys, uint64_t n, uint32_t* d_owner, uint32_t* d_slot,
                         cudaStream_t s);
void launch_gather_rows_by_key(ps_store* ps, uint64_t first_key, uint64_t n, float* d_out, cudaStream_t s);
// keys64 -> keysA (range-checked)
void launch_prepare_keys(ps_store* ps, const uint64_t* d_keys, uint64_t n, cudaStream_t s);
// sort keysA (values = occurrence index), reduce `upd` rows per key, apply to the store, and add the
// first `loss_blocks` loss partials to *d_loss_accum (if not null)
void run_push_pipeline(ps_store* ps, uint32_t n, const float* d_upd, double* d_loss_accum, uint32_t loss_blocks,
                       cudaStream_t s);
// the two halves of the above: sort keysA (returns which buffer holds the result), then reduce and apply.
// With d_scales, occurrence o contributes d_scales[o] times a shared source row of d_upd: row 2e for slot 0
// of example e = o / slots, row 2e + 1 for its other slots.
int run_push_sort(ps_store* ps, uint32_t n, cudaStream_t s);
void run_push_reduce(ps_store* ps, uint32_t n, int which, const float* d_upd, double* d_loss_accum,
                     uint32_t loss_blocks, cudaStream_t s, const float* d_scales = nullptr, uint32_t slots = 0);

// push by atomic adds, no sort (ps_set_push_mode)
void run_push_atomic(ps_store* ps, const uint64_t* d_keys, uint64_t n, const float* d_upd, cudaStream_t s);

// MF step working on the sorted occurrences directly (rows of at most 512 values): gradient, reduction,
// then the fix-up launch that also moves the staged rows into the store
void run_mf_fused(ps_store* ps, uint32_t n_cells, int which, uint64_t col_key_base, float lr, float lambda,
                  double* d_loss_accum, cudaStream_t s, bool gather4);
// ---- mf_col.cu ----
// MF step as one launch over the column side of the sorted occurrences (rows of at most 128 values).  launch_mf_plan
// goes on the stream the sort ran on, right after it; run_mf_col on the caller's stream after the join.
void launch_mf_plan(ps_store* ps, uint32_t n_cells, int which, cudaStream_t side);
void run_mf_col(ps_store* ps, uint32_t n_cells, int which, float lr, float lambda, double* d_loss_accum, cudaStream_t s);

// ComplEx: reduce GRADIENT rows (2 dim values per occurrence, in ps->upd) into AdaGrad steps per key; dim even, <= 128
void run_kge_reduce(ps_store* ps, uint32_t n, int which, uint32_t dim, float lr, float eps, double* d_loss_accum,
                    uint32_t loss_blocks, cudaStream_t s);

// ---- localize.cu ----
// busy_keys: sorted keys of a call that may run beside this relocation (null: none); moving keys among them keep
// table entry and row until run_localize_deferred, which the caller enqueues once that call is through.
void run_localize(ps_store* ps, uint32_t worker, uint32_t n, int which, cudaStream_t s,
                  const uint32_t* busy_keys = nullptr, uint32_t n_busy = 0);
void run_localize_deferred(ps_store* ps, uint32_t worker, uint32_t n, cudaStream_t s);

// ---- steps.cu ----
// launch_keys_* write the keys of a batch's occurrence slots to keysA (they depend on the batch
// only, so they and the sort can run beside the gradient kernel); launch_step_* write the slots'
// update rows to `upd` (launch_step_sgns: two source rows per center and one factor per slot, to be
// reduced with run_push_reduce's d_scales) and return the number of per-block loss partials they wrote.
// ---- rescal.cu ----
void launch_keys_rescal(ps_store* ps, const uint32_t* d_s, const uint32_t* d_r, const uint32_t* d_o,
                        const uint32_t* d_neg_ent, uint64_t n, uint32_t n_neg, uint64_t rel_key_base, uint32_t dim,
                        cudaStream_t s);
uint32_t launch_grad_rescal(ps_store* ps, const uint32_t* d_s, const uint32_t* d_r, const uint32_t* d_o,
                            const uint32_t* d_neg_ent, const uint8_t* d_neg_side, uint64_t n, uint32_t n_neg,
                            uint64_t rel_key_base, uint32_t dim, cudaStream_t s);
void launch_keys_kge(ps_store* ps, const uint32_t* d_s, const uint32_t* d_r, const uint32_t* d_o,
                     const uint32_t* d_neg_ent, uint64_t n, uint32_t n_neg, uint64_t rel_key_base, cudaStream_t s);
void launch_keys_sgns(ps_store* ps, const uint32_t* d_tokens, uint64_t tok_first, uint64_t first_pos,
                      uint64_t n_centers, uint64_t corpus_len, uint32_t window, const uint32_t* d_negs, uint32_t n_neg,
                      uint64_t out_key_base, cudaStream_t s);
uint32_t launch_step_mf(ps_store* ps, const uint32_t* d_i, const uint32_t* d_j, const float* d_v, uint64_t n,
                        uint64_t col_key_base, float lr, float lambda, cudaStream_t s);
// grad_only: the update rows hold gradients (2 dim values each), to be reduced with run_kge_reduce
uint32_t launch_step_kge(ps_store* ps, const uint32_t* d_s, const uint32_t* d_r, const uint32_t* d_o,
                         const uint32_t* d_neg_ent, const uint8_t* d_neg_side, uint64_t n, uint32_t n_neg,
                         uint64_t rel_key_base, uint32_t dim, float lr, float eps, bool grad_only, cudaStream_t s);
float* sgns_scales(ps_store* ps, uint64_t n_centers);     // where launch_step_sgns puts the per-slot factors
uint32_t launch_step_sgns(ps_store* ps, const uint32_t* d_tokens, uint64_t tok_first, uint64_t first_pos,
                          uint64_t n_centers, uint64_t corpus_len, uint32_t window, const uint32_t* d_negs,
                          uint32_t n_neg, uint64_t out_key_base, float lr, cudaStream_t s);

// ---- device helpers ----
#ifdef __CUDACC__
// epoch 0: a call without later kernels to cancel (pull, set rows, get location); only the sticky code is latched
__device__ __forceinline__ void latch_error(DevStatus* st, unsigned int epoch, unsigned int code) {
    atomicCAS(&st->sticky, 0u, code);
    if (epoch != 0u) atomicExch(&st->call_err_epoch[epoch & 3u], epoch);
}
__device__ __forceinline__ bool call_failed(const DevStatus* st, unsigned int epoch) {
    return *((const volatile unsigned int*)&st->call_err_epoch[epoch & 3u]) == epoch;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ uint64_t phys_row(uint2 e, uint64_t S) { return (uint64_t)e.x * S + e.y; }
// AdaGrad's step -lr g / (sqrt(x) + eps), x = accumulator + g^2, with the hardware reciprocal square root and
// reciprocal (each within 2 ulp, far inside the fp32 tolerance of the result); x = 0 is kept away from 0 * inf
__device__ __forceinline__ float adagrad_step(float g, float x, float lr, float eps) {
    const float root = x > 0.f ? x * rsqrtf(x) : 0.f;
    return __fdividef(-lr * g, root + eps);
}

constexpr unsigned kBarrierSpins = 1u << 21;     // x ~100 ns: gives up after about a fifth of a second

// Barrier over all blocks of a cooperative launch.  bar[0] counts arrivals and only grows while the kernel
// runs: the k-th barrier is passed once it reaches k times the number of blocks.  bar[1] counts the blocks that
// have left the kernel; the last one to leave puts both words back to zero, so a launch always starts from
// zero without a clearing step in between.
__device__ __forceinline__ bool grid_barrier(unsigned int* bar, unsigned int target, int* s_ok) {
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;\n" ::"l"(bar) : "memory");
        unsigned int seen = 0, spins = 0;
        for (;;) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];\n" : "=r"(seen) : "l"(bar) : "memory");
            if (seen >= target || spins >= kBarrierSpins) break;
            __nanosleep(spins < 256 ? 20 : 100);
            ++spins;
        }
        *s_ok = seen >= target;
    }
    __syncthreads();
    return *s_ok != 0;
}
// The same barrier in two halves, for a block that has work to do between arriving and needing the others' results:
// everything the block wrote before grid_arrive is visible to a block that has passed grid_wait.
__device__ __forceinline__ void grid_arrive(unsigned int* bar) {
    __syncthreads();
    if (threadIdx.x == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;\n" ::"l"(bar) : "memory");
}
__device__ __forceinline__ bool grid_wait(unsigned int* bar, unsigned int target, int* s_ok) {
    if (threadIdx.x == 0) {
        unsigned int seen = 0, spins = 0;
        for (;;) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];\n" : "=r"(seen) : "l"(bar) : "memory");
            if (seen >= target || spins >= kBarrierSpins) break;
            __nanosleep(spins < 256 ? 20 : 100);
            ++spins;
        }
        *s_ok = seen >= target;
    }
    __syncthreads();
    return *s_ok != 0;
}
__device__ __forceinline__ void grid_leave(unsigned int* bar, unsigned int n_blocks) {
    if (threadIdx.x == 0 && atomicAdd(bar + 1, 1u) == n_blocks - 1) {
        // every other block has left, so nobody is waiting on the arrival count any more
        atomicExch(bar, 0u);
        atomicExch(bar + 1, 0u);
    }
}

// ---- bulk asynchronous copies global -> shared, reporting to a barrier word in shared memory ----
__device__ __forceinline__ unsigned smem_addr(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory"); }
// one arrival that also announces `bytes` of copies
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
// 16-byte aligned source and destination, size a multiple of 16 bytes
__device__ __forceinline__ void bulk_g2s(void* smem, const void* gmem, unsigned bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(
                     smem_addr(smem)),
                 "l"(gmem), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}
// Waits for the phase of the given parity to complete; gives up (false) after a bounded number of polls.  Each poll
// may stay suspended in hardware for up to kBarSuspendNs (it returns as soon as the phase completes), so that a
// waiting warp does not spend issue slots on polling: about a quarter of a second per call at most.
constexpr unsigned kBarPollLimit = 1u << 17;
constexpr unsigned kBarSuspendNs = 2000;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity) {
    const unsigned a = smem_addr(bar);
    for (unsigned i = 0; i < kBarPollLimit; ++i) {
        unsigned done;
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(done)
            : "r"(a), "r"(parity), "r"(kBarSuspendNs)
            : "memory");
        if (done) return true;
    }
    return false;
}

// shared -> global, tracked in the issuing thread's bulk groups
__device__ __forceinline__ void bulk_s2g(void* gmem, const void* smem, unsigned bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;\n" ::"l"(gmem), "r"(smem_addr(smem)), "r"(bytes)
                 : "memory");
}
// Four rows of a 2-D tensor (one row per box) into consecutive rows of shared memory with ONE instruction of the TMA
// unit: column x (x times the element size a multiple of 16 bytes), rows y0..y3.  The destination is 128-byte aligned.
__device__ __forceinline__ void tma_gather4(void* smem, const CUtensorMap* map, int x, int y0, int y1, int y2, int y3,
                                            uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, "
        "%5, %6}], [%7];\n" ::"r"(smem_addr(smem)),
        "l"(map), "r"(x), "r"(y0), "r"(y1), "r"(y2), "r"(y3), "r"(smem_addr(bar))
        : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;\n" ::: "memory"); }
// until at most kPending of this thread's bulk groups still have to READ their source
template <int kPending>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;\n" ::"n"(kPending) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }

// Exclusive scan of one value per thread over a block of 256 threads.
// `smem` must hold 8 uint32.  Returns the exclusive prefix; *total = block sum.
__device__ __forceinline__ uint32_t block_exclusive_scan_256(uint32_t v, uint32_t* smem, uint32_t* total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    uint32_t incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) smem[w] = incl;
    __syncthreads();
    uint32_t wbase = 0, tot = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        uint32_t t = smem[i];
        if (i < w) wbase += t;
        tot += t;
    }
    __syncthreads();
    *total = tot;
    return wbase + incl - v;
}
#endif

}  // namespace psb
