/*
 * ps.h -- C interface of the HBM-resident parameter store.
 *
 * One NVIDIA B200 holds every parameter row, a location table
 * key -> (owner, slot) and one free-slot stack per logical worker.  The calls
 * are the primitives of a parameter server with dynamic parameter allocation
 * (Renz-Wieland et al., VLDB 2020): pull and push (Section 2.1, Table 2),
 * localize (Sections 2.3, 3.1, 3.2), plus three fused minibatch steps
 * (pull -> per-example gradient -> push) for the tasks of Section 4.1.
 *
 * Conventions that hold for every call
 * ------------------------------------
 * Memory.   The library never allocates device memory.  Every `d_*` pointer is
 *           DEVICE memory owned by the caller and must stay valid until the
 *           stream has executed the call.  Buffers of rows (`d_vals`,
 *           `d_out`, `d_updates`) must be 16-byte aligned: they are moved as
 *           128-bit vectors and by bulk copies; a misaligned one is refused
 *           with PS_ERR_INVALID_ARG.  Every `h_*` pointer is HOST memory
 *           owned by the caller.  The library owns only the host handle.
 * Streams.  `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *           Every call except ps_create/ps_destroy/ps_sync/ps_export*, the
 *           counters and the `*_host` variants only enqueues work and returns;
 *           stream order is program order, which gives each key a single
 *           serial history (the per-key sequential consistency of Section 3.4).
 * Keys.     Dense in [0, num_keys) (the dense store of Section 3.7); duplicates
 *           are allowed in every key list: pull returns one row per
 *           occurrence, push sums, localize collapses.
 * Batch semantics.  Inside one call every read sees the state before the call;
 *           all additive terms of the call are summed per key (fp64) and added
 *           once, row = (float)((double)row + sum).  Results do not depend on
 *           thread scheduling: there are no floating-point atomics.
 * Errors.   Host-detectable errors (null pointer, size beyond the workspace,
 *           worker out of range) return at once and enqueue nothing.  Errors
 *           only the device can see (key out of range, partition full) make the
 *           offending CALL a no-op for store, table and free lists, latch the
 *           first such code on the device, and surface at the next ps_sync.
 *           Nothing ever traps, asserts or aborts.
 */
#ifndef PS_B200_PS_H
#define PS_B200_PS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ps_store ps_store_t;     /* opaque host handle */
typedef int ps_status_t;

enum {
    PS_OK = 0,
    PS_ERR_INVALID_ARG = 1,     /* null pointer, zero size where one is needed, bad config */
    PS_ERR_KEY_RANGE = 2,       /* a key (or an index that forms one) is >= num_keys */
    PS_ERR_WORKER_RANGE = 3,    /* worker >= num_workers */
    PS_ERR_CAPACITY = 4,        /* localize: the requester's partition has too few free slots */
    PS_ERR_WORKSPACE = 5,       /* the call needs more key occurrences than the workspace was sized for */
    PS_ERR_CUDA = 6,            /* a CUDA runtime call failed */
    PS_ERR_UNSUPPORTED = 7      /* configuration outside what the kernels implement */
};

typedef struct {
    uint64_t num_keys;          /* K; must be < 2^32 - 1 */
    uint32_t row_len;           /* fp32 values per key, optimizer state included; multiple of 4 */
    uint32_t num_workers;       /* N logical workers = partitions of the store; <= 65536 */
    uint64_t slots_per_part;    /* S, capacity of each partition; >= ceil(K/N), < 2^32 */
    int32_t device;             /* CUDA device ordinal */
} ps_config_t;

typedef struct {
    size_t store_bytes;         /* N * S * row_len * 4 */
    size_t table_bytes;         /* K * 8: (uint32 owner, uint32 slot) per key */
    size_t freelist_bytes;      /* N stack heights, then N stacks of S uint32 */
    size_t workspace_bytes;     /* scratch for calls of up to max_batch_keys key occurrences */
} ps_sizes_t;

/* Sizes of the four device buffers the caller must allocate (256-byte aligned).
 * `max_batch_keys` bounds the key occurrences of any later call: n for
 * pull/push/localize, 2n for ps_step_mf, (3 + n_neg) * n for ps_step_kge,
 * (2 + n_neg + dim) * n for ps_step_rescal,
 * n_centers * (1 + 2 * window * (1 + n_neg)), and at least 3 * n_centers,
 * for ps_step_sgns. */
ps_status_t ps_query_sizes(const ps_config_t* cfg, uint64_t max_batch_keys, ps_sizes_t* out);

/* Creates the host handle around caller-allocated device buffers of at least
 * the queried sizes.  Synchronous.  The store's contents are left as they are;
 * call ps_init_range_partition before anything else. */
ps_status_t ps_create(const ps_config_t* cfg, void* d_store, void* d_table, void* d_freelists,
                      void* d_workspace, size_t workspace_bytes, uint64_t max_batch_keys,
                      ps_store_t** out);

/* Frees the host handle only (after synchronising the device work it issued). */
ps_status_t ps_destroy(ps_store_t* ps);

/* Static initial allocation by range partitioning (Section 3.5; classic PSs,
 * Section 2.1): with B = ceil(K/N), key k goes to owner k / B, slot k % B.
 * Partition p's free stack then holds S-1, ..., cnt_p bottom to top, so its
 * lowest free slot is taken first.  Row values are not touched. */
ps_status_t ps_init_range_partition(ps_store_t* ps, void* stream);

/* Overwrites the rows of `d_keys` (n keys, distinct) with `d_vals` (n x row_len). */
ps_status_t ps_set_rows(ps_store_t* ps, const uint64_t* d_keys, uint64_t n, const float* d_vals,
                        void* stream);

/* pull (Table 2): d_out[t, :] = current row of d_keys[t], t < n; location-transparent. */
ps_status_t ps_pull(ps_store_t* ps, const uint64_t* d_keys, uint64_t n, float* d_out, void* stream);

/* push (Table 2; cumulative, Section 2.1): row(k) += sum over {t : d_keys[t] = k} of
 * d_updates[t, :].  Occurrences are sorted by key and reduced segment by segment. */
ps_status_t ps_push(ps_store_t* ps, const uint64_t* d_keys, uint64_t n, const float* d_updates,
                    void* stream);

/* localize (Sections 3.1, 3.2): every distinct key of the call that `worker` does
 * not own moves, with its whole row, into worker's partition, and the location
 * table is rewritten -- the end state of the relocation protocol of Figure 4.
 * Calls apply in stream order, so a key localized by several workers ends at
 * the last requester (localization conflicts, Section 3.2).
 * Slot policy: moved keys in ascending order; the m-th takes the m-th slot from
 * the top of worker's free stack; afterwards each vacated slot is pushed onto
 * its old owner's stack, ascending by key.  If worker has fewer free slots
 * than keys to move: PS_ERR_CAPACITY is latched and nothing changes.
 * Stores of more than 1024 partitions take at most 2^20 keys per call
 * (PS_ERR_UNSUPPORTED beyond; split the call). */
ps_status_t ps_localize(ps_store_t* ps, uint32_t worker, const uint64_t* d_keys, uint64_t n,
                        void* stream);

/* Pre-localization (Section 2.2 "latency hiding", Section 2.3, Appendix A: while a worker processes one data
 * point it localizes the parameters of the next one, negatives included).  The call is ps_localize for the keys
 * of the NEXT batch, enqueued on `loc_stream`, a stream other than the one the handle's most recent call (the
 * step or push of the current batch) was issued on, so that it runs beside that call:
 *   - it starts once every call made before the most recent one has finished;
 *   - keys that the most recent call does not touch are relocated beside it; keys that it does touch keep their
 *     table entry and their row until it has finished, and are relocated then (both on `loc_stream`);
 *   - every call made on the handle afterwards, on any stream, is ordered after the whole relocation.
 * The result (table, free stacks, rows) is that of ps_localize issued right after the most recent call.
 * If there is nothing to run beside (the most recent call was not a step or push, or was issued on
 * `loc_stream`), or the store has more than 1024 partitions, the call is an ordinary ps_localize on `loc_stream`
 * ordered after everything issued so far.  One such call per step; do not capture it into a CUDA graph. */
ps_status_t ps_localize_beside(ps_store_t* ps, uint32_t worker, const uint64_t* d_keys, uint64_t n,
                               void* loc_stream);

/* Counters over all localize calls of the handle so far (Table 5 of the paper reports the like: relocations,
 * local and non-local accesses).  Synchronous.
 *   requested      keys handed in, repeats included
 *   moved          keys relocated (= ps_rows_moved)
 *   already_local  distinct keys of a call that the requester owned already
 *   moved_again    relocated keys that had left their initial partition before, i.e. that were taken from a
 *                  worker that had localized them earlier: the localization conflicts of Section 3.2
 *   deferred       relocated keys that had to wait for the call running beside a ps_localize_beside */
typedef struct {
    uint64_t requested, moved, already_local, moved_again, deferred;
} ps_localize_stats_t;
ps_status_t ps_localize_stats(ps_store_t* ps, ps_localize_stats_t* h_out);

/* One SGD minibatch of low-rank matrix factorization (task of Section 4.1).
 * Key i is row factor w_i (i < col_key_base); key col_key_base + j is column
 * factor h_j.  For each of n cells (d_i[t], d_j[t], d_v[t]), at the pre-batch
 * state: e = v - <w, h>; loss e^2/2 + lambda/2 (|w|^2 + |h|^2);
 * w += lr (e h - lambda w), h += lr (e w - lambda h), summed per key.
 * *d_loss_accum (device, may be NULL) += the batch's loss. */
ps_status_t ps_step_mf(ps_store_t* ps, const uint32_t* d_i, const uint32_t* d_j, const float* d_v,
                       uint64_t n, uint64_t col_key_base, float lr, float lambda,
                       double* d_loss_accum, void* stream);

/* One minibatch of ComplEx with AdaGrad and negative sampling (Section 4.1,
 * Appendix A).  Key e is an entity (e < rel_key_base), key rel_key_base + r a
 * relation.  A row is [Re | Im | G_Re | G_Im], dim_complex fp32 each
 * (row_len = 4 * dim_complex); G are the AdaGrad accumulators.
 * Data point t = triple (d_s[t], d_r[t], d_o[t]) plus n_neg negatives
 * (n_neg <= 29): negative q replaces the subject (d_neg_side[t*n_neg+q] = 0)
 * or the object (1) by entity d_neg_ent[t*n_neg+q].  Score
 * phi = Re sum e_s w_r conj(e_o); loss softplus(-y phi).  For each distinct
 * key of a data point, g = its gradient of the data point's loss at the
 * pre-batch state; the call pushes dG = g*g and
 * dtheta = -lr g / (sqrt(G + g*g) + eps), summed per key. */
ps_status_t ps_step_kge(ps_store_t* ps, const uint32_t* d_s, const uint32_t* d_r, const uint32_t* d_o,
                        const uint32_t* d_neg_ent, const uint8_t* d_neg_side, uint64_t n,
                        uint32_t n_neg, uint64_t rel_key_base, uint32_t dim_complex, float lr,
                        float eps, double* d_loss_accum, void* stream);

/* One minibatch of RESCAL with AdaGrad and negative sampling (Section 4.1 names the
 * model, Table 4 its sizes: entity dimension dim, relation dimension dim * dim;
 * training as for ComplEx, Appendix A).  All rows have one length, so a
 * relation's matrix is dim keys, one per matrix row: key e < rel_key_base is
 * entity e with row [x | G]; key rel_key_base + r * dim + a is row a of R_r with
 * row [R_r[a][0..dim) | G]; G are the AdaGrad accumulators (row_len = 2 * dim).
 * Score phi = x_s^T R_r x_o; data points, negatives, loss and the AdaGrad push
 * per distinct key of a data point are those of ps_step_kge.
 * dim: a multiple of 4 from 4 to 128; n_neg <= 29; a call has
 * (2 + n_neg + dim) * n key occurrences.  Device arrays as for ps_step_kge.
 * Errors: PS_ERR_INVALID_ARG (null array, row_len != 2 * dim, rel_key_base past
 * the keys), PS_ERR_UNSUPPORTED (dim or n_neg outside the limits),
 * PS_ERR_WORKSPACE; an index out of range makes the call a no-op and latches
 * PS_ERR_KEY_RANGE. */
ps_status_t ps_step_rescal(ps_store_t* ps, const uint32_t* d_s, const uint32_t* d_r, const uint32_t* d_o,
                           const uint32_t* d_neg_ent, const uint8_t* d_neg_side, uint64_t n,
                           uint32_t n_neg, uint64_t rel_key_base, uint32_t dim, float lr, float eps,
                           double* d_loss_accum, void* stream);

/* One minibatch of skip-gram with negative sampling (Section 4.1, Appendix A).
 * Key w is the input vector of word w (w < out_key_base), key out_key_base + w
 * its output vector.  d_tokens is the whole stream (corpus_len tokens); the
 * centers are positions [first_pos, first_pos + n_centers); contexts of p are
 * the positions q != p, |q - p| <= window, inside the stream.  Pairs (p, q) are
 * numbered from 0 in (p, q) ascending order; pair z uses
 * d_negs[z*n_neg .. z*n_neg + n_neg).  Per pair and target (u, y) in
 * {(context, 1), (negative, 0)...}: x = <v, u>, g = sigmoid(x) - y,
 * u += -lr g v, v += -lr g u, summed per key.  row_len <= 512. */
ps_status_t ps_step_sgns(ps_store_t* ps, const uint32_t* d_tokens, uint64_t first_pos,
                         uint64_t n_centers, uint64_t corpus_len, uint32_t window,
                         const uint32_t* d_negs, uint32_t n_neg, uint64_t out_key_base, float lr,
                         double* d_loss_accum, void* stream);

/* The same steps for callers whose batch lives in HOST memory (pinned memory
 * makes the copies asynchronous).  Each copies the batch into the workspace,
 * runs the step, copies the accumulated loss back to *h_loss and waits for the
 * stream.  ps_step_sgns_host takes the tokens [tok_first, tok_first + tok_count)
 * that cover the batch's window; first_pos and corpus_len stay absolute. */
ps_status_t ps_step_mf_host(ps_store_t* ps, const uint32_t* h_i, const uint32_t* h_j, const float* h_v,
                            uint64_t n, uint64_t col_key_base, float lr, float lambda,
                            double* d_loss_accum, double* h_loss, void* stream);
ps_status_t ps_step_kge_host(ps_store_t* ps, const uint32_t* h_s, const uint32_t* h_r, const uint32_t* h_o,
                             const uint32_t* h_neg_ent, const uint8_t* h_neg_side, uint64_t n,
                             uint32_t n_neg, uint64_t rel_key_base, uint32_t dim_complex, float lr,
                             float eps, double* d_loss_accum, double* h_loss, void* stream);
ps_status_t ps_step_sgns_host(ps_store_t* ps, const uint32_t* h_tokens, uint64_t tok_first,
                              uint64_t tok_count, uint64_t first_pos, uint64_t n_centers,
                              uint64_t corpus_len, uint32_t window, const uint32_t* h_negs,
                              uint64_t n_negs, uint32_t n_neg, uint64_t out_key_base, float lr,
                              double* d_loss_accum, double* h_loss, void* stream);

/* The push for callers that cannot allocate device memory (the paper has no
 * counterpart to this entry point).  It is meant for code that runs where
 * cudaMalloc is off limits: a plug-in inside an application whose own pool holds
 * all GPU memory, a process with a fixed memory budget, a latency-critical loop
 * that cannot afford the device-wide synchronisation an allocation implies.
 * Such a caller cannot provide the workspace of ps_create, so this call needs
 * no handle: all scratch memory (sort buffers, partial sums) lives in a static
 * device array inside the library, about 2.3 MB, present on every GPU that
 * loads the library until the process exits.  The call itself calls neither
 * cudaMalloc nor cudaFree nor anything else that allocates.
 *   d_store, d_table: a store and its location table as laid out by ps_create /
 *   ps_init_range_partition (N * S rows of row_len fp32; (uint32 owner, uint32
 *   slot) per key), on the CURRENT device; num_keys, row_len, slots_per_part as
 *   in ps_config_t.  Result: exactly that of ps_push on the same arguments.
 * Limits: n <= PS_PUSH_STATIC_MAX_KEYS and row_len <= PS_PUSH_STATIC_MAX_ROW_LEN
 * (a multiple of 4); larger n returns PS_ERR_WORKSPACE, larger row_len
 * PS_ERR_UNSUPPORTED, and nothing is enqueued.
 * The call enqueues on `stream`, WAITS for it, and returns PS_ERR_KEY_RANGE
 * (store untouched) if a key is >= num_keys.
 * The first call on each device looks up the array's device address; make that
 * first call outside any stream capture.  Every call on a GPU uses the same
 * array: two calls that overlap in time on one GPU (different streams or
 * threads) race on it, so serialise them. */
#define PS_PUSH_STATIC_MAX_KEYS 16384
#define PS_PUSH_STATIC_MAX_ROW_LEN 256
ps_status_t ps_push_static(void* d_store, const void* d_table, uint64_t num_keys, uint32_t row_len,
                           uint64_t slots_per_part, const uint64_t* d_keys, uint64_t n,
                           const float* d_updates, void* stream);

/* d_owner[t], d_slot[t] = current location of d_keys[t]. */
ps_status_t ps_get_location(ps_store_t* ps, const uint64_t* d_keys, uint64_t n, uint32_t* d_owner,
                            uint32_t* d_slot, void* stream);

/* Synchronous copies for tests.  ps_export: rows by key (K x row_len), owner
 * and slot of every key (any pointer may be NULL to skip it).
 * ps_export_freelists: the N stacks (N x S, entries above a stack's height are
 * unspecified) and the N heights. */
ps_status_t ps_export(ps_store_t* ps, float* h_rows_by_key, uint32_t* h_owner, uint32_t* h_slot);
ps_status_t ps_export_freelists(ps_store_t* ps, uint32_t* h_stacks, uint64_t* h_tops);

/* Waits for `stream`; returns and clears the first error latched on the device. */
ps_status_t ps_sync(ps_store_t* ps, void* stream);

/* Latency hiding across steps, after the paper's pre-localization (Section 2.2,
 * "latency hiding": prepare the next data point's parameters while the current
 * one is processed).  It concerns ps_step_*, ps_push and ps_localize.
 * Off (default): such a call reads its batch arrays (indices, keys) only after
 * everything already enqueued on `stream`.  On: the keys of the batch are
 * extracted and sorted on an internal stream as soon as the call is made,
 * beside the kernels of earlier calls, so those arrays must be complete at
 * call time (no writes to them still pending on `stream`).
 * Results are identical in both modes.
 * The ps_step_* calls (device-batch variants) may be captured into a CUDA graph
 * on `stream`; an internal stream (the handle has three: ps_step_mf calls use
 * them in turn so that the sorts of two later steps overlap) joins the capture
 * at the first captured call that uses it and is joined back before each call
 * returns.  Begin a capture only when the
 * handle's earlier work has completed. */
ps_status_t ps_set_pipelining(ps_store_t* ps, int on);

/* Overlap of host batches with the steps before them (the same latency hiding of
 * Section 2.2, one level further out: the next batch travels while the current
 * one is processed).  It concerns the ps_step_*_host calls.
 * Off (default): such a call copies its batch on `stream`, runs the step, copies
 * the loss back and waits for the stream.
 * On: the batch is copied on an internal stream into one of three staging areas
 * as soon as the step that last used the area is through, the step's kernels
 * wait for that copy, and the call returns WITHOUT waiting: the h_* arrays must
 * stay unchanged, and *h_loss is not valid, until ps_sync (or another wait for
 * `stream`) has returned.  Give every call in flight its own h_loss word.  With
 * ps_set_pipelining on, the key sort of the next batch also starts as soon as its
 * copy has landed.  Results are identical in both modes.  The switch itself waits
 * for the device.  Do not capture ps_step_*_host calls into a CUDA graph. */
ps_status_t ps_set_host_overlap(ps_store_t* ps, int on);

/* How ps_push adds (Section 2.1: the push is cumulative; the paper's servers serialise the adds of a key with
 * latches, Section 3.7).
 *   PS_PUSH_SORTED (default): occurrences sorted by key, per-key sums in fp64, one rounding, one write per key;
 *     results are reproducible bit for bit.
 *   PS_PUSH_ATOMIC: no sort; every occurrence adds its row with vector atomic adds.  Kept as a measured
 *     alternative: each term is rounded into the row as it arrives and the order is the hardware's, so keys
 *     with more than two terms in a call are not reproducible from run to run (and differ from the sorted
 *     push in the last bits).  Integer-valued updates are exact either way.  Not limited by the workspace. */
enum { PS_PUSH_SORTED = 0, PS_PUSH_ATOMIC = 1 };
ps_status_t ps_set_push_mode(ps_store_t* ps, int mode);

/* Which kernels ps_step_mf uses on rows of at most 128 values (results are the same to rounding order; both
 * sum a key's terms in fp64 in the order of the sorted occurrences and round once).
 *   PS_MF_BY_COLUMN: one launch that visits the column-factor occurrences only; each forms its cell's terms
 *     for both factors (the tasks of Section 4.1 draw the rows of a batch from far more rows than the batch has
 *     cells, so a row factor nearly always has one cell).  Row keys with several cells in a batch are summed by
 *     the last of their cells to finish; a batch in which few row keys carry most cells is served slowly.
 *   PS_MF_SYMMETRIC: row and column occurrences are reduced alike, then a second launch finishes the
 *     segments that cross tile borders.  The rows of four positions are fetched by one instruction of the TMA unit
 *     (tile::gather4 on the store as a 2-D tensor); PS_MF_SYMMETRIC_ROW_COPIES: by one bulk copy per row instead
 *     (also what is used where the tensor cannot be described: rows of more than 256 values, 2^31 rows or more).
 *   PS_MF_AUTO (default): symmetric (the faster of the two on the 10M x 1M matrix of Section 4.1 as measured on
 *     B200: 45 against 49 microseconds per step of 65,536 cells). */
enum { PS_MF_AUTO = 0, PS_MF_BY_COLUMN = 1, PS_MF_SYMMETRIC = 2, PS_MF_SYMMETRIC_ROW_COPIES = 3 };
ps_status_t ps_set_mf_path(ps_store_t* ps, int path);

/* Self-test of the bounded device-side waits.  Every wait inside the kernels (the grid barrier of the one-launch
 * sort and relocation, the arrival of bulk copies) gives up after a bounded number of polls, latches PS_ERR_CUDA and
 * lets the kernel return, so that a lost arrival never hangs the GPU.  This call makes that happen on purpose, the
 * harmless way: two blocks wait at the sort's barrier for a third that does not exist, for about a fifth of a
 * second.  The next ps_sync returns PS_ERR_CUDA and puts the barrier back in order; the handle is usable after it. */
ps_status_t ps_selftest_barrier_timeout(ps_store_t* ps, void* stream);

/* Number of kernels this handle has launched so far. */
uint64_t ps_launch_count(const ps_store_t* ps);

/* Synchronous: *h_out = rows relocated by all successful ps_localize calls of this handle. */
ps_status_t ps_rows_moved(ps_store_t* ps, uint64_t* h_out);

/* Per-kernel timing for measurement runs.  After ps_profile_start the next
 * `max_launches` kernel launches of this handle are bracketed by CUDA events on
 * their stream.  ps_profile_stop waits for the device, writes one line per
 * kernel, "name launches total_microseconds\n", in first-launch order, into
 * h_report (NUL-terminated, truncated to `capacity` bytes) and turns timing off.
 * Each bracketed launch first waits for the whole device to go idle, so a time
 * is that of the kernel running alone (nothing beside it on the internal
 * stream): calls made while profiling is on run serialised, must not be captured
 * into a CUDA graph, and must not be timed end to end. */
ps_status_t ps_profile_start(ps_store_t* ps, uint32_t max_launches);
ps_status_t ps_profile_stop(ps_store_t* ps, char* h_report, size_t capacity);

/* One epoch of matrix factorization under parameter blocking (Section 2.2 "parameter blocking", Section 4.1,
 * Appendix A: the schedule of distributed SGD).  The handle's N workers split the rows into N contiguous blocks of
 * ceil(rows / N) and the columns into N blocks of ceil(cols / N); worker w keeps row block w for the whole
 * epoch (its row factors are localized to it first); the epoch has N subepochs; in subepoch s worker w localizes
 * the column factors of block (w + s) mod N and then runs minibatches of `batch` cells (ps_step_mf) over the
 * cells of (row block w, that column block).  Within a subepoch no two workers touch a common parameter; stream
 * order is the barrier between subepochs.
 * The cells must be grouped by stratum: h_offsets (host, N * N + 1 entries) gives for stratum (s, w), at index
 * s * N + w, the range [h_offsets[x], h_offsets[x + 1]) of its cells in d_i, d_j, d_v.  Key i is row factor i,
 * key rows + j column factor j; rows + cols = num_keys.  A partition holds at most the keys it started with, its
 * row block and one column block: slots_per_part >= ceil(K / N) + ceil(rows / N) + ceil(cols / N) always suffices.
 * Enqueues on `stream`; errors as for ps_localize and ps_step_mf. */
ps_status_t ps_dsgd_epoch_mf(ps_store_t* ps, const uint32_t* d_i, const uint32_t* d_j, const float* d_v,
                             const uint64_t* h_offsets, uint64_t rows, uint64_t cols, uint64_t batch, float lr,
                             float lambda, double* d_loss_accum, void* stream);

/* ---- sparse-map front end (Section 3.7: a server keeps its parameters "in dense arrays or sparse maps") ----
 * Translates arbitrary 64-bit keys into the dense keys 0 .. capacity-1 that every call above takes, so that a
 * store created with num_keys = capacity serves non-contiguous keys.  A key gets the next unused dense key the
 * first time it is seen; within one call new keys are numbered in order of first occurrence, so the translation
 * is reproducible by a sequential program.  The key with all 64 bits set is reserved.
 * The map lives in caller-allocated device memory (256-byte aligned) of ps_keymap_query_bytes bytes; calls of up
 * to max_batch_keys keys.  ps_keymap_create enqueues the clearing of that memory on `stream`.
 *   ps_keymap_insert   d_dense[t] = dense key of d_sparse[t], adding unseen keys.  A call that would exceed the
 *                      capacity adds nothing, writes all ones to d_dense and latches PS_ERR_CAPACITY; a call that
 *                      holds the reserved key adds nothing and latches PS_ERR_KEY_RANGE.
 *   ps_keymap_lookup   the same without adding: all ones for a key that was never inserted.
 *   ps_keymap_sync     waits for `stream`, returns and clears the latched code; *h_size (may be NULL) = dense keys
 *                      handed out so far.  After a failed insert, sync before the next insert.
 * Calls on one map are ordered by the caller (one stream, or events). */
typedef struct ps_keymap ps_keymap_t;
ps_status_t ps_keymap_query_bytes(uint64_t capacity, uint64_t max_batch_keys, size_t* out);
ps_status_t ps_keymap_create(uint64_t capacity, uint64_t max_batch_keys, void* d_mem, size_t bytes, int32_t device,
                             void* stream, ps_keymap_t** out);
ps_status_t ps_keymap_destroy(ps_keymap_t* map);
ps_status_t ps_keymap_insert(ps_keymap_t* map, const uint64_t* d_sparse, uint64_t n, uint64_t* d_dense, void* stream);
ps_status_t ps_keymap_lookup(ps_keymap_t* map, const uint64_t* d_sparse, uint64_t n, uint64_t* d_dense, void* stream);
ps_status_t ps_keymap_sync(ps_keymap_t* map, void* stream, uint64_t* h_size);
uint64_t ps_keymap_launch_count(const ps_keymap_t* map);

const char* ps_status_string(ps_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* PS_B200_PS_H */
