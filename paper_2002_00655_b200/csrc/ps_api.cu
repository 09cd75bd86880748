// The exported C interface (include/ps.h): argument checks, workspace layout,
// and the order in which the kernels of a call are enqueued.
#include <map>
#include <new>
#include <stdio.h>
#include <stdlib.h>
#include <string>
#include <string.h>
#include <vector>

#include "ps_internal.cuh"

namespace psb {

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

WsLayout ws_layout(const ps_config_t& cfg, uint64_t max_keys) {
    WsLayout l;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        const size_t at = off;
        off = align_up(off + bytes, 256);
        return at;
    };
    const uint64_t mk = max_keys ? max_keys : 1;
    const size_t sort_tiles = (mk + kSortTile / 2 - 1) / (kSortTile / 2);   // the sort's blocks, at its shortest tile
    // tiles of the reduction: 32 positions, or 8 for the matrix-factorization step on rows of at most 128 values
    const size_t tile_len = cfg.row_len <= 128 ? 8 : kReduceTile;
    const size_t reduce_tiles = (mk + tile_len - 1) / tile_len;
    const size_t groups = (mk + tile_len * 64 - 1) / (tile_len * 64);
    const size_t row_bytes = (size_t)cfg.row_len * 4;
    l.status = take(sizeof(DevStatus));
    for (int b = 0; b < kSortSets; ++b) {
        l.keysA[b] = take(mk * 4);
        l.keysB[b] = take(mk * 4);
        l.valsA[b] = take(mk * 4);
        l.valsB[b] = take(mk * 4);
        l.tile_state[b] = take((size_t)kMaxSortPasses * sort_tiles * kRadix * 4);
        l.sort_ctl[b] = take(((size_t)kSortCtlWords + groups) * 4);
        l.rec[b] = take(mk * 16);
        l.cellpos[b] = take(mk * 4);
        l.mf_dup[b] = take((mk / 2 + 1 + mk / 512 + 2) * 16);      // per column position, then per block of 256 of them
        l.mf_tickets[b] = take((mk / 2 + 1 + mk / 512 + 4) * 4);
        l.starters[b] = take(reduce_tiles * 16);
        l.starter_count[b] = take(4);
    }
    l.scan_sums = take(((mk + 255) / 256) * 4);
    // localize in one launch: a count per block (at most 512 blocks), then one per block and partition (stores of
    // at most 1024 partitions; larger ones take the path that sorts by old owner)
    l.loc_counts = take((size_t)512 * 4 + (size_t)512 * (cfg.num_workers <= 1024 ? cfg.num_workers : 1) * 4);
    l.loc_scratch = take(mk * 5 * 4);
    l.upd = take(mk * (row_bytes > 32 ? row_bytes : 32));
    l.carry = take(reduce_tiles * 2 * (size_t)cfg.row_len * 8);
    l.group_sum = take(groups * (size_t)cfg.row_len * 8);
    l.loss_partial = take(tmax<size_t>(kMaxLossBlocks, mk / 256 + 1) * 8);
    l.apply_rows = take(mk * 8);
    for (int b = 0; b < kHostStages; ++b) l.staging[b] = take(mk * 8 + 256);
    l.total = off;
    return l;
}

struct ProfRec {
    const char* name;
    cudaEvent_t a, b;
};
struct Profile {
    std::vector<ProfRec> recs;
    size_t cap;
    bool open;          // an event pair has been started and not yet closed
};

void prof_before(ps_store* ps, const char* name, cudaStream_t s) {
    Profile* p = ps->prof;
    p->open = false;
    if (p->recs.size() >= p->cap) return;
    ProfRec r;
    r.name = name;
    if (cudaEventCreate(&r.a) != cudaSuccess) return;
    if (cudaEventCreate(&r.b) != cudaSuccess) {
        cudaEventDestroy(r.a);
        return;
    }
    // Every timed launch starts on an idle device, so that a kernel's time is its own and not that of
    // whatever the other stream runs beside it.  Profiling therefore serialises the calls it covers.
    cudaDeviceSynchronize();
    cudaEventRecord(r.a, s);
    p->recs.push_back(r);
    p->open = true;
}

void prof_after(ps_store* ps, cudaStream_t s) {
    Profile* p = ps->prof;
    if (p->open) cudaEventRecord(p->recs.back().b, s);
    p->open = false;
}

static ps_status_t cuda_ok(cudaError_t e) { return e == cudaSuccess ? PS_OK : PS_ERR_CUDA; }

static int bits_for(uint64_t max_value) {
    int b = 0;
    while (b < 32 && (max_value >> b) != 0) ++b;
    return b < 1 ? 1 : b;
}

static ps_status_t check_cfg(const ps_config_t* cfg) {
    if (!cfg) return PS_ERR_INVALID_ARG;
    if (cfg->num_keys == 0 || cfg->row_len == 0 || cfg->num_workers == 0) return PS_ERR_INVALID_ARG;
    if (cfg->num_keys >= 0xFFFFFFFFull) return PS_ERR_UNSUPPORTED;
    if (cfg->row_len % 4 != 0) return PS_ERR_UNSUPPORTED;
    if (cfg->num_workers > 65536) return PS_ERR_UNSUPPORTED;
    const uint64_t B = (cfg->num_keys + cfg->num_workers - 1) / cfg->num_workers;
    if (cfg->slots_per_part < B) return PS_ERR_INVALID_ARG;
    if (cfg->slots_per_part >= 0xFFFFFFFFull) return PS_ERR_UNSUPPORTED;
    return PS_OK;
}


// Errors raised by a launch itself (bad configuration) show up here; errors inside kernels
// are reported through the device status word.
static ps_status_t after_launch() { return cuda_ok(cudaGetLastError()); }


// Calls that sort rotate through the handle's sets of sort buffers.
static void next_epoch(ps_store* ps);
static SortSet* next_set(ps_store* ps) {
    // The call's number for the device-side error marks advances with the buffer sets: at most kSortSets such calls
    // are in flight, so their numbers never collide modulo the marks' slots (calls that sort nothing take no number).
    next_epoch(ps);
    ps->cur_set = (ps->cur_set + 1) % kSortSets;
    SortSet* ss = &ps->sets[ps->cur_set];
    ps->keysA = ss->keysA; ps->keysB = ss->keysB; ps->valsA = ss->valsA; ps->valsB = ss->valsB;
    ps->tile_state = ss->tile_state; ps->sort_ctl = ss->sort_ctl; ps->group_done = ss->group_done;
    ps->starters = ss->starters; ps->starter_count = ss->starter_count; ps->rec = ss->rec; ps->cellpos = ss->cellpos;
    ps->mf_dup = ss->mf_dup; ps->mf_tickets = ss->mf_tickets;
    ps->side_idx = 0;
    ps->side = ps->sides[0];
    return ss;
}
// For a call whose sort takes about as long as the rest of the step: successive calls take the side streams in
// turn, so that the sort of the step after next can run beside the sort of the next one (each has its own buffer set).
static void alternate_side(ps_store* ps) {
    static_assert(kSortSets >= kSideStreams + 1, "a sort in flight per internal stream and one set being read");
    ps->side_alt = (ps->side_alt + 1) % kSideStreams;
    ps->side_idx = ps->side_alt;
    ps->side = ps->sides[ps->side_idx];
}

// The keys of a step's occurrences depend on the batch alone, so their extraction and sort run on the
// handle's side stream while gradient kernels run on the caller's; both meet before the reduction.
// Ordered mode: the side stream starts after everything already enqueued on the caller's stream.
// Pipelined mode: it starts as soon as the buffer set's previous user is done, i.e. beside the previous
// step's kernels; the batch arrays must then be complete when the call is made.
static bool fork_side(ps_store* ps, SortSet* ss, cudaStream_t s, bool reads_table = false) {
    // for a relocation that may be asked to run beside this call (ps_localize_beside): everything earlier ends here
    ss->sorted_which = -1;
    if (cudaEventRecord(ps->ev_before, s) != cudaSuccess) return false;
    if (ss->loc_reader) {                           // a relocation on another stream was reading this set's sorted keys
        ss->loc_reader = false;
        if (cudaStreamWaitEvent(ps->side, ps->ev_loc, 0) != cudaSuccess) return false;
    }
    // When the caller's stream enters or leaves a CUDA-graph capture, events recorded on the other side of
    // that border cannot be waited on, and the side stream has to join (or leave) the capture: the first
    // call after such a change forks in ordered mode and forgets the older events.
    if (ps->batch_ready) {                  // the call's batch is still being copied from the host on the copy stream
        const cudaEvent_t ev = ps->batch_ready;
        ps->batch_ready = nullptr;
        if (cudaStreamWaitEvent(ps->side, ev, 0) != cudaSuccess) return false;
    }
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    unsigned long long id = 0;
    if (cudaStreamGetCaptureInfo(s, &cs, &id) != cudaSuccess) return false;
    if (cs != cudaStreamCaptureStatusActive) id = 0;
    if (id != ps->capture_id) {
        ps->capture_id = id;
        for (int b = 0; b < kSortSets; ++b) ps->sets[b].used = false;
    }
    const bool crossed = id != ps->side_capture_id[ps->side_idx];       // this side stream is still on the other side
    ps->side_capture_id[ps->side_idx] = id;
    // a sort that reads the location table (the matrix-factorization records) must come after a call that rewrote it
    // (every side stream on its own: the one that did not fork ordered has still not seen the rewrite)
    const bool ordered = crossed || (reads_table && ps->table_dirty[ps->side_idx]);
    if (ordered) ps->table_dirty[ps->side_idx] = false;
    if (ps->pipelined && !ordered) return !ss->used || cudaStreamWaitEvent(ps->side, ss->ev_free, 0) == cudaSuccess;
    return cudaEventRecord(ps->ev_fork, s) == cudaSuccess && cudaStreamWaitEvent(ps->side, ps->ev_fork, 0) == cudaSuccess;
}
static bool join_side(ps_store* ps, cudaStream_t s) {
    return cudaEventRecord(ps->ev_join, ps->side) == cudaSuccess && cudaStreamWaitEvent(s, ps->ev_join, 0) == cudaSuccess;
}
// after the call's sort has been enqueued on the side stream: where its sorted keys are, for ps_localize_beside
static bool sorted_keys_at(ps_store* ps, SortSet* ss, int which, uint32_t n) {
    ss->sorted_which = which;
    ss->sorted_n = n;
    ps->last_set = ss;
    return cudaEventRecord(ps->ev_sorted, ps->side) == cudaSuccess;
}
// after the last kernel of a call that used the set
static ps_status_t release_set(SortSet* ss, cudaStream_t s) {
    ss->used = true;
    if (cudaEventRecord(ss->ev_free, s) != cudaSuccess) return PS_ERR_CUDA;
    return cuda_ok(cudaGetLastError());
}

static void next_epoch(ps_store* ps) {
    ps->epoch++;
    if (ps->epoch == 0) ps->epoch = 1;
}

}  // namespace psb

using namespace psb;

extern "C" {

ps_status_t ps_query_sizes(const ps_config_t* cfg, uint64_t max_batch_keys, ps_sizes_t* out) {
    if (!out) return PS_ERR_INVALID_ARG;
    const ps_status_t c = check_cfg(cfg);
    if (c != PS_OK) return c;
    if (max_batch_keys == 0 || max_batch_keys >= (1ull << 30)) return PS_ERR_INVALID_ARG;
    const uint64_t N = cfg->num_workers, S = cfg->slots_per_part;
    out->store_bytes = (size_t)(N * S) * cfg->row_len * 4;
    out->table_bytes = (size_t)cfg->num_keys * 8;
    out->freelist_bytes = align_up((size_t)N * 8, 256) + (size_t)(N * S) * 4;
    out->workspace_bytes = ws_layout(*cfg, max_batch_keys).total;
    return PS_OK;
}

ps_status_t ps_create(const ps_config_t* cfg, void* d_store, void* d_table, void* d_freelists, void* d_workspace,
                      size_t workspace_bytes, uint64_t max_batch_keys, ps_store_t** out) {
    if (!out || !d_store || !d_table || !d_freelists || !d_workspace) return PS_ERR_INVALID_ARG;
    ps_sizes_t sz;
    const ps_status_t c = ps_query_sizes(cfg, max_batch_keys, &sz);
    if (c != PS_OK) return c;
    if (workspace_bytes < sz.workspace_bytes) return PS_ERR_WORKSPACE;
    if (((uintptr_t)d_store | (uintptr_t)d_table | (uintptr_t)d_freelists | (uintptr_t)d_workspace) & 15)
        return PS_ERR_INVALID_ARG;
    if (cudaSetDevice(cfg->device) != cudaSuccess) return PS_ERR_CUDA;
    ps_store* ps = new (std::nothrow) ps_store();
    if (!ps) return PS_ERR_INVALID_ARG;
    memset(ps, 0, sizeof(*ps));
    ps->cfg = *cfg;
    ps->max_keys = max_batch_keys;
    ps->key_bits = bits_for(cfg->num_keys);                 // keys 0..K, K marks "no key"
    ps->sort_blocks_cap = div_up_u32(max_batch_keys, kSortTile / 2);
    ps->owner_bits = bits_for(cfg->num_workers - 1);
    ps->store = (float*)d_store;
    ps->table = (uint2*)d_table;
    ps->tops = (unsigned long long*)d_freelists;
    ps->stacks = (uint32_t*)((char*)d_freelists + align_up((size_t)cfg->num_workers * 8, 256));
    ps->ws = (char*)d_workspace;
    ps->ws_bytes = workspace_bytes;
    const WsLayout l = ws_layout(*cfg, max_batch_keys);
    ps->status = (DevStatus*)(ps->ws + l.status);
    for (int b = 0; b < kSortSets; ++b) {
        SortSet& ss = ps->sets[b];
        ss.keysA = (uint32_t*)(ps->ws + l.keysA[b]);
        ss.keysB = (uint32_t*)(ps->ws + l.keysB[b]);
        ss.valsA = (uint32_t*)(ps->ws + l.valsA[b]);
        ss.valsB = (uint32_t*)(ps->ws + l.valsB[b]);
        ss.tile_state = (uint32_t*)(ps->ws + l.tile_state[b]);
        ss.sort_ctl = (uint32_t*)(ps->ws + l.sort_ctl[b]);
        ss.group_done = ss.sort_ctl + kSortCtlWords;
        ss.rec = (uint4*)(ps->ws + l.rec[b]);
        ss.cellpos = (uint32_t*)(ps->ws + l.cellpos[b]);
        ss.mf_dup = (uint4*)(ps->ws + l.mf_dup[b]);
        ss.mf_tickets = (unsigned int*)(ps->ws + l.mf_tickets[b]);
        ss.starters = (uint4*)(ps->ws + l.starters[b]);
        ss.starter_count = (unsigned int*)(ps->ws + l.starter_count[b]);
        ss.used = false;
    }
    ps->cur_set = kSortSets - 1;
    next_set(ps);
    ps->scan_sums = (uint32_t*)(ps->ws + l.scan_sums);
    ps->loc_counts = (uint32_t*)(ps->ws + l.loc_counts);
    ps->loc_scratch = (uint32_t*)(ps->ws + l.loc_scratch);
    ps->upd = (float*)(ps->ws + l.upd);
    ps->carry = (double*)(ps->ws + l.carry);
    ps->group_sum = (double*)(ps->ws + l.group_sum);
    ps->loss_partial = (double*)(ps->ws + l.loss_partial);
    ps->apply_rows = (uint64_t*)(ps->ws + l.apply_rows);
    for (int b = 0; b < kHostStages; ++b) ps->stagings[b] = ps->ws + l.staging[b];
    ps->staging = ps->stagings[0];
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess || sms <= 0) {
        delete ps;
        return PS_ERR_CUDA;
    }
    ps->sm_count = sms;
    if (cudaMemset(ps->status, 0, sizeof(DevStatus)) != cudaSuccess) {
        delete ps;
        return PS_ERR_CUDA;
    }
    // the sort's grid barrier re-arms itself after every use, but has to start from zero
    for (int b = 0; b < kSortSets; ++b)
        if (cudaMemset(ps->sets[b].sort_ctl, 0, kSortCtlWords * sizeof(uint32_t)) != cudaSuccess) {
            delete ps;
            return PS_ERR_CUDA;
        }
    // the side stream's small kernels should not queue behind the gradient kernel's waves of blocks
    int prio_lo = 0, prio_hi = 0;
    cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);
    for (int b = 0; b < kSideStreams; ++b)
        if (cudaStreamCreateWithPriority(&ps->sides[b], cudaStreamNonBlocking, prio_hi) != cudaSuccess) {
            delete ps;
            return PS_ERR_CUDA;
        }
    if (cudaEventCreateWithFlags(&ps->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ps->ev_join, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ps->ev_before, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ps->ev_sorted, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ps->ev_loc, cudaEventDisableTiming) != cudaSuccess) {
        delete ps;
        return PS_ERR_CUDA;
    }
    for (int b = 0; b < kSortSets; ++b)
        if (cudaEventCreateWithFlags(&ps->sets[b].ev_free, cudaEventDisableTiming) != cudaSuccess) {
            delete ps;
            return PS_ERR_CUDA;
        }
    if (cudaStreamCreateWithFlags(&ps->copy, cudaStreamNonBlocking) != cudaSuccess) {
        delete ps;
        return PS_ERR_CUDA;
    }
    for (int b = 0; b < kHostStages; ++b)
        if (cudaEventCreateWithFlags(&ps->ev_copied[b], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ps->ev_consumed[b], cudaEventDisableTiming) != cudaSuccess) {
            delete ps;
            return PS_ERR_CUDA;
        }
    // The store as a 2-D tensor for the TMA unit: one instruction of the matrix-factorization step then fetches four
    // rows (tile::gather4).  Rows of up to 256 values, row numbers that fit a signed 32-bit coordinate; where the
    // driver lacks the entry point or refuses the shape, the step uses one bulk copy per row instead.
    ps->row_map_ok = false;
    if (cfg->row_len <= 256 && (uint64_t)cfg->num_workers * cfg->slots_per_part < (1ull << 31)) {
        typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                      const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) == cudaSuccess && fn &&
            qr == cudaDriverEntryPointSuccess) {
            const cuuint64_t dims[2] = {cfg->row_len, (cuuint64_t)cfg->num_workers * cfg->slots_per_part};
            const cuuint64_t strides[1] = {(cuuint64_t)cfg->row_len * 4};
            const cuuint32_t box[2] = {cfg->row_len, 1};
            const cuuint32_t estr[2] = {1, 1};
            const CUresult r = ((encode_fn)fn)(&ps->row_map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, d_store, dims, strides, box,
                                               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                               CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            ps->row_map_ok = r == CUDA_SUCCESS;
        }
        cudaGetLastError();
    }
    *out = ps;
    return PS_OK;
}

ps_status_t ps_destroy(ps_store_t* ps) {
    if (!ps) return PS_ERR_INVALID_ARG;
    cudaSetDevice(ps->cfg.device);
    cudaDeviceSynchronize();
    if (ps->prof) ps_profile_stop(ps, nullptr, 0);
    cudaEventDestroy(ps->ev_fork);
    cudaEventDestroy(ps->ev_join);
    cudaEventDestroy(ps->ev_before);
    cudaEventDestroy(ps->ev_sorted);
    cudaEventDestroy(ps->ev_loc);
    for (int b = 0; b < kSortSets; ++b) cudaEventDestroy(ps->sets[b].ev_free);
    for (int b = 0; b < kSideStreams; ++b) cudaStreamDestroy(ps->sides[b]);
    cudaStreamDestroy(ps->copy);
    for (int b = 0; b < kHostStages; ++b) {
        cudaEventDestroy(ps->ev_copied[b]);
        cudaEventDestroy(ps->ev_consumed[b]);
    }
    delete ps;
    return PS_OK;
}

// a relocation enqueued on another stream by ps_localize_beside comes before every later call of the handle
static bool after_relocation(ps_store* ps, cudaStream_t s) {
    ps->last_set = nullptr;
    ps->last_stream = s;
    return !ps->loc_pending || cudaStreamWaitEvent(s, ps->ev_loc, 0) == cudaSuccess;
}

#define PS_BEGIN_CALL(ps)                                            \
    if (!(ps)) return PS_ERR_INVALID_ARG;                           \
    cudaStream_t s = (cudaStream_t)stream;                          \
    if (!after_relocation(ps, s)) return PS_ERR_CUDA;

ps_status_t ps_init_range_partition(ps_store_t* ps, void* stream) {
    PS_BEGIN_CALL(ps);
    launch_init_range_partition(ps, s);
    for (int b = 0; b < kSideStreams; ++b) ps->table_dirty[b] = true;
    return after_launch();
}

ps_status_t ps_set_rows(ps_store_t* ps, const uint64_t* d_keys, uint64_t n, const float* d_vals, void* stream) {
    PS_BEGIN_CALL(ps);
    if (n == 0) return PS_OK;
    if (!d_keys || !d_vals || ((uintptr_t)d_vals & 15)) return PS_ERR_INVALID_ARG;
    launch_set_rows(ps, d_keys, n, d_vals, s);
    return after_launch();
}

ps_status_t ps_pull(ps_store_t* ps, const uint64_t* d_keys, uint64_t n, float* d_out, void* stream) {
    PS_BEGIN_CALL(ps);
    if (n == 0) return PS_OK;
    if (!d_keys || !d_out || ((uintptr_t)d_out & 15)) return PS_ERR_INVALID_ARG;
    launch_pull(ps, d_keys, n, d_out, s);
    return after_launch();
}

ps_status_t ps_push(ps_store_t* ps, const uint64_t* d_keys, uint64_t n, const float* d_updates, void* stream) {
    PS_BEGIN_CALL(ps);
    if (n == 0) return PS_OK;
    if (!d_keys || !d_updates || ((uintptr_t)d_updates & 15)) return PS_ERR_INVALID_ARG;
    if (ps->push_mode == PS_PUSH_ATOMIC) {
        SortSet* ss = next_set(ps);                         // (for the call's number; nothing is sorted)
        run_push_atomic(ps, d_keys, n, d_updates, s);
        return release_set(ss, s);
    }
    if (n > ps->max_keys) return PS_ERR_WORKSPACE;
    SortSet* ss = next_set(ps);
    if (!fork_side(ps, ss, s)) return PS_ERR_CUDA;         // the keys are sorted beside earlier calls' kernels
    const int which = radix_sort_keys64(ps, d_keys, (uint32_t)n, ps->side, ps->starter_count,
                                        div_up_u32(n, kGroupSpan));
    if (!sorted_keys_at(ps, ss, which, (uint32_t)n) || !join_side(ps, s)) return PS_ERR_CUDA;
    run_push_reduce(ps, (uint32_t)n, which, d_updates, nullptr, 0, s);
    return release_set(ss, s);
}

ps_status_t ps_localize(ps_store_t* ps, uint32_t worker, const uint64_t* d_keys, uint64_t n, void* stream) {
    PS_BEGIN_CALL(ps);
    if (worker >= ps->cfg.num_workers) return PS_ERR_WORKER_RANGE;
    if (n == 0) return PS_OK;
    if (!d_keys) return PS_ERR_INVALID_ARG;
    if (n > ps->max_keys) return PS_ERR_WORKSPACE;
    // stores of more than 1024 partitions: one block scans the call's per-chunk counts in shared memory
    if (n > (1u << 20) && ps->cfg.num_workers > 1024) return PS_ERR_UNSUPPORTED;
    SortSet* ss = next_set(ps);
    if (!fork_side(ps, ss, s)) return PS_ERR_CUDA;
    const int which = radix_sort_keys64(ps, d_keys, (uint32_t)n, ps->side, nullptr, 0);
    if (!join_side(ps, s)) return PS_ERR_CUDA;
    run_localize(ps, worker, (uint32_t)n, which, s);
    for (int b = 0; b < kSideStreams; ++b) ps->table_dirty[b] = true;
    return release_set(ss, s);
}

ps_status_t ps_localize_beside(ps_store_t* ps, uint32_t worker, const uint64_t* d_keys, uint64_t n, void* loc_stream) {
    if (!ps) return PS_ERR_INVALID_ARG;
    cudaStream_t ls = (cudaStream_t)loc_stream;
    // Nothing to run beside (the most recent call sorted no keys, or was made on this very stream), or a store
    // with more partitions than the one-launch relocation serves: an ordinary localize, after everything so far.
    SortSet* busy = ps->last_set;
    if (!busy || busy->sorted_which < 0 || ps->last_stream == ls || ps->cfg.num_workers > 1024) {
        if (ps->last_stream != ls) {
            if (cudaEventRecord(ps->ev_before, ps->last_stream) != cudaSuccess ||
                cudaStreamWaitEvent(ls, ps->ev_before, 0) != cudaSuccess)
                return PS_ERR_CUDA;
        }
        const cudaStream_t was = ps->last_stream;
        const ps_status_t c = ps_localize(ps, worker, d_keys, n, loc_stream);
        if (c != PS_OK || n == 0 || was == ls) return c;
        if (cudaEventRecord(ps->ev_loc, ls) != cudaSuccess) return PS_ERR_CUDA;
        ps->loc_pending = true;
        return PS_OK;
    }
    if (worker >= ps->cfg.num_workers) return PS_ERR_WORKER_RANGE;
    if (n == 0) return PS_OK;
    if (!d_keys) return PS_ERR_INVALID_ARG;
    if (n > ps->max_keys) return PS_ERR_WORKSPACE;
    // an earlier relocation of this kind comes first; so does everything before the call to run beside, and that
    // call's key sort, whose result says which keys it touches
    if (ps->loc_pending && cudaStreamWaitEvent(ls, ps->ev_loc, 0) != cudaSuccess) return PS_ERR_CUDA;
    if (cudaStreamWaitEvent(ls, ps->ev_before, 0) != cudaSuccess || cudaStreamWaitEvent(ls, ps->ev_sorted, 0) != cudaSuccess)
        return PS_ERR_CUDA;
    const uint32_t* busy_keys = busy->sorted_which ? busy->keysB : busy->keysA;
    const uint32_t n_busy = busy->sorted_n;
    const cudaEvent_t busy_done = busy->ev_free;
    SortSet* ss = next_set(ps);
    ss->sorted_which = -1;
    const int which = radix_sort_keys64(ps, d_keys, (uint32_t)n, ls, nullptr, 0);
    run_localize(ps, worker, (uint32_t)n, which, ls, busy_keys, n_busy);
    if (cudaStreamWaitEvent(ls, busy_done, 0) != cudaSuccess) return PS_ERR_CUDA;
    run_localize_deferred(ps, worker, (uint32_t)n, ls);
    // (a later sort that reads the table forks after the caller's stream, which waits for ev_loc: table_dirty)
    for (int b = 0; b < kSideStreams; ++b) ps->table_dirty[b] = true;
    busy->loc_reader = true;
    if (cudaEventRecord(ps->ev_loc, ls) != cudaSuccess) return PS_ERR_CUDA;
    ps->loc_pending = true;
    ps->last_set = nullptr;                         // (a second relocation beside the same call would have to wait for this one's deferred half)
    return release_set(ss, ls);
}

ps_status_t ps_localize_stats(ps_store_t* ps, ps_localize_stats_t* h_out) {
    if (!ps || !h_out) return PS_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return PS_ERR_CUDA;
    DevStatus st;
    if (cudaMemcpy(&st, ps->status, sizeof st, cudaMemcpyDeviceToHost) != cudaSuccess) return PS_ERR_CUDA;
    h_out->requested = st.loc_requested;
    h_out->moved = st.rows_moved;
    h_out->already_local = st.loc_already_local;
    h_out->moved_again = st.loc_moved_again;
    h_out->deferred = st.loc_deferred;
    return PS_OK;
}

ps_status_t ps_step_mf(ps_store_t* ps, const uint32_t* d_i, const uint32_t* d_j, const float* d_v, uint64_t n,
                       uint64_t col_key_base, float lr, float lambda, double* d_loss_accum, void* stream) {
    PS_BEGIN_CALL(ps);
    if (n == 0) return PS_OK;
    if (!d_i || !d_j || !d_v) return PS_ERR_INVALID_ARG;
    if (2 * n > ps->max_keys) return PS_ERR_WORKSPACE;
    if (col_key_base > ps->cfg.num_keys) return PS_ERR_INVALID_ARG;
    SortSet* ss = next_set(ps);
    alternate_side(ps);
    if (!fork_side(ps, ss, s, true)) return PS_ERR_CUDA;
    // rows short enough to be staged whole, and row numbers that fit the 32-bit fields of the sort's records
    const bool fused = ps->cfg.row_len <= 128 && (uint64_t)ps->cfg.num_workers * ps->cfg.slots_per_part < (1ull << 32);
    // The one-launch form over the column side is taken on request only: on the 10M x 1M matrix it runs at 49 us
    // per step against 45 for the symmetric form (its launch takes 35 to 41 us, the two of the symmetric form 42,
    // but it adds a kernel to the internal stream, whose sort is what bounds the step).
    const bool by_column = fused && ps->mf_path == 1;
    const int which = radix_sort_mf(ps, d_i, d_j, d_v, (uint32_t)n, col_key_base, fused, ps->side, ps->starter_count,
                                    div_up_u32(2 * n, fused ? 64 * 8 : kGroupSpan));
    if (!sorted_keys_at(ps, ss, which, (uint32_t)(2 * n))) return PS_ERR_CUDA;
    if (by_column) {
        launch_mf_plan(ps, (uint32_t)n, which, ps->side);
        if (!join_side(ps, s)) return PS_ERR_CUDA;
        run_mf_col(ps, (uint32_t)n, which, lr, lambda, d_loss_accum, s);
        return release_set(ss, s);
    }
    if (fused) {
        // gradient and reduction in one kernel over the sorted occurrences: no update rows
        if (!join_side(ps, s)) return PS_ERR_CUDA;
        run_mf_fused(ps, (uint32_t)n, which, col_key_base, lr, lambda, d_loss_accum, s,
                     ps->row_map_ok && ps->mf_path != PS_MF_SYMMETRIC_ROW_COPIES);
        return release_set(ss, s);
    }
    const uint32_t lb = launch_step_mf(ps, d_i, d_j, d_v, n, col_key_base, lr, lambda, s);
    if (!join_side(ps, s)) return PS_ERR_CUDA;
    run_push_reduce(ps, (uint32_t)(2 * n), which, ps->upd, d_loss_accum, d_loss_accum ? lb : 0, s);
    return release_set(ss, s);
}

ps_status_t ps_step_kge(ps_store_t* ps, const uint32_t* d_s, const uint32_t* d_r, const uint32_t* d_o,
                        const uint32_t* d_neg_ent, const uint8_t* d_neg_side, uint64_t n, uint32_t n_neg,
                        uint64_t rel_key_base, uint32_t dim_complex, float lr, float eps, double* d_loss_accum,
                        void* stream) {
    PS_BEGIN_CALL(ps);
    if (n == 0) return PS_OK;
    if (!d_s || !d_r || !d_o || (n_neg && (!d_neg_ent || !d_neg_side))) return PS_ERR_INVALID_ARG;
    if (n_neg > 29) return PS_ERR_UNSUPPORTED;
    if (dim_complex == 0 || ps->cfg.row_len != 4 * (uint64_t)dim_complex) return PS_ERR_INVALID_ARG;
    if ((3 + (uint64_t)n_neg) * n > ps->max_keys) return PS_ERR_WORKSPACE;
    if (rel_key_base > ps->cfg.num_keys) return PS_ERR_INVALID_ARG;
    const uint32_t occ = (uint32_t)((3 + (uint64_t)n_neg) * n);
    SortSet* ss = next_set(ps);
    if (!fork_side(ps, ss, s)) return PS_ERR_CUDA;
    launch_keys_kge(ps, d_s, d_r, d_o, d_neg_ent, n, n_neg, rel_key_base, ps->side);
    const int which = run_push_sort(ps, occ, ps->side);
    if (!sorted_keys_at(ps, ss, which, occ)) return PS_ERR_CUDA;
    // gradient rows + AdaGrad inside the reduction where a gradient row is whole float4s and fits the reduction's staging
    const bool grad_only = dim_complex % 2 == 0 && dim_complex <= 128;
    const uint32_t lb = launch_step_kge(ps, d_s, d_r, d_o, d_neg_ent, d_neg_side, n, n_neg, rel_key_base, dim_complex,
                                        lr, eps, grad_only, s);
    if (!join_side(ps, s)) return PS_ERR_CUDA;
    if (grad_only) run_kge_reduce(ps, occ, which, dim_complex, lr, eps, d_loss_accum, d_loss_accum ? lb : 0, s);
    else run_push_reduce(ps, occ, which, ps->upd, d_loss_accum, d_loss_accum ? lb : 0, s);
    return release_set(ss, s);
}

ps_status_t ps_step_rescal(ps_store_t* ps, const uint32_t* d_s, const uint32_t* d_r, const uint32_t* d_o,
                           const uint32_t* d_neg_ent, const uint8_t* d_neg_side, uint64_t n, uint32_t n_neg,
                           uint64_t rel_key_base, uint32_t dim, float lr, float eps, double* d_loss_accum,
                           void* stream) {
    PS_BEGIN_CALL(ps);
    if (n == 0) return PS_OK;
    if (!d_s || !d_r || !d_o || (n_neg && (!d_neg_ent || !d_neg_side))) return PS_ERR_INVALID_ARG;
    if (n_neg > 29 || dim < 4 || dim > 128 || dim % 4 != 0) return PS_ERR_UNSUPPORTED;
    if (ps->cfg.row_len != 2 * (uint64_t)dim) return PS_ERR_INVALID_ARG;
    if ((2 + (uint64_t)n_neg + dim) * n > ps->max_keys) return PS_ERR_WORKSPACE;
    if (rel_key_base > ps->cfg.num_keys) return PS_ERR_INVALID_ARG;
    const uint32_t occ = (uint32_t)((2 + (uint64_t)n_neg + dim) * n);
    SortSet* ss = next_set(ps);
    if (!fork_side(ps, ss, s)) return PS_ERR_CUDA;
    launch_keys_rescal(ps, d_s, d_r, d_o, d_neg_ent, n, n_neg, rel_key_base, dim, ps->side);
    const int which = run_push_sort(ps, occ, ps->side);
    if (!sorted_keys_at(ps, ss, which, occ)) return PS_ERR_CUDA;
    // gradient rows of dim values per occurrence; AdaGrad inside the reduction, to which a row [dim | dim] is what
    // [Re Im | G_Re G_Im] of dim / 2 complex dimensions is
    const uint32_t lb = launch_grad_rescal(ps, d_s, d_r, d_o, d_neg_ent, d_neg_side, n, n_neg, rel_key_base, dim, s);
    if (!join_side(ps, s)) return PS_ERR_CUDA;
    run_kge_reduce(ps, occ, which, dim / 2, lr, eps, d_loss_accum, d_loss_accum ? lb : 0, s);
    return release_set(ss, s);
}

// ---- self-test of the bounded waits ----
// Two blocks meet at the sort's grid barrier and wait for a third arrival that never comes.  The wait is bounded
// (kBarrierSpins polls, about a fifth of a second): the blocks give up, latch PS_ERR_CUDA and return, leaving the
// barrier's count where it stood, which is the state ps_sync has to clean up after a sort that gave up.
__global__ void barrier_timeout_kernel(unsigned int* bar, DevStatus* st) {
    __shared__ int s_ok;
    if (!grid_barrier(bar, gridDim.x + 1, &s_ok) && threadIdx.x == 0) atomicCAS(&st->sticky, 0u, (unsigned int)PS_ERR_CUDA);
}

ps_status_t ps_selftest_barrier_timeout(ps_store_t* ps, void* stream) {
    PS_BEGIN_CALL(ps);
    SortSet* ss = next_set(ps);
    unsigned int* bar = ps->sort_ctl;
    DevStatus* st = ps->status;
    void* args[] = {(void*)&bar, (void*)&st};
    cudaLaunchCooperativeKernel((const void*)barrier_timeout_kernel, dim3(2), dim3(64), args, 0, s);
    ps->launches++;
    return release_set(ss, s);
}

// ---- parameter blocking for matrix factorization ----
__global__ void key_range_kernel(uint64_t* out, uint64_t first, uint64_t n) {
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < n) out[t] = first + t;
}

// localize(worker, keys first .. first + count), in pieces the workspace has room for
static ps_status_t localize_range(ps_store* ps, uint32_t worker, uint64_t first, uint64_t count, void* stream) {
    cudaStream_t s = (cudaStream_t)stream;
    uint64_t* d_keys = (uint64_t*)ps->stagings[0];
    for (uint64_t done = 0; done < count;) {
        const uint64_t c = tmin<uint64_t>(count - done, ps->max_keys);
        key_range_kernel<<<div_up_u32(c, 256), 256, 0, s>>>(d_keys, first + done, c);
        ps->launches++;
        const ps_status_t rc = ps_localize(ps, worker, d_keys, c, stream);
        if (rc != PS_OK) return rc;
        done += c;
    }
    return PS_OK;
}

ps_status_t ps_dsgd_epoch_mf(ps_store_t* ps, const uint32_t* d_i, const uint32_t* d_j, const float* d_v,
                             const uint64_t* h_offsets, uint64_t rows, uint64_t cols, uint64_t batch, float lr,
                             float lambda, double* d_loss_accum, void* stream) {
    if (!ps || !d_i || !d_j || !d_v || !h_offsets || batch == 0) return PS_ERR_INVALID_ARG;
    const uint64_t N = ps->cfg.num_workers;
    if (rows == 0 || cols == 0 || rows + cols != ps->cfg.num_keys) return PS_ERR_INVALID_ARG;
    for (uint64_t x = 0; x < N * N; ++x)
        if (h_offsets[x] > h_offsets[x + 1]) return PS_ERR_INVALID_ARG;
    const uint64_t rsize = (rows + N - 1) / N, csize = (cols + N - 1) / N;
    // The key lists of the relocations are written on the caller's stream right before use: their sorts must
    // not start ahead of that, so the relocations run in ordered mode whatever the handle is set to.
    const bool was = ps->pipelined;
    ps_status_t rc = PS_OK;
    ps->pipelined = false;
    for (uint64_t w = 0; w < N && rc == PS_OK; ++w)            // a worker's row factors live with it throughout
        if (w * rsize < rows) rc = localize_range(ps, (uint32_t)w, w * rsize, tmin<uint64_t>(rsize, rows - w * rsize), stream);
    for (uint64_t sub = 0; sub < N && rc == PS_OK; ++sub) {
        // subepoch start: worker w localizes column block (w + sub) mod N (stream order is the barrier between subepochs)
        ps->pipelined = false;
        for (uint64_t w = 0; w < N && rc == PS_OK; ++w) {
            const uint64_t blk = (w + sub) % N;
            if (blk * csize < cols)
                rc = localize_range(ps, (uint32_t)w, rows + blk * csize, tmin<uint64_t>(csize, cols - blk * csize), stream);
        }
        ps->pipelined = was;
        // the workers' strata: no two of them share a parameter, so their minibatches are independent
        for (uint64_t w = 0; w < N && rc == PS_OK; ++w) {
            const uint64_t lo = h_offsets[sub * N + w], hi = h_offsets[sub * N + w + 1];
            for (uint64_t at = lo; at < hi && rc == PS_OK; at += batch) {
                const uint64_t c = tmin<uint64_t>(batch, hi - at);
                rc = ps_step_mf(ps, d_i + at, d_j + at, d_v + at, c, rows, lr, lambda, d_loss_accum, stream);
            }
        }
    }
    ps->pipelined = was;
    return rc;
}

static ps_status_t sgns_checks(ps_store_t* ps, uint64_t first_pos, uint64_t n_centers, uint64_t corpus_len,
                               uint32_t window, uint32_t n_neg, uint64_t out_key_base, uint64_t* occ) {
    if (first_pos + n_centers > corpus_len) return PS_ERR_INVALID_ARG;
    if (ps->cfg.row_len > 512) return PS_ERR_UNSUPPORTED;
    if (out_key_base > ps->cfg.num_keys) return PS_ERR_INVALID_ARG;
    *occ = n_centers * (1 + (uint64_t)2 * window * (1 + (uint64_t)n_neg));
    // two source rows per center and one factor per slot share the update buffer
    if (*occ > ps->max_keys || 3 * n_centers > ps->max_keys) return PS_ERR_WORKSPACE;
    return PS_OK;
}

ps_status_t ps_step_sgns(ps_store_t* ps, const uint32_t* d_tokens, uint64_t first_pos, uint64_t n_centers,
                         uint64_t corpus_len, uint32_t window, const uint32_t* d_negs, uint32_t n_neg,
                         uint64_t out_key_base, float lr, double* d_loss_accum, void* stream) {
    PS_BEGIN_CALL(ps);
    if (n_centers == 0) return PS_OK;
    if (!d_tokens || (n_neg && window && !d_negs)) return PS_ERR_INVALID_ARG;
    uint64_t occ;
    const ps_status_t c = sgns_checks(ps, first_pos, n_centers, corpus_len, window, n_neg, out_key_base, &occ);
    if (c != PS_OK) return c;
    SortSet* ss = next_set(ps);
    if (!fork_side(ps, ss, s)) return PS_ERR_CUDA;
    launch_keys_sgns(ps, d_tokens, 0, first_pos, n_centers, corpus_len, window, d_negs, n_neg, out_key_base, ps->side);
    const int which = run_push_sort(ps, (uint32_t)occ, ps->side);
    if (!sorted_keys_at(ps, ss, which, (uint32_t)occ)) return PS_ERR_CUDA;
    const uint32_t lb = launch_step_sgns(ps, d_tokens, 0, first_pos, n_centers, corpus_len, window, d_negs, n_neg,
                                         out_key_base, lr, s);
    if (!join_side(ps, s)) return PS_ERR_CUDA;
    run_push_reduce(ps, (uint32_t)occ, which, ps->upd, d_loss_accum, d_loss_accum ? lb : 0, s,
                    sgns_scales(ps, n_centers), (uint32_t)(occ / n_centers));
    return release_set(ss, s);
}

// ---- host-batch variants ----
// Where a host batch is copied to and on which stream.  Plain mode: the one staging area, the caller's stream.
// Overlapped mode (ps_set_host_overlap): the next of kHostStages areas, on the handle's copy stream, as soon as
// the step that last read that area is through; the step's kernels then wait for the copy, not the other way round.
struct HostBatch {
    char* buf;
    cudaStream_t cs;
    int slot;               // -1 in plain mode
};
static bool host_batch_begin(ps_store* ps, cudaStream_t s, HostBatch* hb) {
    if (!ps->host_overlap) {
        hb->buf = ps->stagings[0];
        hb->cs = s;
        hb->slot = -1;
        return true;
    }
    ps->host_slot = (ps->host_slot + 1) % kHostStages;
    hb->slot = ps->host_slot;
    hb->buf = ps->stagings[hb->slot];
    hb->cs = ps->copy;
    return !ps->consumed_valid[hb->slot] || cudaStreamWaitEvent(ps->copy, ps->ev_consumed[hb->slot], 0) == cudaSuccess;
}
// after the copies have been enqueued: every stream that reads the batch waits for them
static bool host_batch_copied(ps_store* ps, cudaStream_t s, const HostBatch& hb) {
    if (hb.slot < 0) return true;
    if (cudaEventRecord(ps->ev_copied[hb.slot], ps->copy) != cudaSuccess ||
        cudaStreamWaitEvent(s, ps->ev_copied[hb.slot], 0) != cudaSuccess)
        return false;
    ps->batch_ready = ps->ev_copied[hb.slot];       // picked up by the step's fork of the side stream
    return true;
}
static ps_status_t finish_host_step(ps_store* ps, const HostBatch& hb, double* d_loss_accum, double* h_loss,
                                    cudaStream_t s) {
    if (d_loss_accum && h_loss &&
        cudaMemcpyAsync(h_loss, d_loss_accum, sizeof(double), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return PS_ERR_CUDA;
    if (hb.slot >= 0) {                              // overlapped mode: nothing waits; the area is free once s gets here
        if (cudaEventRecord(ps->ev_consumed[hb.slot], s) != cudaSuccess) return PS_ERR_CUDA;
        ps->consumed_valid[hb.slot] = true;
        return PS_OK;
    }
    if (cudaStreamSynchronize(s) != cudaSuccess) return PS_ERR_CUDA;
    return PS_OK;
}

ps_status_t ps_step_mf_host(ps_store_t* ps, const uint32_t* h_i, const uint32_t* h_j, const float* h_v, uint64_t n,
                            uint64_t col_key_base, float lr, float lambda, double* d_loss_accum, double* h_loss,
                            void* stream) {
    if (!ps) return PS_ERR_INVALID_ARG;
    if (n == 0) return PS_OK;
    if (!h_i || !h_j || !h_v) return PS_ERR_INVALID_ARG;
    if (2 * n > ps->max_keys) return PS_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    HostBatch hb;
    if (!host_batch_begin(ps, s, &hb)) return PS_ERR_CUDA;
    uint32_t* d_i = (uint32_t*)hb.buf;
    uint32_t* d_j = d_i + n;
    float* d_v = (float*)(d_j + n);
    if (cudaMemcpyAsync(d_i, h_i, n * 4, cudaMemcpyHostToDevice, hb.cs) != cudaSuccess ||
        cudaMemcpyAsync(d_j, h_j, n * 4, cudaMemcpyHostToDevice, hb.cs) != cudaSuccess ||
        cudaMemcpyAsync(d_v, h_v, n * 4, cudaMemcpyHostToDevice, hb.cs) != cudaSuccess)
        return PS_ERR_CUDA;
    if (!host_batch_copied(ps, s, hb)) return PS_ERR_CUDA;
    const bool was = ps->pipelined;         // plain mode: the batch arrives on the caller's stream, order the side stream after it
    if (hb.slot < 0) ps->pipelined = false;
    const ps_status_t c = ps_step_mf(ps, d_i, d_j, d_v, n, col_key_base, lr, lambda, d_loss_accum, stream);
    ps->pipelined = was;
    if (c != PS_OK) return c;
    return finish_host_step(ps, hb, d_loss_accum, h_loss, s);
}

ps_status_t ps_step_kge_host(ps_store_t* ps, const uint32_t* h_s, const uint32_t* h_r, const uint32_t* h_o,
                             const uint32_t* h_neg_ent, const uint8_t* h_neg_side, uint64_t n, uint32_t n_neg,
                             uint64_t rel_key_base, uint32_t dim_complex, float lr, float eps, double* d_loss_accum,
                             double* h_loss, void* stream) {
    if (!ps) return PS_ERR_INVALID_ARG;
    if (n == 0) return PS_OK;
    if (!h_s || !h_r || !h_o || (n_neg && (!h_neg_ent || !h_neg_side))) return PS_ERR_INVALID_ARG;
    if ((3 + (uint64_t)n_neg) * n > ps->max_keys) return PS_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    HostBatch hb;
    if (!host_batch_begin(ps, s, &hb)) return PS_ERR_CUDA;
    uint32_t* d_s = (uint32_t*)hb.buf;
    uint32_t* d_r = d_s + n;
    uint32_t* d_o = d_r + n;
    uint32_t* d_ne = d_o + n;
    uint8_t* d_ns = (uint8_t*)(d_ne + n * n_neg);
    if (cudaMemcpyAsync(d_s, h_s, n * 4, cudaMemcpyHostToDevice, hb.cs) != cudaSuccess ||
        cudaMemcpyAsync(d_r, h_r, n * 4, cudaMemcpyHostToDevice, hb.cs) != cudaSuccess ||
        cudaMemcpyAsync(d_o, h_o, n * 4, cudaMemcpyHostToDevice, hb.cs) != cudaSuccess)
        return PS_ERR_CUDA;
    if (n_neg && (cudaMemcpyAsync(d_ne, h_neg_ent, n * n_neg * 4, cudaMemcpyHostToDevice, hb.cs) != cudaSuccess ||
                  cudaMemcpyAsync(d_ns, h_neg_side, n * n_neg, cudaMemcpyHostToDevice, hb.cs) != cudaSuccess))
        return PS_ERR_CUDA;
    if (!host_batch_copied(ps, s, hb)) return PS_ERR_CUDA;
    const bool was = ps->pipelined;         // plain mode: the batch arrives on the caller's stream, order the side stream after it
    if (hb.slot < 0) ps->pipelined = false;
    const ps_status_t c = ps_step_kge(ps, d_s, d_r, d_o, d_ne, d_ns, n, n_neg, rel_key_base, dim_complex, lr, eps,
                                      d_loss_accum, stream);
    ps->pipelined = was;
    if (c != PS_OK) return c;
    return finish_host_step(ps, hb, d_loss_accum, h_loss, s);
}

ps_status_t ps_step_sgns_host(ps_store_t* ps, const uint32_t* h_tokens, uint64_t tok_first, uint64_t tok_count,
                              uint64_t first_pos, uint64_t n_centers, uint64_t corpus_len, uint32_t window,
                              const uint32_t* h_negs, uint64_t n_negs, uint32_t n_neg, uint64_t out_key_base,
                              float lr, double* d_loss_accum, double* h_loss, void* stream) {
    if (!ps) return PS_ERR_INVALID_ARG;
    if (n_centers == 0) return PS_OK;
    if (!h_tokens || (n_negs && !h_negs)) return PS_ERR_INVALID_ARG;
    uint64_t occ;
    ps_status_t c = sgns_checks(ps, first_pos, n_centers, corpus_len, window, n_neg, out_key_base, &occ);
    if (c != PS_OK) return c;
    // the tokens handed over must cover the batch's window
    const uint64_t need_lo = first_pos >= window ? first_pos - window : 0;
    uint64_t need_hi = first_pos + n_centers - 1 + window;
    if (need_hi > corpus_len - 1) need_hi = corpus_len - 1;
    if (tok_first > need_lo || tok_first + tok_count <= need_hi) return PS_ERR_INVALID_ARG;
    if ((tok_count + n_negs) * 4 > ps->max_keys * 8) return PS_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    if (!after_relocation(ps, s)) return PS_ERR_CUDA;
    HostBatch hb;
    if (!host_batch_begin(ps, s, &hb)) return PS_ERR_CUDA;
    uint32_t* d_tok = (uint32_t*)hb.buf;
    uint32_t* d_negs = d_tok + tok_count;
    if (cudaMemcpyAsync(d_tok, h_tokens, tok_count * 4, cudaMemcpyHostToDevice, hb.cs) != cudaSuccess) return PS_ERR_CUDA;
    if (n_negs && cudaMemcpyAsync(d_negs, h_negs, n_negs * 4, cudaMemcpyHostToDevice, hb.cs) != cudaSuccess)
        return PS_ERR_CUDA;
    if (!host_batch_copied(ps, s, hb)) return PS_ERR_CUDA;
    SortSet* ss = next_set(ps);
    if (hb.slot >= 0) {
        if (!fork_side(ps, ss, s)) return PS_ERR_CUDA;      // waits for the copy; pipelined or ordered as the handle is set
    } else if (cudaEventRecord(ps->ev_fork, s) != cudaSuccess || cudaStreamWaitEvent(ps->side, ps->ev_fork, 0) != cudaSuccess) {
        return PS_ERR_CUDA;                                  // the batch was just copied on the caller's stream
    }
    launch_keys_sgns(ps, d_tok, tok_first, first_pos, n_centers, corpus_len, window, d_negs, n_neg, out_key_base,
                     ps->side);
    const int which = run_push_sort(ps, (uint32_t)occ, ps->side);
    const uint32_t lb = launch_step_sgns(ps, d_tok, tok_first, first_pos, n_centers, corpus_len, window, d_negs, n_neg,
                                         out_key_base, lr, s);
    if (!join_side(ps, s)) return PS_ERR_CUDA;
    run_push_reduce(ps, (uint32_t)occ, which, ps->upd, d_loss_accum, d_loss_accum ? lb : 0, s,
                    sgns_scales(ps, n_centers), (uint32_t)(occ / n_centers));
    c = release_set(ss, s);
    if (c != PS_OK) return c;
    return finish_host_step(ps, hb, d_loss_accum, h_loss, s);
}

ps_status_t ps_get_location(ps_store_t* ps, const uint64_t* d_keys, uint64_t n, uint32_t* d_owner, uint32_t* d_slot,
                            void* stream) {
    PS_BEGIN_CALL(ps);
    if (n == 0) return PS_OK;
    if (!d_keys || !d_owner || !d_slot) return PS_ERR_INVALID_ARG;
    launch_get_location(ps, d_keys, n, d_owner, d_slot, s);
    return after_launch();
}

ps_status_t ps_export(ps_store_t* ps, float* h_rows_by_key, uint32_t* h_owner, uint32_t* h_slot) {
    if (!ps) return PS_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return PS_ERR_CUDA;
    const uint64_t K = ps->cfg.num_keys;
    const uint32_t L = ps->cfg.row_len;
    if (h_rows_by_key) {
        const uint64_t chunk = ps->max_keys;                // rows that fit in the update-row scratch
        for (uint64_t k0 = 0; k0 < K; k0 += chunk) {
            const uint64_t c = K - k0 < chunk ? K - k0 : chunk;
            launch_gather_rows_by_key(ps, k0, c, ps->upd, 0);
            if (cudaMemcpy(h_rows_by_key + k0 * L, ps->upd, c * L * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
                return PS_ERR_CUDA;
        }
    }
    if (h_owner || h_slot) {
        uint2* tmp = (uint2*)malloc(K * sizeof(uint2));
        if (!tmp) return PS_ERR_INVALID_ARG;
        if (cudaMemcpy(tmp, ps->table, K * sizeof(uint2), cudaMemcpyDeviceToHost) != cudaSuccess) {
            free(tmp);
            return PS_ERR_CUDA;
        }
        for (uint64_t k = 0; k < K; ++k) {
            if (h_owner) h_owner[k] = tmp[k].x;
            if (h_slot) h_slot[k] = tmp[k].y;
        }
        free(tmp);
    }
    return after_launch();
}

ps_status_t ps_export_freelists(ps_store_t* ps, uint32_t* h_stacks, uint64_t* h_tops) {
    if (!ps) return PS_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return PS_ERR_CUDA;
    const uint64_t N = ps->cfg.num_workers, S = ps->cfg.slots_per_part;
    if (h_stacks && cudaMemcpy(h_stacks, ps->stacks, N * S * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
        return PS_ERR_CUDA;
    if (h_tops && cudaMemcpy(h_tops, ps->tops, N * 8, cudaMemcpyDeviceToHost) != cudaSuccess) return PS_ERR_CUDA;
    return PS_OK;
}

ps_status_t ps_sync(ps_store_t* ps, void* stream) {
    if (!ps) return PS_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaStreamSynchronize(s) != cudaSuccess) return PS_ERR_CUDA;
    if (ps->loc_pending) {                          // a relocation on another stream belongs to what this call waits for
        if (cudaEventSynchronize(ps->ev_loc) != cudaSuccess) return PS_ERR_CUDA;
        ps->loc_pending = false;
    }
    unsigned int code = 0;
    if (cudaMemcpy(&code, &ps->status->sticky, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return PS_ERR_CUDA;
    if (code != 0 && cudaMemset(&ps->status->sticky, 0, 4) != cudaSuccess) return PS_ERR_CUDA;
    if (code == PS_ERR_CUDA) {                  // a sort that gave up inside its grid barrier leaves it mid-count
        if (cudaDeviceSynchronize() != cudaSuccess) return PS_ERR_CUDA;
        for (int b = 0; b < kSortSets; ++b)
            if (cudaMemset(ps->sets[b].sort_ctl, 0, kSortCtlWords * sizeof(uint32_t)) != cudaSuccess) return PS_ERR_CUDA;
    }
    return (ps_status_t)code;
}

ps_status_t ps_set_host_overlap(ps_store_t* ps, int on) {
    if (!ps) return PS_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return PS_ERR_CUDA;     // no host batch in flight across the switch
    ps->host_overlap = on != 0;
    for (int b = 0; b < kHostStages; ++b) ps->consumed_valid[b] = false;
    ps->batch_ready = nullptr;
    return PS_OK;
}

ps_status_t ps_set_pipelining(ps_store_t* ps, int on) {
    if (!ps) return PS_ERR_INVALID_ARG;
    ps->pipelined = on != 0;
    return PS_OK;
}

ps_status_t ps_set_push_mode(ps_store_t* ps, int mode) {
    if (!ps || (mode != PS_PUSH_SORTED && mode != PS_PUSH_ATOMIC)) return PS_ERR_INVALID_ARG;
    ps->push_mode = mode;
    return PS_OK;
}

ps_status_t ps_set_mf_path(ps_store_t* ps, int path) {
    if (!ps || path < 0 || path > 3) return PS_ERR_INVALID_ARG;
    ps->mf_path = path;
    return PS_OK;
}

uint64_t ps_launch_count(const ps_store_t* ps) { return ps ? ps->launches : 0; }

ps_status_t ps_rows_moved(ps_store_t* ps, uint64_t* h_out) {
    if (!ps || !h_out) return PS_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return PS_ERR_CUDA;
    unsigned long long v = 0;
    if (cudaMemcpy(&v, &ps->status->rows_moved, 8, cudaMemcpyDeviceToHost) != cudaSuccess) return PS_ERR_CUDA;
    *h_out = v;
    return PS_OK;
}

ps_status_t ps_profile_start(ps_store_t* ps, uint32_t max_launches) {
    if (!ps || ps->prof || max_launches == 0) return PS_ERR_INVALID_ARG;
    Profile* p = new (std::nothrow) Profile();
    if (!p) return PS_ERR_INVALID_ARG;
    p->cap = max_launches;
    p->open = false;
    p->recs.reserve(max_launches);
    ps->prof = p;
    return PS_OK;
}

ps_status_t ps_profile_stop(ps_store_t* ps, char* h_report, size_t capacity) {
    if (!ps || !ps->prof) return PS_ERR_INVALID_ARG;
    Profile* p = ps->prof;
    ps->prof = nullptr;
    const ps_status_t rc = cudaDeviceSynchronize() == cudaSuccess ? PS_OK : PS_ERR_CUDA;
    std::map<std::string, std::pair<uint64_t, double>> agg;
    std::vector<std::string> order;
    for (const ProfRec& r : p->recs) {
        float ms = 0.f;
        if (rc == PS_OK && cudaEventElapsedTime(&ms, r.a, r.b) == cudaSuccess) {
            if (!agg.count(r.name)) order.push_back(r.name);
            agg[r.name].first += 1;
            agg[r.name].second += (double)ms * 1000.0;
        }
        cudaEventDestroy(r.a);
        cudaEventDestroy(r.b);
    }
    delete p;
    if (h_report && capacity) {
        size_t used = 0;
        h_report[0] = 0;
        for (const std::string& name : order) {
            char line[256];
            const int len = snprintf(line, sizeof line, "%s %llu %.3f\n", name.c_str(),
                                     (unsigned long long)agg[name].first, agg[name].second);
            if (len < 0 || used + (size_t)len + 1 > capacity) break;
            memcpy(h_report + used, line, (size_t)len + 1);
            used += (size_t)len;
        }
    }
    return rc;
}

const char* ps_status_string(ps_status_t status) {
    switch (status) {
        case PS_OK: return "ok";
        case PS_ERR_INVALID_ARG: return "invalid argument";
        case PS_ERR_KEY_RANGE: return "key out of range";
        case PS_ERR_WORKER_RANGE: return "worker out of range";
        case PS_ERR_CAPACITY: return "partition full";
        case PS_ERR_WORKSPACE: return "workspace too small for this call";
        case PS_ERR_CUDA: return "CUDA runtime error";
        case PS_ERR_UNSUPPORTED: return "unsupported configuration";
        default: return "unknown status";
    }
}

}  // extern "C"
