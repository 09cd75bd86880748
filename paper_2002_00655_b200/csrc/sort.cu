// Stable least-significant-digit radix sort of (key, value) pairs, 8 bits per
// pass, as ONE kernel launch.  It orders the key occurrences of a batch so that
// the push can reduce them segment by segment (cumulative push, Section 2.1 of
// the paper) and so that localize sees each distinct key once, in ascending
// order.
//
// The batches are small (10^5 .. 10^6 keys), so the sort is bound by launch and
// memory latency, not by bandwidth.  All passes therefore run inside one
// cooperative kernel of at most one block per SM; a block owns a contiguous
// chunk of positions in every pass.  Per pass a block needs, for each digit,
// the number of keys with that digit in all chunks before its own.  Those
// counts are gathered while the PREVIOUS pass scatters: a key that goes to
// position pos adds one to counter [next pass][chunk of pos][next digit].  So
// a pass is: grid barrier, read one column of counters per digit, rank the
// chunk's keys tile by tile (warp match + per-warp counters: stable), scatter.
// The key source of the first pass and the sink of the last pass are functors:
// a step extracts its keys from the batch arrays inside the sort, and the
// matrix-factorization step has the last pass emit, per sorted position, the
// addresses the gradient kernel needs instead of bare (key, index) pairs.
//
// The only waiting is the grid barrier; it is bounded, and a block that gives
// up latches an error and returns.
#include "ps_internal.cuh"

namespace psb {

struct SortParams {
    uint32_t *kA, *vA, *kB, *vB;        // pass p reads (kA, vA) if (start + p) is even, else (kB, vB)
    int start;
    uint32_t n_host;
    const unsigned int* n_dev;
    int n_passes;
    uint32_t tiles_per_block;
    uint32_t* counts;                   // [pass][block][digit]
    unsigned int* bar;
    unsigned int* zero_a;               // words cleared before the first barrier (counters of later kernels)
    uint32_t n_zero_a;
    unsigned int* zero_b;
    DevStatus* st;
    unsigned int epoch;
};

// ---- key sources: key of occurrence idx.  kFromBuffer: the keys are already in the pass-0 input buffer. ----
struct SrcBuffer {
    static constexpr bool kFromBuffer = true;
    __device__ __forceinline__ uint32_t operator()(uint32_t, const SortParams&) const { return 0u; }
};
// 64-bit caller keys, range-checked (push, localize)
struct SrcKeys64 {
    static constexpr bool kFromBuffer = false;
    const uint64_t* keys;
    uint64_t K;
    __device__ __forceinline__ uint32_t operator()(uint32_t idx, const SortParams& P) const {
        const uint64_t k = keys[idx];
        if (k >= K) {
            latch_error(P.st, P.epoch, PS_ERR_KEY_RANGE);
            return (uint32_t)K;
        }
        return (uint32_t)k;
    }
};
// occurrences of a batch of matrix cells: 2t = row factor of cell t, 2t + 1 = its column factor
struct SrcMF {
    static constexpr bool kFromBuffer = false;
    const uint32_t *ci, *cj;
    uint64_t col_base, K;
    __device__ __forceinline__ uint32_t operator()(uint32_t idx, const SortParams& P) const {
        const uint32_t t = idx >> 1;
        const uint64_t kw = ci[t], kh = col_base + cj[t];
        if (kw >= col_base || kh >= K) {
            latch_error(P.st, P.epoch, PS_ERR_KEY_RANGE);
            return (uint32_t)K;
        }
        return (idx & 1u) ? (uint32_t)kh : (uint32_t)kw;
    }
};

// ---- sinks of the last pass ----
struct SinkPairs {
    static constexpr bool kPairs = true;
};
// Matrix factorization: besides the sorted key, one record per sorted position with everything the gradient
// kernel would otherwise have to chase through three dependent loads: {key, value of the cell, physical
// row of the key, physical row of the cell's other factor}.  (It says {cell, ...}: the key is in the sorted key array.)
struct SinkMF {
    static constexpr bool kPairs = false;
    const uint32_t *ci, *cj;
    const float* cv;
    uint32_t col_base, K;
    const uint2* table;
    uint64_t S;
    uint4* rec;
    uint32_t* cellpos;                  // sorted position of each cell's row-factor occurrence
};

// Exclusive scan of one value per digit held by threads 0..255 of a block of kThreads; every thread calls.
template <int kThreads>
__device__ __forceinline__ uint32_t scan_digits(uint32_t v, uint32_t* sm8, uint32_t* total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    uint32_t incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31 && w < 8) sm8[w] = incl;
    __syncthreads();
    uint32_t wbase = 0, tot = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t t = sm8[i];
        if (i < w) wbase += t;
        tot += t;
    }
    __syncthreads();
    *total = tot;
    return wbase + incl - v;
}

// A tile is kThreads x kItems keys.  Small sorts use many threads with few keys each (every phase of a pass is a
// short chain of dependent steps, and all SMs get a tile); large sorts use 256 threads with 8 keys each.
template <class Src, class Sink, int kThreads, int kItems>
__global__ void __launch_bounds__(kThreads, kThreads == 256 ? 3 : 2)
sort_all_kernel(Src src, Sink sink, SortParams P) {
    constexpr int kTile = kThreads * kItems;
    constexpr int kWarps = kThreads / 32;
    constexpr int kQ = kThreads / 64;                // threads per group of four digits in the counter read
    constexpr int kRowsAtOnce = kThreads >= 512 ? 16 : 8;
    __shared__ uint32_t digit_base[kRadix];          // global position of the tile's first key with each digit
    __shared__ uint32_t local_base[kRadix];          // the same inside the tile
    __shared__ uint32_t warp_hist[kWarps][kRadix];
    extern __shared__ uint32_t s_dyn[];               // the tile in digit order, on its way out: keys, then values
    uint32_t* const s_key = s_dyn;
    uint32_t* const s_val = s_dyn + kTile;
    __shared__ uint32_t sm[8];
    __shared__ int s_ok;
    const uint32_t n = P.n_dev ? tmin<uint32_t>(*((const volatile unsigned int*)P.n_dev), P.n_host) : P.n_host;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const bool digit_thread = tid < kRadix;
    const int dg = tid & (kRadix - 1);
    const uint32_t b = blockIdx.x, G = gridDim.x;
    const uint32_t chunk = P.tiles_per_block * kTile;
    const uint64_t c0_64 = (uint64_t)b * chunk;
    const uint32_t c0 = c0_64 < n ? (uint32_t)c0_64 : n;
    const uint32_t c1 = (uint64_t)c0 + chunk < n ? c0 + chunk : n;
    const uint32_t my_tiles = (c1 - c0 + kTile - 1) / kTile;
    const unsigned lt = (1u << lane) - 1u;
    unsigned int barriers = 0;

    // ---- before the first barrier: clear what must start at zero, count the digits of pass 0 ----
    if (digit_thread) {
        for (int p = 1; p < P.n_passes; ++p) P.counts[((size_t)p * G + b) * kRadix + tid] = 0u;
        digit_base[tid] = 0u;
    }
    if (b == 0) {
        for (uint32_t i = tid; i < P.n_zero_a; i += kThreads) P.zero_a[i] = 0u;
        if (tid == 0 && P.zero_b) P.zero_b[0] = P.zero_b[1] = 0u;     // (the list counter of the coming reduction and its neighbour)
    }
    __syncthreads();
    uint32_t key0[kItems];                           // keys of the chunk's first tile stay in registers for pass 0
#pragma unroll
    for (int it = 0; it < kItems; ++it) key0[it] = 0u;
    uint32_t* kin0 = (P.start & 1) ? P.kB : P.kA;
    for (uint32_t t = 0; t < my_tiles; ++t) {
        const uint32_t tb = c0 + t * kTile + w * (32 * kItems);
        uint32_t kk[kItems];
#pragma unroll
        for (int it = 0; it < kItems; ++it) {
            const uint32_t idx = tb + it * 32 + lane;
            kk[it] = 0u;
            if (idx < c1) kk[it] = Src::kFromBuffer ? __ldcg(kin0 + idx) : src(idx, P);
        }
#pragma unroll
        for (int it = 0; it < kItems; ++it) {
            const uint32_t idx = tb + it * 32 + lane;
            if (idx < c1) {
                if (!Src::kFromBuffer && t > 0) kin0[idx] = kk[it];
                atomicAdd(&digit_base[kk[it] & (kRadix - 1)], 1u);
            }
            if (t == 0) key0[it] = kk[it];
        }
    }
    __syncthreads();
    if (digit_thread) P.counts[(size_t)b * kRadix + tid] = digit_base[tid];
    if (!grid_barrier(P.bar, ++barriers * G, &s_ok)) {
        if (tid == 0) atomicCAS(&P.st->sticky, 0u, (unsigned int)PS_ERR_CUDA);
        return;
    }

    for (int p = 0; p < P.n_passes; ++p) {
        const bool from_a = ((P.start + p) & 1) == 0;
        uint32_t* kin = from_a ? P.kA : P.kB;
        uint32_t* vin = from_a ? P.vA : P.vB;
        uint32_t* kout = from_a ? P.kB : P.kA;
        uint32_t* vout = from_a ? P.vB : P.vA;
        const int shift = p * kRadixBits;
        const bool last = p + 1 == P.n_passes;
        uint32_t key[kItems], val[kItems];
        // the keys of the chunk's first tile are asked for now, so that they travel beside the counters below
        auto load_tile = [&](uint32_t t) {
            const uint32_t tb = c0 + t * kTile + w * (32 * kItems);
#pragma unroll
            for (int it = 0; it < kItems; ++it) {
                const uint32_t idx = tb + it * 32 + lane;
                key[it] = 0u;
                val[it] = idx;
                if (idx < c1) {
                    if (p == 0) {
                        key[it] = (t == 0) ? key0[it] : __ldcg(kin + idx);
                    } else {
                        key[it] = __ldcg(kin + idx);
                        val[it] = __ldcg(vin + idx);
                    }
                }
            }
        };
        if (my_tiles > 0) load_tile(0);
        // ---- per digit: keys with that digit in the chunks before this block's, and in all chunks.  Thread
        // (q, d4) adds up four digits over every kQ-th block; the kQ partial sums meet in shared memory.
        {
            const int q = tid >> 6, d4 = tid & 63;
            const uint4* col = reinterpret_cast<const uint4*>(P.counts + (size_t)p * G * kRadix) + d4;
            uint4 before = make_uint4(0u, 0u, 0u, 0u), total = before;
            for (uint32_t r0 = q; r0 < G; r0 += kRowsAtOnce * kQ) {
                uint4 c[kRowsAtOnce];
#pragma unroll
                for (int k = 0; k < kRowsAtOnce; ++k)
                    c[k] = r0 + kQ * k < G ? __ldcg(col + (size_t)(r0 + kQ * k) * (kRadix / 4)) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int k = 0; k < kRowsAtOnce; ++k) {
                    total.x += c[k].x; total.y += c[k].y; total.z += c[k].z; total.w += c[k].w;
                    if (r0 + kQ * k < b) { before.x += c[k].x; before.y += c[k].y; before.z += c[k].z; before.w += c[k].w; }
                }
            }
            uint32_t* part = &warp_hist[0][0];        // [2][kQ][256], free between tiles
            reinterpret_cast<uint4*>(part + q * kRadix)[d4] = before;
            reinterpret_cast<uint4*>(part + (kQ + q) * kRadix)[d4] = total;
            __syncthreads();
            uint32_t bf = 0, tt = 0;
            if (digit_thread) {
#pragma unroll
                for (int i = 0; i < kQ; ++i) {
                    bf += part[i * kRadix + tid];
                    tt += part[(kQ + i) * kRadix + tid];
                }
            }
            uint32_t tot;
            const uint32_t gbase = scan_digits<kThreads>(tt, sm, &tot);            // has barriers
            if (digit_thread) digit_base[tid] = gbase + bf;
        }
        for (uint32_t t = 0; t < my_tiles; ++t) {
            if (t > 0) load_tile(t);
#pragma unroll
            for (int i = tid; i < kWarps * kRadix; i += kThreads) (&warp_hist[0][0])[i] = 0u;
            __syncthreads();
            const uint32_t t0 = c0 + t * kTile;
            const uint32_t tb = t0 + w * (32 * kItems);
            const uint32_t in_tile = tmin<uint32_t>((uint32_t)kTile, c1 - t0);
            uint32_t rank[kItems];
            unsigned peers[kItems];
            // lanes of the warp that hold the same digit (lanes past the end get a pseudo-digit of their own)
#pragma unroll
            for (int it = 0; it < kItems; ++it) {
                const bool valid = tb + it * 32 + lane < c1;
                const uint32_t digit = (key[it] >> shift) & (kRadix - 1);
                peers[it] = __match_any_sync(0xffffffffu, valid ? digit : (kRadix + lane));
            }
#pragma unroll
            for (int it = 0; it < kItems; ++it) {
                const bool valid = tb + it * 32 + lane < c1;
                const uint32_t digit = (key[it] >> shift) & (kRadix - 1);
                const int leader = __ffs(peers[it]) - 1;
                uint32_t old = 0;
                if (valid && lane == leader) {
                    old = warp_hist[w][digit];
                    warp_hist[w][digit] = old + __popc(peers[it]);
                }
                old = __shfl_sync(0xffffffffu, old, leader);
                rank[it] = old + __popc(peers[it] & lt);
                __syncwarp();
            }
            __syncthreads();
            // thread d: this tile's count of digit d; the per-warp counters become offsets inside the digit
            uint32_t run = 0;
            if (digit_thread) {
#pragma unroll
                for (int i = 0; i < kWarps; ++i) {
                    const uint32_t c = warp_hist[i][tid];
                    warp_hist[i][tid] = run;
                    run += c;
                }
            }
            uint32_t tile_tot;
            const uint32_t lb = scan_digits<kThreads>(run, sm, &tile_tot);         // has barriers
            if (digit_thread) local_base[tid] = lb;
            __syncthreads();
            // the tile in digit order in shared memory, so that the stores below walk runs of equal digits
#pragma unroll
            for (int it = 0; it < kItems; ++it) {
                if (tb + it * 32 + lane < c1) {
                    const uint32_t digit = (key[it] >> shift) & (kRadix - 1);
                    const uint32_t lp = local_base[digit] + warp_hist[w][digit] + rank[it];
                    s_key[lp] = key[it];
                    s_val[lp] = val[it];
                }
            }
            __syncthreads();
            uint32_t pos[kItems];
#pragma unroll
            for (int it = 0; it < kItems; ++it) {
                const uint32_t j = it * kThreads + tid;
                key[it] = j < in_tile ? s_key[j] : 0u;
                val[it] = j < in_tile ? s_val[j] : 0u;
                const uint32_t digit = (key[it] >> shift) & (kRadix - 1);
                pos[it] = digit_base[digit] + (j - local_base[digit]);
            }
            if (!last) {
#pragma unroll
                for (int it = 0; it < kItems; ++it) {
                    const bool valid = it * kThreads + tid < in_tile;
                    if (valid) {
                        kout[pos[it]] = key[it];
                        vout[pos[it]] = val[it];
                    }
                    // one more key with this digit of the next pass in the chunk the key lands in; lanes that
                    // agree on both send one addition
                    const uint32_t nd = (key[it] >> (shift + kRadixBits)) & (kRadix - 1);
                    const uint32_t cell = valid ? (pos[it] / chunk) * kRadix + nd : 0xFFFFFFFFu - lane;
                    const unsigned same = __match_any_sync(0xffffffffu, cell);
                    if (valid && lane == __ffs(same) - 1)
                        atomicAdd(P.counts + (size_t)(p + 1) * G * kRadix + cell, (uint32_t)__popc(same));
                }
            } else if constexpr (Sink::kPairs) {
#pragma unroll
                for (int it = 0; it < kItems; ++it) {
                    if (it * kThreads + tid < in_tile) {
                        kout[pos[it]] = key[it];
                        vout[pos[it]] = val[it];
                    }
                }
            } else {
                // four items at a time: all their index loads, then all table loads, then the records
                constexpr int kAtOnce = kItems < 4 ? kItems : 4;
#pragma unroll
                for (int i0 = 0; i0 < kItems; i0 += kAtOnce) {
                    uint32_t pk[kAtOnce];
                    float cval[kAtOnce];
                    uint2 e_own[kAtOnce], e_par[kAtOnce];
#pragma unroll
                    for (int i = 0; i < kAtOnce; ++i) {
                        const int it = i0 + i;
                        const bool live = it * kThreads + tid < in_tile && key[it] < sink.K;
                        const uint32_t cell = val[it] >> 1;
                        pk[i] = sink.K;
                        cval[i] = 0.f;
                        if (live) {
                            pk[i] = (val[it] & 1u) ? sink.ci[cell] : sink.col_base + sink.cj[cell];
                            cval[i] = sink.cv[cell];
                        }
                    }
#pragma unroll
                    for (int i = 0; i < kAtOnce; ++i) {
                        const bool live = pk[i] < sink.K;       // cells with an index out of range carry the mark K
                        e_own[i] = live ? sink.table[key[i0 + i]] : make_uint2(0u, 0u);
                        e_par[i] = live ? sink.table[pk[i]] : make_uint2(0u, 0u);
                    }
#pragma unroll
                    for (int i = 0; i < kAtOnce; ++i) {
                        const int it = i0 + i;
                        if (it * kThreads + tid < in_tile) {
                            kout[pos[it]] = key[it];
                            if (!(val[it] & 1u)) sink.cellpos[val[it] >> 1] = pos[it];
                            sink.rec[pos[it]] = make_uint4(val[it] >> 1, __float_as_uint(cval[i]),
                                                           (uint32_t)phys_row(e_own[i], sink.S),
                                                           (uint32_t)phys_row(e_par[i], sink.S));
                        }
                    }
                }
            }
            __syncthreads();
            if (digit_thread) digit_base[tid] += run;           // the chunk's next tile starts after this one
        }
        if (!last && !grid_barrier(P.bar, ++barriers * G, &s_ok)) {
            if (tid == 0) atomicCAS(&P.st->sticky, 0u, (unsigned int)PS_ERR_CUDA);
            return;
        }
    }
    grid_leave(P.bar, G);
}

// Small sorts: few blocks of many threads.  The sort of the next step runs beside the current step's kernels;
// its blocks spend most of their life waiting at grid barriers, so it should hold few SMs' registers while it
// does, and the cost of a pass grows with the number of blocks (barrier, counter read) more than with the keys
// per block.
constexpr int kSmallThreads = 512, kSmallItems = 4;      // tiles of 2048 keys
constexpr int kSmallTile = kSmallThreads * kSmallItems;
static_assert(kSmallTile >= kSortTile / 2, "the digit counters are sized for tiles of at least kSortTile / 2 keys");

template <class Src, class Sink>
static int sort_launch(ps_store* ps, const Src& src, const Sink& sink, uint32_t n, const unsigned int* n_dev, int bits,
                       cudaStream_t stream, int start, unsigned int* zero_me, uint32_t zero_groups) {
    if (bits < 1) bits = 1;
    SortParams P;
    P.kA = ps->keysA; P.vA = ps->valsA; P.kB = ps->keysB; P.vB = ps->valsB;
    P.start = start;
    P.n_host = n;
    P.n_dev = n_dev;
    P.n_passes = (bits + kRadixBits - 1) / kRadixBits;
    const uint32_t max_grid = (uint32_t)tmax(ps->sm_count, 1);
    // short tiles while they still give every block at most one (and the counters have room for that many blocks)
    const bool small = n <= max_grid * (uint32_t)kSmallTile && div_up_u32(n, kSmallTile) <= ps->sort_blocks_cap;
    const uint32_t tile = small ? kSmallTile : kSortTile;
    const uint32_t n_tiles = div_up_u32(n, tile);
    P.tiles_per_block = div_up_u32(n_tiles, max_grid);
    const uint32_t grid = div_up_u32(n_tiles, P.tiles_per_block);
    P.counts = ps->tile_state;
    P.bar = ps->sort_ctl;
    P.zero_a = ps->group_done;
    P.n_zero_a = zero_groups;
    P.zero_b = zero_me;
    P.st = ps->status;
    P.epoch = ps->epoch;
    if (ps->prof) prof_before(ps, "sort_all_kernel", stream);
    void* args[] = {(void*)&src, (void*)&sink, (void*)&P};
    // cooperative: the blocks wait for one another at the grid barrier, so all of them must be resident
    if (small) {
        static std::atomic<unsigned long long> attr_set{0};
        const void* fn = (const void*)sort_all_kernel<Src, Sink, kSmallThreads, kSmallItems>;
        const size_t smem = (size_t)2 * kSmallTile * sizeof(uint32_t);
        opt_in_smem(fn, smem, &attr_set);
        cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kSmallThreads), args, smem, stream);
    } else {
        static std::atomic<unsigned long long> attr_set{0};
        const void* fn = (const void*)sort_all_kernel<Src, Sink, kSortThreads, kSortItems>;
        const size_t smem = (size_t)2 * kSortTile * sizeof(uint32_t);
        opt_in_smem(fn, smem, &attr_set);
        cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kSortThreads), args, smem, stream);
    }
    if (ps->prof) prof_after(ps, stream);
    ps->launches++;
    return (start + P.n_passes) & 1;
}

int radix_sort_pairs(ps_store* ps, uint32_t n, const unsigned int* n_dev, int bits, cudaStream_t stream, int start,
                     unsigned int* zero_me, uint32_t zero_groups) {
    if (n == 0) return start;
    return sort_launch(ps, SrcBuffer{}, SinkPairs{}, n, n_dev, bits, stream, start, zero_me, zero_groups);
}

int radix_sort_keys64(ps_store* ps, const uint64_t* d_keys, uint32_t n, cudaStream_t stream, unsigned int* zero_me,
                      uint32_t zero_groups) {
    if (n == 0) return 0;
    SrcKeys64 src{d_keys, ps->cfg.num_keys};
    return sort_launch(ps, src, SinkPairs{}, n, nullptr, ps->key_bits, stream, 0, zero_me, zero_groups);
}

int radix_sort_mf(ps_store* ps, const uint32_t* d_i, const uint32_t* d_j, const float* d_v, uint32_t n_cells,
                  uint64_t col_key_base, bool records, cudaStream_t stream, unsigned int* zero_me,
                  uint32_t zero_groups) {
    if (n_cells == 0) return 0;
    SrcMF src{d_i, d_j, col_key_base, ps->cfg.num_keys};
    if (!records)
        return sort_launch(ps, src, SinkPairs{}, 2 * n_cells, nullptr, ps->key_bits, stream, 0, zero_me, zero_groups);
    SinkMF sink{d_i, d_j, d_v, (uint32_t)col_key_base, (uint32_t)ps->cfg.num_keys, ps->table,
                ps->cfg.slots_per_part, ps->rec, ps->cellpos};
    return sort_launch(ps, src, sink, 2 * n_cells, nullptr, ps->key_bits, stream, 0, zero_me, zero_groups);
}

}  // namespace psb
