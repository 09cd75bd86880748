// Stable least-significant-digit radix sort of (key, value) pairs, 8 bits per
// pass.  It orders the key occurrences of a batch so that the push can reduce
// them segment by segment (cumulative push, Section 2.1 of the paper) and so
// that localize sees each distinct key once, in ascending order.
//
// Per pass: (1) per-tile digit histograms, (2) one block per digit scans that
// digit's counts across tiles, (3) each tile ranks its keys stably (warp
// match + per-warp counters) and scatters.  No inter-block waiting anywhere.
#include "ps_internal.cuh"

namespace psb {

__global__ void __launch_bounds__(kSortThreads)
sort_hist_kernel(const uint32_t* __restrict__ keys, uint32_t n_host, const unsigned int* __restrict__ n_dev,
                 int shift, uint32_t* __restrict__ counts, uint32_t n_tiles, unsigned int* __restrict__ zero_me) {
    __shared__ uint32_t h[kRadix];
    if (zero_me && blockIdx.x == 0 && threadIdx.x == 0) *zero_me = 0u;      // a counter a later kernel of the call uses
    const uint32_t n = n_dev ? tmin<uint32_t>(*n_dev, n_host) : n_host;
    h[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t base = blockIdx.x * kSortTile;
#pragma unroll
    for (int it = 0; it < kSortItems; ++it) {
        uint32_t idx = base + it * kSortThreads + threadIdx.x;
        if (idx < n) atomicAdd(&h[(keys[idx] >> shift) & (kRadix - 1)], 1u);
    }
    __syncthreads();
    counts[threadIdx.x * n_tiles + blockIdx.x] = h[threadIdx.x];
}

// Block d turns counts[d][0..n_tiles) into its exclusive prefix and writes the digit total.
__global__ void __launch_bounds__(256)
sort_scan_kernel(uint32_t* __restrict__ counts, uint32_t n_tiles, uint32_t* __restrict__ totals) {
    __shared__ uint32_t sm[8];
    uint32_t* row = counts + (size_t)blockIdx.x * n_tiles;
    uint32_t running = 0;
    for (uint32_t c0 = 0; c0 < n_tiles; c0 += 256) {
        uint32_t i = c0 + threadIdx.x;
        uint32_t v = i < n_tiles ? row[i] : 0;
        uint32_t tot;
        uint32_t ex = block_exclusive_scan_256(v, sm, &tot);
        if (i < n_tiles) row[i] = running + ex;
        running += tot;
    }
    if (threadIdx.x == 0) totals[blockIdx.x] = running;
}

template <bool kIota>
__global__ void __launch_bounds__(kSortThreads)
sort_scatter_kernel(const uint32_t* __restrict__ kin, const uint32_t* __restrict__ vin,
                    uint32_t* __restrict__ kout, uint32_t* __restrict__ vout, uint32_t n_host,
                    const unsigned int* __restrict__ n_dev, int shift, const uint32_t* __restrict__ counts,
                    uint32_t n_tiles, const uint32_t* __restrict__ totals) {
    __shared__ uint32_t digit_base[kRadix];
    __shared__ uint32_t warp_hist[kSortThreads / 32][kRadix];
    __shared__ uint32_t sm[8];
    const uint32_t n = n_dev ? tmin<uint32_t>(*n_dev, n_host) : n_host;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    {
        uint32_t tot;
        uint32_t ex = block_exclusive_scan_256(totals[tid], sm, &tot);
        digit_base[tid] = ex + counts[(size_t)tid * n_tiles + blockIdx.x];
#pragma unroll
        for (int i = 0; i < kSortThreads / 32; ++i) warp_hist[i][tid] = 0;
    }
    __syncthreads();
    const uint32_t chunk = blockIdx.x * kSortTile + w * (32 * kSortItems);
    uint32_t key[kSortItems], rank[kSortItems];
    const unsigned lt = (1u << lane) - 1u;
#pragma unroll
    for (int it = 0; it < kSortItems; ++it) {
        const uint32_t idx = chunk + it * 32 + lane;
        const bool valid = idx < n;
        key[it] = valid ? kin[idx] : 0u;
        const uint32_t digit = (key[it] >> shift) & (kRadix - 1);
        // lanes past the end get a pseudo-digit of their own so that they match nobody
        const unsigned peers = __match_any_sync(0xffffffffu, valid ? digit : (kRadix + lane));
        const int leader = __ffs(peers) - 1;
        uint32_t old = 0;
        if (valid && lane == leader) {
            old = warp_hist[w][digit];
            warp_hist[w][digit] = old + __popc(peers);
        }
        old = __shfl_sync(0xffffffffu, old, leader);
        rank[it] = old + __popc(peers & lt);
        __syncwarp();
    }
    __syncthreads();
    {
        uint32_t run = 0;
#pragma unroll
        for (int i = 0; i < kSortThreads / 32; ++i) {
            uint32_t t = warp_hist[i][tid];
            warp_hist[i][tid] = run;
            run += t;
        }
    }
    __syncthreads();
#pragma unroll
    for (int it = 0; it < kSortItems; ++it) {
        const uint32_t idx = chunk + it * 32 + lane;
        if (idx < n) {
            const uint32_t digit = (key[it] >> shift) & (kRadix - 1);
            const uint32_t pos = digit_base[digit] + warp_hist[w][digit] + rank[it];
            kout[pos] = key[it];
            vout[pos] = kIota ? idx : vin[idx];
        }
    }
}

int radix_sort_pairs(ps_store* ps, uint32_t n, const unsigned int* n_dev, int bits, bool iota_vals,
                     cudaStream_t stream, int start, unsigned int* zero_me) {
    if (n == 0) return start;
    const uint32_t n_tiles = div_up_u32(n, kSortTile);
    uint32_t *kin = ps->keysA, *vin = ps->valsA, *kout = ps->keysB, *vout = ps->valsB;
    if (start) {
        kin = ps->keysB; vin = ps->valsB; kout = ps->keysA; vout = ps->valsA;
    }
    int which = start;
    if (bits < 1) bits = 1;
    for (int shift = 0; shift < bits; shift += kRadixBits) {
        PS_LAUNCH(ps, sort_hist_kernel, n_tiles, kSortThreads, stream, kin, n, n_dev, shift, ps->hist, n_tiles,
                  shift == 0 ? zero_me : nullptr);
        PS_LAUNCH(ps, sort_scan_kernel, kRadix, 256, stream, ps->hist, n_tiles, ps->totals);
        if (iota_vals && shift == 0)
            PS_LAUNCH(ps, sort_scatter_kernel<true>, n_tiles, kSortThreads, stream, kin, vin, kout, vout, n, n_dev,
                      shift, ps->hist, n_tiles, ps->totals);
        else
            PS_LAUNCH(ps, sort_scatter_kernel<false>, n_tiles, kSortThreads, stream, kin, vin, kout, vout, n,
                      n_dev, shift, ps->hist, n_tiles, ps->totals);
        uint32_t* t;
        t = kin; kin = kout; kout = t;
        t = vin; vin = vout; vout = t;
        which ^= 1;
    }
    return which;
}

}  // namespace psb
