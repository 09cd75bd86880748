// Stable least-significant-digit radix sort of (key, value) pairs, 8 bits per
// pass.  It orders the key occurrences of a batch so that the push can reduce
// them segment by segment (cumulative push, Section 2.1 of the paper) and so
// that localize sees each distinct key once, in ascending order.
//
// One kernel builds the digit histograms of every pass at once (they do not
// depend on the order of the keys).  Each pass is then a single kernel: a block
// takes the next tile (an atomic ticket, so every earlier tile is already
// running or done), ranks its keys stably inside the tile (warp match +
// per-warp counters), publishes its per-digit counts, obtains the counts of all
// earlier tiles by looking back over their published words (count-only or
// running-total, one 32-bit word per tile and digit), and scatters.
// The only waiting is the look-back; it is bounded, and a block that gives up
// latches an error and writes nothing.
#include "ps_internal.cuh"

namespace psb {

constexpr uint32_t kFlagCount = 1u << 30;    // the word holds this tile's count
constexpr uint32_t kFlagTotal = 2u << 30;    // the word holds the total up to and including this tile
constexpr uint32_t kValueMask = (1u << 30) - 1u;
constexpr int kLookbackSpins = 1 << 22;
constexpr int kLookbackWindow = 16;

// ctl layout: [kMaxPasses][kRadix] histograms, then kMaxPasses tickets.
__global__ void __launch_bounds__(kSortThreads)
sort_hist_kernel(const uint32_t* __restrict__ keys, uint32_t n_host, const unsigned int* __restrict__ n_dev,
                 int n_passes, uint32_t* __restrict__ ctl, uint32_t* __restrict__ tile_state, uint32_t n_tiles,
                 unsigned int* __restrict__ zero_me) {
    __shared__ uint32_t h[kMaxSortPasses][kRadix];
    if (zero_me && blockIdx.x == 0 && threadIdx.x == 0) *zero_me = 0u;      // a counter a later kernel of the call uses
    const uint32_t n = n_dev ? tmin<uint32_t>(*n_dev, n_host) : n_host;
    for (int p = 0; p < n_passes; ++p) {
        h[p][threadIdx.x] = 0;
        tile_state[((size_t)p * n_tiles + blockIdx.x) * kRadix + threadIdx.x] = 0u;
    }
    __syncthreads();
    const uint32_t base = blockIdx.x * kSortTile;
#pragma unroll
    for (int it = 0; it < kSortItems; ++it) {
        const uint32_t idx = base + it * kSortThreads + threadIdx.x;
        if (idx < n) {
            const uint32_t key = keys[idx];
            for (int p = 0; p < n_passes; ++p) atomicAdd(&h[p][(key >> (p * kRadixBits)) & (kRadix - 1)], 1u);
        }
    }
    __syncthreads();
    for (int p = 0; p < n_passes; ++p) {
        const uint32_t c = h[p][threadIdx.x];
        if (c) atomicAdd(&ctl[p * kRadix + threadIdx.x], c);
    }
}

template <bool kIota>
__global__ void __launch_bounds__(kSortThreads)
sort_pass_kernel(const uint32_t* __restrict__ kin, const uint32_t* __restrict__ vin, uint32_t* __restrict__ kout,
                 uint32_t* __restrict__ vout, uint32_t n_host, const unsigned int* __restrict__ n_dev, int pass,
                 uint32_t* __restrict__ ctl, uint32_t* __restrict__ tile_state, uint32_t n_tiles, DevStatus* st) {
    __shared__ uint32_t digit_base[kRadix];
    __shared__ uint32_t warp_hist[kSortThreads / 32][kRadix];
    __shared__ uint32_t sm[8];
    __shared__ uint32_t s_tile;
    __shared__ int s_gave_up;
    const uint32_t n = n_dev ? tmin<uint32_t>(*n_dev, n_host) : n_host;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int shift = pass * kRadixBits;
    if (tid == 0) {
        s_tile = atomicAdd(&ctl[kMaxSortPasses * kRadix + pass], 1u);
        s_gave_up = 0;
    }
    uint32_t tot;
    const uint32_t global_base = block_exclusive_scan_256(ctl[pass * kRadix + tid], sm, &tot);   // has a barrier
#pragma unroll
    for (int i = 0; i < kSortThreads / 32; ++i) warp_hist[i][tid] = 0;
    __syncthreads();
    const uint32_t tile = s_tile;
    if (tile >= n_tiles) return;
    const uint32_t chunk = tile * kSortTile + w * (32 * kSortItems);
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
        // thread d: this tile's count of digit d; the per-warp counters become offsets inside the tile
        uint32_t run = 0;
#pragma unroll
        for (int i = 0; i < kSortThreads / 32; ++i) {
            const uint32_t t = warp_hist[i][tid];
            warp_hist[i][tid] = run;
            run += t;
        }
        const volatile uint32_t* tile_state_v = tile_state;
        volatile uint32_t* mine = tile_state + ((size_t)pass * n_tiles + tile) * kRadix + tid;
        uint32_t before = 0;
        if (tile == 0) {
            *mine = kFlagTotal | run;
        } else {
            *mine = kFlagCount | run;
            // Look back over earlier tiles until one of them shows a running total.  The words of
            // kLookbackWindow tiles are requested together; one that is not published yet is polled.
            bool done = false;
            for (uint32_t t = tile; t > 0 && !done; t = t > kLookbackWindow ? t - kLookbackWindow : 0) {
                uint32_t word[kLookbackWindow];
#pragma unroll
                for (int k = 0; k < kLookbackWindow; ++k) {
                    word[k] = 0u;
                    if (t > (uint32_t)k) word[k] = *(tile_state_v + ((size_t)pass * n_tiles + (t - 1 - k)) * kRadix + tid);
                }
#pragma unroll
                for (int k = 0; k < kLookbackWindow; ++k) {
                    if (done || t <= (uint32_t)k) continue;
                    uint32_t wv = word[k];
                    int spins = 0;
                    while ((wv & ~kValueMask) == 0u && spins < kLookbackSpins) {
                        __nanosleep(32);
                        wv = *(tile_state_v + ((size_t)pass * n_tiles + (t - 1 - k)) * kRadix + tid);
                        ++spins;
                    }
                    if ((wv & ~kValueMask) == 0u) {
                        s_gave_up = 1;
                        done = true;
                    } else {
                        before += wv & kValueMask;
                        if (wv & kFlagTotal) done = true;
                    }
                }
            }
            *mine = kFlagTotal | (before + run);
        }
        digit_base[tid] = global_base + before;
    }
    __syncthreads();
    if (s_gave_up) {                                    // nothing is written; the call's results are void
        if (tid == 0) atomicCAS(&st->sticky, 0u, (unsigned int)PS_ERR_CUDA);
        return;
    }
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
                     cudaStream_t stream, int start, unsigned int* zero_me, uint32_t zero_groups) {
    if (n == 0) return start;
    const uint32_t n_tiles = div_up_u32(n, kSortTile);
    uint32_t *kin = ps->keysA, *vin = ps->valsA, *kout = ps->keysB, *vout = ps->valsB;
    if (start) {
        kin = ps->keysB; vin = ps->valsB; kout = ps->keysA; vout = ps->valsA;
    }
    int which = start;
    if (bits < 1) bits = 1;
    const int n_passes = (bits + kRadixBits - 1) / kRadixBits;
    cudaMemsetAsync(ps->sort_ctl, 0, (kSortCtlWords + (size_t)zero_groups) * sizeof(uint32_t), stream);
    PS_LAUNCH(ps, sort_hist_kernel, n_tiles, kSortThreads, stream, kin, n, n_dev, n_passes, ps->sort_ctl,
              ps->tile_state, n_tiles, zero_me);
    for (int pass = 0; pass < n_passes; ++pass) {
        if (iota_vals && pass == 0)
            PS_LAUNCH(ps, sort_pass_kernel<true>, n_tiles, kSortThreads, stream, kin, vin, kout, vout, n, n_dev, pass,
                      ps->sort_ctl, ps->tile_state, n_tiles, ps->status);
        else
            PS_LAUNCH(ps, sort_pass_kernel<false>, n_tiles, kSortThreads, stream, kin, vin, kout, vout, n, n_dev, pass,
                      ps->sort_ctl, ps->tile_state, n_tiles, ps->status);
        uint32_t* t;
        t = kin; kin = kout; kout = t;
        t = vin; vin = vout; vout = t;
        which ^= 1;
    }
    return which;
}

}  // namespace psb
