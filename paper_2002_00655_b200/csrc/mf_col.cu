// One minibatch of matrix factorization as ONE launch over the column side of the sorted occurrences.
//
// The occurrences of a batch (2t: row factor of cell t, 2t + 1: its column factor) arrive sorted by key with a
// record {cell, value, row of the key, row of the other factor} per position (sort.cu).  Row keys sort first, so
// the second half of the positions holds the column-factor occurrences, one per cell, grouped by column.  This
// kernel walks only those: a position has both rows of its cell in hand, so it forms e = v - <w, h>, the cell's
// loss, the cell's term for its column factor (summed per segment in fp64, as for a push) AND the cell's term
// for its row factor.
//
// Row factors.  A row key that occurs once in the batch (nearly all of them when the rows of a batch are drawn
// from many more rows than the batch has cells) has exactly one reader, this position, which writes the new row
// in place.  A row key that occurs m > 1 times has m readers, the column positions of its m cells.  Each leaves
// its term in a scratch row (indexed by the sorted position of the row-factor occurrence it stands for) and
// takes a ticket from a counter of that key; the one that draws the last ticket knows that every reader has
// read, adds the m terms in position order in fp64 and writes the row.  No position of the row side is visited.
//
// Column factors.  Eight lanes handle a tile of eight consecutive positions (a warp: four tiles, every
// instruction serves four positions).  A segment inside one tile is finished there and written in place: its
// readers are the positions of the segment itself.  Parts of segments that cross tile borders go to shared
// memory and are chained per block (256 positions) in position order; a segment inside the block is finished by
// the group that holds its first part.  A segment that crosses block borders leaves one fp64 part per block in
// global memory; the blocks it touches are found by probing the sorted keys at the block borders, each takes a
// ticket from the counter of the block in which the segment starts, and the block that draws the last one adds
// the parts in block order and writes the row.  Every sum's shape is a function of the sorted positions only, so
// results are reproducible bit for bit; there is no second launch, no staging of new rows, and no waiting.
//
// Rows are read with plain 128-bit loads into registers, the partner row of the next walk step while the
// current one is worked on (bulk asynchronous copies of 400-byte rows are served at one per ~27 ns and SM,
// which bounded the earlier form of this step).
#include "ps_internal.cuh"

namespace psb {

struct d4c {
    double x, y, z, w;
};

constexpr int kColBlockPos = 256;                   // column positions per block

// ---- side stream, after the sort: what each column position needs to know about its cell's ROW key ----
// dup[q] = {s, m, r}: the row key of the cell at column position q occurs m times in the batch, its occurrences are
// the sorted positions s .. s + m - 1, and this cell's is s + r.  Also clears the tickets of the coming launch.
__global__ void __launch_bounds__(256)
mf_plan_kernel(const uint32_t* __restrict__ sk, const uint4* __restrict__ rec, const uint32_t* __restrict__ cellpos,
               uint32_t n, uint32_t p0, uint4* __restrict__ dup, uint4* __restrict__ blk,
               unsigned int* __restrict__ dup_ticket, unsigned int* __restrict__ seg_ticket, uint32_t n_blocks,
               const DevStatus* st, unsigned int epoch) {
    const uint32_t q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q < n_blocks + 1) seg_ticket[q] = 0u;
    if (call_failed(st, epoch)) return;             // (a key out of range: the records are not valid)
    // ---- warp wq < n_blocks: which blocks of the coming launch do the segments that cross block wq's borders touch?
    // blk[wq] = {first block of the segment that enters wq, last block of that segment, last block of the segment
    // that leaves wq, flags: 1 = one enters, 2 = one leaves}.  The blocks a long segment covers all BEGIN with its
    // key, so a warp probes 32 block borders at a time.
    const uint32_t wq = q >> 5;
    const int lane = threadIdx.x & 31;
    if (wq < n_blocks) {
        const unsigned full = 0xffffffffu;
        const uint64_t bbase = (uint64_t)p0 + (uint64_t)wq * kColBlockPos;
        const uint64_t bend = tmin<uint64_t>(bbase + kColBlockPos, n) - 1;
        const uint32_t k_in = sk[bbase], k_out = sk[bend];
        const bool enters = wq > 0 && sk[bbase - 1] == k_in;
        const bool leaves = bend + 1 < n && sk[bend + 1] == k_out;
        uint32_t e_bs = wq, e_be = wq, l_be = wq;
        if (enters) {                               // blocks before this one that begin with the key
            uint32_t back = 0;
            for (;;) {
                const int64_t bb = (int64_t)wq - 1 - (int64_t)back - lane;
                const bool hit = bb >= 0 && sk[(uint64_t)p0 + (uint64_t)bb * kColBlockPos] == k_in;
                const unsigned m = __ballot_sync(full, hit);
                const uint32_t c = m == full ? 32u : (uint32_t)(__ffs(~m) - 1);
                back += c;
                if (c < 32u) break;
            }
            const uint32_t fb = wq - back;          // begins with the key; the segment starts there or in the block before
            e_bs = (fb > 0 && sk[(uint64_t)p0 + (uint64_t)fb * kColBlockPos - 1] == k_in) ? fb - 1 : fb;
        }
        auto blocks_after = [&](uint32_t key) {     // blocks after this one that begin with the key
            uint32_t fwd = 0;
            for (;;) {
                const uint64_t bb = (uint64_t)wq + 1 + fwd + lane;
                const bool hit = bb < n_blocks && sk[(uint64_t)p0 + bb * kColBlockPos] == key;
                const unsigned m = __ballot_sync(full, hit);
                const uint32_t c = m == full ? 32u : (uint32_t)(__ffs(~m) - 1);
                fwd += c;
                if (c < 32u) break;
            }
            return fwd;
        };
        if (leaves) l_be = wq + blocks_after(k_out);
        if (enters) e_be = (leaves && k_in == k_out) ? l_be : wq;
        if (lane == 0) blk[wq] = make_uint4(e_bs, e_be, l_be, (enters ? 1u : 0u) | (leaves ? 2u : 0u));
    }
    const uint32_t pos = p0 + q;
    if (pos >= n) return;
    const uint4 me = rec[pos];
    const uint32_t pp = cellpos[me.x];              // sorted position of the cell's row-factor occurrence
    const uint32_t key = sk[pp];
    const bool left = pp > 0 && sk[pp - 1] == key, right = pp + 1 < p0 && sk[pp + 1] == key;
    uint32_t s = pp, e = pp + 1;                    // the run of the key: [s, e)
    if (left) {                                     // first position that holds the key
        uint32_t lo = 0, hi = pp - 1;               // sk[hi] == key
        while (lo < hi) {
            const uint32_t mid = (lo + hi) >> 1;
            if (sk[mid] < key) lo = mid + 1; else hi = mid;
        }
        s = lo;
    }
    if (right) {                                    // first position after pp that does not
        uint32_t lo = pp + 2, hi = p0;              // sk[lo - 1] == key
        while (lo < hi) {
            const uint32_t mid = (lo + hi) >> 1;
            if (sk[mid] <= key) lo = mid + 1; else hi = mid;
        }
        e = lo;
    }
    dup[q] = make_uint4(s, e - s, pp - s, 0u);
    if (e - s > 1 && pp == s) dup_ticket[s] = 0u;
}

enum : uint32_t { cUsable = 1, cBegin = 2, cEnd = 4, cParked = 8, cFromPrev = 16, cSingle = 32 };
enum : uint32_t { mHead = 1, mThrough = 2, mTail = 4 };

// A row in the registers of the eight lanes of a group: kC float4 per lane (lane l8 holds float4 number l8 + 8 c)
// and, with kT, one more float per lane (float 32 kC + l8) for rows that end up to eight floats after a multiple of
// 32: a row of 100 values takes 13 registers per lane instead of 16.
template <int kC, int kT>
struct RowF {
    float4 v[kC];
    float t;
};
template <int kC, int kT>
struct RowD {
    d4c v[kC];
    double t;
};

template <int kC, int kT>
__global__ void __launch_bounds__(256, 2)
mf_col_kernel(const uint32_t* __restrict__ sk, const uint4* __restrict__ rec, const uint4* __restrict__ dup,
              const uint4* __restrict__ blk, uint32_t n, uint32_t p0, float lr, float lam, float4* store, uint32_t K,
              uint32_t L4, float4* contrib, unsigned int* dup_ticket, double* bpart, unsigned int* seg_ticket,
              double* loss_partial, double* loss_accum, DevStatus* st, unsigned int epoch) {
    extern __shared__ double s_part[];              // [32 tiles][2][L]: parts entering / leaving a tile; later [8][L] warp sums
    __shared__ uint32_t s_meta[32];
    __shared__ double wl[8];
    __shared__ uint32_t s_last[3];                  // this block drew the last ticket of: the entering segment, the leaving one, the launch
    if (call_failed(st, epoch)) return;
    const unsigned full = 0xffffffffu;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5, sg = lane >> 3, l8 = lane & 7;
    const uint32_t L = L4 * 4, b = blockIdx.x, n_blocks = gridDim.x;
    const uint64_t bbase = (uint64_t)p0 + (uint64_t)b * kColBlockPos;
    const uint64_t base = bbase + (uint64_t)w * 32, pos = base + lane;
    const bool inside = pos < n;
    const uint4 me = inside ? rec[pos] : make_uint4(0u, 0u, 0u, 0u);
    const uint32_t key = inside ? sk[pos] : kSentinelPad;
    const uint4 dp = inside ? dup[pos - p0] : make_uint4(0u, 1u, 0u, 0u);
    const uint4 bi = blk[b];                        // the segments that cross this block's borders (see mf_plan_kernel)
    const float val = __uint_as_float(me.y);
    const uint32_t row = me.z, prow = me.w;
    uint32_t prev = __shfl_up_sync(full, key, 1);
    if (lane == 0) prev = (base > 0 && base - 1 < n) ? sk[base - 1] : kSentinelPad;
    uint32_t next = __shfl_down_sync(full, key, 1);
    if (lane == 31) next = (base + 32 < n) ? sk[base + 32] : kSentinelPad;
    const bool usable = key < K;
    const bool head = key != prev;
    const unsigned head_mask = __ballot_sync(full, head);
    const unsigned at_or_below = head_mask & (0xffffffffu >> (31 - lane));
    const int seg_head = at_or_below ? 31 - __clz(at_or_below) : -1;
    const bool from_prev = usable && seg_head < 8 * sg;             // the segment came in from an earlier tile
    const bool begin_me = usable && (l8 == 0 || head);              // the own row is fetched here
    const bool end_me = usable && (l8 == 7 || key != next);         // the segment's part in the tile ends here
    const bool runs_on = end_me && key == next;                     // ... and goes on in the next tile
    const bool parked = end_me && (from_prev || runs_on);
    const uint32_t flags = (usable ? cUsable : 0u) | (begin_me ? cBegin : 0u) | (end_me ? cEnd : 0u) |
                           (parked ? cParked : 0u) | (from_prev ? cFromPrev : 0u) |
                           ((begin_me && end_me && !parked) ? cSingle : 0u);
    const uint32_t tile = w * 4 + sg;
    {
        const unsigned fp = __ballot_sync(full, from_prev), ro = __ballot_sync(full, runs_on);
        if (l8 == 0)
            s_meta[tile] = (((fp >> (8 * sg)) & 1u) ? mHead : 0u) | ((((fp & ro) >> (8 * sg + 7)) & 1u) ? mThrough : 0u) |
                           ((((ro & ~fp) >> (8 * sg + 7)) & 1u) ? mTail : 0u);
    }
    const uint32_t row_last = __shfl_sync(full, row, 8 * sg + 7);   // the row of the segment that may leave the tile
    const bool tail_lane = kT && (uint32_t)(32 * kC + l8) < L;      // this lane holds one of the row's last floats

    using RF = RowF<kC, kT>;
    using RD = RowD<kC, kT>;
    const float* storef = reinterpret_cast<const float*>(store);
    float* storew = reinterpret_cast<float*>(store);
    auto zero_f = [&](RF& r) {
#pragma unroll
        for (int c = 0; c < kC; ++c) r.v[c] = make_float4(0.f, 0.f, 0.f, 0.f);
        r.t = 0.f;
    };
    auto zero_d = [&](RD& a) {
#pragma unroll
        for (int c = 0; c < kC; ++c) a.v[c] = d4c{0.0, 0.0, 0.0, 0.0};
        a.t = 0.0;
    };
    auto load_row = [&](RF& r, uint32_t rw, bool on) {      // (zeros where the lane holds nothing of the row)
#pragma unroll
        for (int c = 0; c < kC; ++c)
            r.v[c] = (on && (kT || (uint32_t)(l8 + 8 * c) < L4)) ? __ldcg(store + (uint64_t)rw * L4 + l8 + 8 * c)
                                                                : make_float4(0.f, 0.f, 0.f, 0.f);
        r.t = (on && tail_lane) ? __ldcg(storef + (uint64_t)rw * L + 32 * kC + l8) : 0.f;
    };
    auto store_row = [&](const RF& r, uint32_t rw) {
#pragma unroll
        for (int c = 0; c < kC; ++c)
            if (kT || (uint32_t)(l8 + 8 * c) < L4) __stcg(store + (uint64_t)rw * L4 + l8 + 8 * c, r.v[c]);
        if (tail_lane) __stcg(storew + (uint64_t)rw * L + 32 * kC + l8, r.t);
    };
    // a row of doubles in shared or global memory, laid out like the row
    auto put_d = [&](double* dst, const RD& a) {
#pragma unroll
        for (int c = 0; c < kC; ++c) {
            const uint32_t fi = l8 + 8 * c;
            if (!kT && fi >= L4) continue;
            *(double2*)(dst + (size_t)fi * 4) = make_double2(a.v[c].x, a.v[c].y);
            *(double2*)(dst + (size_t)fi * 4 + 2) = make_double2(a.v[c].z, a.v[c].w);
        }
        if (tail_lane) dst[32 * kC + l8] = a.t;
    };
    auto add_d = [&](RD& a, const double* src) {
#pragma unroll
        for (int c = 0; c < kC; ++c) {
            const uint32_t fi = l8 + 8 * c;
            if (!kT && fi >= L4) continue;
            const double2 x = *(const double2*)(src + (size_t)fi * 4), y = *(const double2*)(src + (size_t)fi * 4 + 2);
            a.v[c].x += x.x; a.v[c].y += x.y; a.v[c].z += y.x; a.v[c].w += y.y;
        }
        if (tail_lane) a.t += src[32 * kC + l8];
    };
    // r = (float)((double)r + a): the one rounding of a finished sum
    auto apply_d = [&](RF& r, const RD& a) {
#pragma unroll
        for (int c = 0; c < kC; ++c) {
            r.v[c].x = (float)((double)r.v[c].x + a.v[c].x); r.v[c].y = (float)((double)r.v[c].y + a.v[c].y);
            r.v[c].z = (float)((double)r.v[c].z + a.v[c].z); r.v[c].w = (float)((double)r.v[c].w + a.v[c].w);
        }
        r.t = (float)((double)r.t + a.t);
    };

    // The partner row and, where a part begins, the own row of a walk step are asked for one step ahead.
    RF hb[2], own, ownn;
    RD acc;
    zero_d(acc);
    zero_f(own);
    auto ask_partner = [&](int s2, RF& dst) {
        const int src = 8 * sg + s2;
        const uint32_t f = __shfl_sync(full, flags, src), pr = __shfl_sync(full, prow, src);
        load_row(dst, pr, (f & cUsable) != 0u);
    };
    auto ask_own = [&](int s2, RF& dst) {
        const int src = 8 * sg + s2;
        const uint32_t f = __shfl_sync(full, flags, src), rw = __shfl_sync(full, row, src);
        load_row(dst, rw, (f & cBegin) != 0u);
    };
    ask_own(0, ownn);
    ask_partner(0, hb[0]);
    float nw = 0.f, loss_f = 0.f;
    const float drop = lr * lam, keep = 1.f - lr * lam;            // what a step takes off a row through the regulariser, and leaves
    const bool any_usable = __ballot_sync(full, usable) != 0u;
#pragma unroll 2
    for (int s2 = 0; s2 < 8; ++s2) {
        if (!any_usable) break;
        const int src = 8 * sg + s2;
        const uint32_t f = __shfl_sync(full, flags, src);
        const float v = __shfl_sync(full, val, src);
        const uint32_t prow_s = __shfl_sync(full, prow, src), row_s = __shfl_sync(full, row, src);
        const uint32_t dup_s = __shfl_sync(full, dp.x, src), dup_m = __shfl_sync(full, dp.y, src),
                       dup_r = __shfl_sync(full, dp.z, src);
        const bool live = f & cUsable;
        const RF& h = hb[s2 & 1];
        if (s2 + 1 < 8) ask_partner(s2 + 1, hb[(s2 + 1) & 1]);
        if (f & cBegin) {
            own = ownn;
            nw = own.t * own.t;
#pragma unroll
            for (int c = 0; c < kC; ++c)
                nw += own.v[c].x * own.v[c].x + own.v[c].y * own.v[c].y + own.v[c].z * own.v[c].z + own.v[c].w * own.v[c].w;
            zero_d(acc);
        }
        if (s2 + 1 < 8) ask_own(s2 + 1, ownn);
        float dot = own.t * h.t, nh = h.t * h.t;
#pragma unroll
        for (int c = 0; c < kC; ++c) {
            dot += own.v[c].x * h.v[c].x + own.v[c].y * h.v[c].y + own.v[c].z * h.v[c].z + own.v[c].w * h.v[c].w;
            nh += h.v[c].x * h.v[c].x + h.v[c].y * h.v[c].y + h.v[c].z * h.v[c].z + h.v[c].w * h.v[c].w;
        }
        dot += __shfl_xor_sync(full, dot, 1);
        dot += __shfl_xor_sync(full, dot, 2);
        dot += __shfl_xor_sync(full, dot, 4);
        const float e = v - dot;
        // the cell's loss: the lanes keep their shares of the two squared norms, one lane adds the squared error
        if (live) loss_f += 0.5f * lam * (nw + nh) + (l8 == 0 ? 0.5f * e * e : 0.f);
        // ---- the cell's row factor (the partner): h + lr (e own - lam h) = (lr e) own + (1 - lr lam) h ----
        const float le = lr * e;
        const bool dupl = live && dup_m > 1u;
        if (live && !dupl) {                        // its only reader: the new row goes in place
            RF r;
#pragma unroll
            for (int c = 0; c < kC; ++c) {
                r.v[c].x = fmaf(le, own.v[c].x, keep * h.v[c].x); r.v[c].y = fmaf(le, own.v[c].y, keep * h.v[c].y);
                r.v[c].z = fmaf(le, own.v[c].z, keep * h.v[c].z); r.v[c].w = fmaf(le, own.v[c].w, keep * h.v[c].w);
            }
            r.t = fmaf(le, own.t, keep * h.t);
            store_row(r, prow_s);
        }
        if (__any_sync(full, dupl)) {               // rare: a row key with several cells in the batch
            if (dupl) {                             // the term lr (e own - lam h) on its own
#pragma unroll
                for (int c = 0; c < kC; ++c) {
                    if (!kT && (uint32_t)(l8 + 8 * c) >= L4) continue;
                    float4 t;
                    t.x = fmaf(le, own.v[c].x, -drop * h.v[c].x); t.y = fmaf(le, own.v[c].y, -drop * h.v[c].y);
                    t.z = fmaf(le, own.v[c].z, -drop * h.v[c].z); t.w = fmaf(le, own.v[c].w, -drop * h.v[c].w);
                    contrib[(uint64_t)(dup_s + dup_r) * L4 + l8 + 8 * c] = t;
                }
                if (tail_lane)
                    reinterpret_cast<float*>(contrib)[(uint64_t)(dup_s + dup_r) * L + 32 * kC + l8] = fmaf(le, own.t, -drop * h.t);
                __threadfence();
            }
            __syncwarp();
            uint32_t tk = 0u;
            if (dupl && l8 == 0) tk = atomicAdd(&dup_ticket[dup_s], 1u);
            tk = __shfl_sync(full, tk, lane & ~7);
            if (dupl && tk == dup_m - 1u) {         // every reader of the row has read it: add the terms in position order
                __threadfence();
                RF r = h;
#pragma unroll
                for (int c = 0; c < kC; ++c) {
                    if (!kT && (uint32_t)(l8 + 8 * c) >= L4) continue;
                    d4c a = {0.0, 0.0, 0.0, 0.0};
                    for (uint32_t rr = 0; rr < dup_m; ++rr) {
                        const float4 t = __ldcg(contrib + (uint64_t)(dup_s + rr) * L4 + l8 + 8 * c);
                        a.x += (double)t.x; a.y += (double)t.y; a.z += (double)t.z; a.w += (double)t.w;
                    }
                    r.v[c].x = (float)((double)r.v[c].x + a.x); r.v[c].y = (float)((double)r.v[c].y + a.y);
                    r.v[c].z = (float)((double)r.v[c].z + a.z); r.v[c].w = (float)((double)r.v[c].w + a.w);
                }
                if (tail_lane) {
                    double a = 0.0;
                    for (uint32_t rr = 0; rr < dup_m; ++rr)
                        a += (double)__ldcg(reinterpret_cast<const float*>(contrib) + (uint64_t)(dup_s + rr) * L + 32 * kC + l8);
                    r.t = (float)((double)r.t + a);
                }
                store_row(r, prow_s);
            }
        }
        // ---- the cell's column factor (the own row): term lr (e h - lam own) ----
        if (f & cSingle) {                          // a segment of this one position: the new row in fp32, one rounding of the sum
            RF r;
#pragma unroll
            for (int c = 0; c < kC; ++c) {
                r.v[c].x = fmaf(le, h.v[c].x, keep * own.v[c].x); r.v[c].y = fmaf(le, h.v[c].y, keep * own.v[c].y);
                r.v[c].z = fmaf(le, h.v[c].z, keep * own.v[c].z); r.v[c].w = fmaf(le, h.v[c].w, keep * own.v[c].w);
            }
            r.t = fmaf(le, h.t, keep * own.t);
            store_row(r, row_s);
        } else if (live) {
#pragma unroll
            for (int c = 0; c < kC; ++c) {
                acc.v[c].x += (double)fmaf(le, h.v[c].x, -drop * own.v[c].x); acc.v[c].y += (double)fmaf(le, h.v[c].y, -drop * own.v[c].y);
                acc.v[c].z += (double)fmaf(le, h.v[c].z, -drop * own.v[c].z); acc.v[c].w += (double)fmaf(le, h.v[c].w, -drop * own.v[c].w);
            }
            acc.t += (double)fmaf(le, h.t, -drop * own.t);
            if (f & cEnd) {
                if (f & cParked) {
                    put_d(s_part + ((size_t)tile * 2 + ((f & cFromPrev) ? 0 : 1)) * L, acc);
                } else {                            // the whole segment lies in this tile: nobody else reads its row
                    RF r = own;
                    apply_d(r, acc);
                    store_row(r, row_s);
                }
            }
        }
    }
    // per-block loss partial, fixed order
    {
        const double lw = warp_sum_d((double)loss_f);
        if (lane == 0) wl[w] = lw;
    }
    __syncthreads();
    // ---- chains of parts inside the block, in tile order ----
    // Which tiles a segment runs through is known for the whole block at once (a bit per tile), so a chain's length is
    // known before its first part is read.  The four groups of a warp walk their chains together (the same
    // instructions, each group adding only while its own chain lasts), not one after the other.
    const unsigned thr_mask = __ballot_sync(full, (s_meta[lane] & mThrough) != 0u);
    const uint32_t my_meta = s_meta[tile];
    // the chain that starts with this tile's last part; in tile 0 also the one that enters the block
    auto chain_len = [&](uint32_t t, bool* ends) {
        const unsigned after = t < 31u ? ~(thr_mask >> (t + 1)) : 1u;      // bit j: tile t + 1 + j is not run through
        const uint32_t through_n = (uint32_t)__ffs(after) - 1u;            // (the shift brings in zeros: `after` is never 0)
        *ends = t + through_n + 1u < 32u;
        return tmin<uint32_t>(t + through_n + 1u, 31u) - t;
    };
    const bool has_tail = (my_meta & mTail) != 0u;
    bool tail_ends = false;
    const uint32_t tail_links = has_tail ? chain_len(tile, &tail_ends) : 0u;
    uint32_t max_links = tail_links;
    max_links = tmax(max_links, __shfl_xor_sync(full, max_links, 8));
    max_links = tmax(max_links, __shfl_xor_sync(full, max_links, 16));
    RD a;
    zero_d(a);
    if (has_tail) add_d(a, s_part + ((size_t)tile * 2 + 1) * L);
    for (uint32_t j = 1; j <= max_links; ++j)
        if (j <= tail_links) add_d(a, s_part + ((size_t)(tile + j) * 2) * L);
    if (has_tail) {
        if (tail_ends) {                            // the segment ends inside the block; `own` still holds its row
            RF r = own;
            apply_d(r, a);
            store_row(r, row_last);
        } else {
            put_d(bpart + ((size_t)b * 2 + 1) * L, a);
        }
    }
    if (tile == 0 && (my_meta & mHead)) {           // the segment that enters the block
        bool ends = true;
        const uint32_t links = (my_meta & mThrough) ? chain_len(0, &ends) : 0u;
        zero_d(a);
        for (uint32_t j = 0; j <= links; ++j) add_d(a, s_part + ((size_t)j * 2) * L);
        put_d(bpart + ((size_t)b * 2) * L, a);
    }
    __syncthreads();
    // ---- segments that cross the block's borders take a ticket from the counter of the block they start in; so
    // does the launch as a whole.  One thread each, in different warps.
    const bool enters = bi.w & 1u, leaves = bi.w & 2u;
    const bool through = enters && leaves && bi.y != b;            // the entering segment is also the leaving one
    if (tid == 0) {
        s_last[0] = 0u;
        if (enters) {
            __threadfence();
            s_last[0] = atomicAdd(&seg_ticket[bi.x], 1u) == bi.y - bi.x ? 1u : 0u;
        }
    } else if (tid == 32) {
        s_last[1] = 0u;
        if (leaves && !through) {
            __threadfence();
            s_last[1] = atomicAdd(&seg_ticket[b], 1u) == bi.z - b ? 1u : 0u;
        }
    } else if (tid == 64) {
        double t = 0;
        for (int i = 0; i < 8; ++i) t += wl[i];
        loss_partial[b] = t;
        __threadfence();
        s_last[2] = atomicAdd(&seg_ticket[n_blocks], 1u) == n_blocks - 1 ? 1u : 0u;
    }
    __syncthreads();
    // ---- the block that drew a segment's last ticket adds its parts in block order and writes the row ----
    double* s_sum = s_part;                         // [8 warps][L]
    for (int i = 0; i < 2; ++i) {
        if (!s_last[i]) continue;                   // the same decision in every thread
        __threadfence();
        const uint32_t bs = i == 0 ? bi.x : b, n_parts = (i == 0 ? bi.y : bi.z) - bs + 1;
        const uint32_t fi = lane;                   // rows of at most 32 float4
        d4c a = {0.0, 0.0, 0.0, 0.0};
        if (fi < L4) {
            for (uint32_t j0 = w; j0 < n_parts; j0 += 32) {
                double2 x[4], y[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t j = j0 + 8 * k;
                    x[k] = y[k] = make_double2(0.0, 0.0);
                    if (j < n_parts) {
                        const double* g = bpart + ((size_t)(bs + j) * 2 + (j == 0 ? 1 : 0)) * L + (size_t)fi * 4;
                        x[k] = __ldcg((const double2*)g);
                        y[k] = __ldcg((const double2*)(g + 2));
                    }
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    a.x += x[k].x; a.y += x[k].y; a.z += y[k].x; a.w += y[k].y;
                }
            }
            double* d = s_sum + (size_t)w * L + (size_t)fi * 4;
            d[0] = a.x; d[1] = a.y; d[2] = a.z; d[3] = a.w;
        }
        __syncthreads();
        if (w == 0 && fi < L4) {
            d4c t = {0.0, 0.0, 0.0, 0.0};
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const double* d = s_sum + (size_t)k * L + (size_t)fi * 4;
                t.x += d[0]; t.y += d[1]; t.z += d[2]; t.w += d[3];
            }
            // the segment's row: that of the block's first position (entering) or of its last one (leaving)
            const uint64_t rw = i == 0 ? rec[bbase].z : rec[tmin<uint64_t>(bbase + kColBlockPos, n) - 1].z;
            float4 r = __ldcg(store + rw * L4 + fi);
            r.x = (float)((double)r.x + t.x); r.y = (float)((double)r.y + t.y);
            r.z = (float)((double)r.z + t.z); r.w = (float)((double)r.w + t.w);
            store[rw * L4 + fi] = r;
        }
        __syncthreads();
    }
    // ---- the last block adds the call's loss partials, in index order ----
    if (s_last[2] && loss_accum && w == 0) {
        __threadfence();
        double t = 0;
        for (uint32_t k = lane; k < n_blocks; k += 32) t += __ldcg(loss_partial + k);
        t = warp_sum_d(t);
        if (lane == 0) *loss_accum += t;
    }
}

// after the sort, on the stream the sort ran on
void launch_mf_plan(ps_store* ps, uint32_t n_cells, int which, cudaStream_t side) {
    const uint32_t* sk = which ? ps->keysB : ps->keysA;
    const uint32_t n = 2 * n_cells, p0 = n_cells;
    const uint32_t n_blocks = div_up_u32(n_cells, kColBlockPos);
    const uint32_t threads = tmax<uint32_t>(n_cells, 32 * n_blocks);
    PS_LAUNCH(ps, mf_plan_kernel, div_up_u32(threads, 256), 256, side, sk, ps->rec, ps->cellpos, n, p0, ps->mf_dup,
              ps->mf_dup + ps->max_keys / 2 + 1, ps->mf_tickets, ps->mf_tickets + ps->max_keys / 2 + 1, n_blocks,
              ps->status, ps->epoch);
}

void run_mf_col(ps_store* ps, uint32_t n_cells, int which, float lr, float lambda, double* d_loss_accum, cudaStream_t s) {
    const uint32_t* sk = which ? ps->keysB : ps->keysA;
    const uint32_t n = 2 * n_cells, p0 = n_cells;
    const uint32_t L4 = ps->cfg.row_len / 4;
    const uint32_t blocks = div_up_u32(n_cells, kColBlockPos);
    const size_t smem = (size_t)32 * 2 * ps->cfg.row_len * sizeof(double);
#define COL_ARGS                                                                                                       \
    sk, ps->rec, ps->mf_dup, ps->mf_dup + ps->max_keys / 2 + 1, n, p0, lr, lambda, (float4*)ps->store,                 \
        (uint32_t)ps->cfg.num_keys, L4, (float4*)ps->upd, ps->mf_tickets, ps->carry,                                  \
        ps->mf_tickets + ps->max_keys / 2 + 1, ps->loss_partial, d_loss_accum, ps->status, ps->epoch
#define COL_LAUNCH(kC, kT)                                                                                             \
    do {                                                                                                               \
        static std::atomic<unsigned long long> smem_set{0};                                                            \
        opt_in_smem((const void*)mf_col_kernel<kC, kT>, (size_t)32 * 2 * 32 * (kC + kT) * sizeof(double), &smem_set);  \
        if (ps->prof) prof_before(ps, "mf_col_kernel<" #kC "," #kT ">", s);                                            \
        mf_col_kernel<kC, kT><<<blocks, 256, smem, s>>>(COL_ARGS);                                                     \
        if (ps->prof) prof_after(ps, s);                                                                               \
        ps->launches++;                                                                                                \
    } while (0)
    // whole float4 chunks of eight per group of lanes; a remainder of one or two float4 travels as one float per lane
    const uint32_t full_chunks = L4 / 8, rem = L4 % 8;
    if (rem == 0) {
        if (full_chunks == 1) COL_LAUNCH(1, 0);
        else if (full_chunks == 2) COL_LAUNCH(2, 0);
        else if (full_chunks == 3) COL_LAUNCH(3, 0);
        else COL_LAUNCH(4, 0);
    } else if (rem <= 2 && full_chunks >= 1) {
        if (full_chunks == 1) COL_LAUNCH(1, 1);
        else if (full_chunks == 2) COL_LAUNCH(2, 1);
        else COL_LAUNCH(3, 1);
    } else {
        if (full_chunks == 0) COL_LAUNCH(1, 0);
        else if (full_chunks == 1) COL_LAUNCH(2, 0);
        else if (full_chunks == 2) COL_LAUNCH(3, 0);
        else COL_LAUNCH(4, 0);
    }
#undef COL_LAUNCH
#undef COL_ARGS
}

}  // namespace psb
