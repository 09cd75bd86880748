// Fused pull -> per-example gradient kernels of the three training tasks of
// Section 4.1 / Appendix A of the paper.  One warp handles one example (a
// matrix cell, a knowledge-graph data point with its negatives, a skip-gram
// center word with its window): it looks the example's keys up in the location
// table, gathers their rows with coalesced loads, forms dot products with warp
// shuffles, and writes one additive update row per key occurrence plus that
// occurrence's key.  The push stage (pull_push.cu) then sorts the occurrences
// by key, sums them per key and applies them, so every read in here sees the
// state from before the step.
#include "ps_internal.cuh"

namespace psb {

__device__ __forceinline__ float softplusf(float z) { return fmaxf(z, 0.f) + log1pf(expf(-fabsf(z))); }
__device__ __forceinline__ float sigmoidf(float z) {
    if (z >= 0.f) return 1.f / (1.f + expf(-z));
    const float e = expf(z);
    return e / (1.f + e);
}
__device__ __forceinline__ double softplus_d(double z) { return fmax(z, 0.0) + log1p(exp(-fabs(z))); }
__device__ __forceinline__ double sigmoid_d(double z) {
    if (z >= 0.0) return 1.0 / (1.0 + exp(-z));
    const double e = exp(z);
    return e / (1.0 + e);
}

// Sum of the warps' loss terms -> loss_partial[blockIdx.x]; fixed order.
__device__ __forceinline__ void block_loss_out(double loss, double* __restrict__ loss_partial) {
    __shared__ double wl[8];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) wl[w] = loss;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0;
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += wl[i];
        loss_partial[blockIdx.x] = t;
    }
}

// blocks_per_sm: how many blocks of the kernel an SM holds.  With exactly the resident number of blocks every warp
// loops over its share of the examples, and the shares differ by at most one example; with more blocks than fit, the
// last wave is partly empty.
static uint32_t step_grid(ps_store* ps, uint64_t n_examples, uint32_t blocks_per_sm = 8) {
    uint64_t g = (n_examples + 7) / 8;
    const uint64_t cap = (uint64_t)ps->sm_count * blocks_per_sm;
    if (g > cap) g = cap;
    if (g > kMaxLossBlocks) g = kMaxLossBlocks;
    return g ? (uint32_t)g : 1u;
}

// ------------------------------------------------------------------ MF ----
// kCh = number of float4 a lane holds per row (row_len <= 128 * kCh); 0 = any
// row length, rows re-read from cache for the second pass.
template <int kCh>
__global__ void __launch_bounds__(256)
mf_step_kernel(const uint32_t* __restrict__ ci, const uint32_t* __restrict__ cj, const float* __restrict__ cv,
               uint64_t n, uint64_t col_base, float lr, float lam, const float4* __restrict__ store,
               const uint2* __restrict__ table, uint64_t S, uint64_t K, uint32_t L4,
               float4* __restrict__ upd, double* __restrict__ loss_partial, DevStatus* st, unsigned int epoch) {
    const int lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t n_warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    constexpr int kRegs = kCh > 0 ? kCh : 1;
    double loss = 0;
    for (uint64_t t = warp; t < n; t += n_warps) {
        const uint32_t i = ci[t], j = cj[t];
        const float v = cv[t];
        const uint64_t kw = i, kh = col_base + j;
        if (kw >= col_base || kh >= K) {
            if (lane == 0) latch_error(st, epoch, PS_ERR_KEY_RANGE);
            continue;
        }
        const float4* W = store + phys_row(table[kw], S) * L4;
        const float4* H = store + phys_row(table[kh], S) * L4;
        float4 w[kRegs], h[kRegs];
        float dot = 0.f, nw = 0.f, nh = 0.f;
        if constexpr (kCh > 0) {
#pragma unroll
            for (int c = 0; c < kCh; ++c) {
                const uint32_t f = lane + 32 * c;
                w[c] = f < L4 ? W[f] : make_float4(0.f, 0.f, 0.f, 0.f);
                h[c] = f < L4 ? H[f] : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int c = 0; c < kCh; ++c) {
                dot += w[c].x * h[c].x + w[c].y * h[c].y + w[c].z * h[c].z + w[c].w * h[c].w;
                nw += w[c].x * w[c].x + w[c].y * w[c].y + w[c].z * w[c].z + w[c].w * w[c].w;
                nh += h[c].x * h[c].x + h[c].y * h[c].y + h[c].z * h[c].z + h[c].w * h[c].w;
            }
        } else {
            for (uint32_t f = lane; f < L4; f += 32) {
                const float4 a = W[f], b = H[f];
                dot += a.x * b.x + a.y * b.y + a.z * b.z + a.w * b.w;
                nw += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
                nh += b.x * b.x + b.y * b.y + b.z * b.z + b.w * b.w;
            }
        }
        dot = warp_sum(dot);
        nw = warp_sum(nw);
        nh = warp_sum(nh);
        const float e = v - dot;
        loss += (double)(0.5f * e * e + 0.5f * lam * (nw + nh));
        float4* UW = upd + (2 * t) * L4;
        float4* UH = upd + (2 * t + 1) * L4;
        auto emit = [&](uint32_t f, const float4& a, const float4& b) {
            float4 dw, dh;
            dw.x = lr * (e * b.x - lam * a.x); dw.y = lr * (e * b.y - lam * a.y);
            dw.z = lr * (e * b.z - lam * a.z); dw.w = lr * (e * b.w - lam * a.w);
            dh.x = lr * (e * a.x - lam * b.x); dh.y = lr * (e * a.y - lam * b.y);
            dh.z = lr * (e * a.z - lam * b.z); dh.w = lr * (e * a.w - lam * b.w);
            UW[f] = dw;
            UH[f] = dh;
        };
        if constexpr (kCh > 0) {
#pragma unroll
            for (int c = 0; c < kCh; ++c) {
                const uint32_t f = lane + 32 * c;
                if (f < L4) emit(f, w[c], h[c]);
            }
        } else {
            for (uint32_t f = lane; f < L4; f += 32) emit(f, W[f], H[f]);
        }
    }
    block_loss_out(loss, loss_partial);
}

// Rows of at most 128 values: one float4 per lane and row.  A warp works on kCells cells at a time so
// that their index, table and row loads are all in flight together (each cell is a chain of three
// dependent loads; one cell per warp leaves the memory system idle most of the time).
template <int kCells>
__global__ void __launch_bounds__(256)
mf_step_small_kernel(const uint32_t* __restrict__ ci, const uint32_t* __restrict__ cj, const float* __restrict__ cv,
                     uint64_t n, uint64_t col_base, float lr, float lam, const float4* __restrict__ store,
                     const uint2* __restrict__ table, uint64_t S, uint64_t K, uint32_t L4,
                     float4* __restrict__ upd, double* __restrict__ loss_partial, DevStatus* st,
                     unsigned int epoch) {
    const int lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t n_warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    const bool act = (uint32_t)lane < L4;
    double loss = 0;
    for (uint64_t t0 = warp * kCells; t0 < n; t0 += n_warps * kCells) {
        uint64_t kw[kCells], kh[kCells];
        float v[kCells];
        bool ok[kCells];
#pragma unroll
        for (int c = 0; c < kCells; ++c) {
            const uint64_t t = t0 + c;
            ok[c] = t < n;
            kw[c] = ok[c] ? ci[t] : 0;
            kh[c] = ok[c] ? col_base + cj[t] : 0;
            v[c] = ok[c] ? cv[t] : 0.f;
            if (ok[c] && (kw[c] >= col_base || kh[c] >= K)) {
                if (lane == 0) latch_error(st, epoch, PS_ERR_KEY_RANGE);
                ok[c] = false;
            }
        }
        uint2 ew[kCells], eh[kCells];
#pragma unroll
        for (int c = 0; c < kCells; ++c) {
            ew[c] = ok[c] ? table[kw[c]] : make_uint2(0, 0);
            eh[c] = ok[c] ? table[kh[c]] : make_uint2(0, 0);
        }
        float4 w[kCells], h[kCells];
#pragma unroll
        for (int c = 0; c < kCells; ++c) {
            const bool ld = ok[c] && act;
            w[c] = ld ? store[phys_row(ew[c], S) * L4 + lane] : make_float4(0.f, 0.f, 0.f, 0.f);
            h[c] = ld ? store[phys_row(eh[c], S) * L4 + lane] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int c = 0; c < kCells; ++c) {
            float dot = w[c].x * h[c].x + w[c].y * h[c].y + w[c].z * h[c].z + w[c].w * h[c].w;
            float nw = w[c].x * w[c].x + w[c].y * w[c].y + w[c].z * w[c].z + w[c].w * w[c].w;
            float nh = h[c].x * h[c].x + h[c].y * h[c].y + h[c].z * h[c].z + h[c].w * h[c].w;
            dot = warp_sum(dot);
            nw = warp_sum(nw);
            nh = warp_sum(nh);
            if (!ok[c]) continue;
            const float e = v[c] - dot;
            loss += (double)(0.5f * e * e + 0.5f * lam * (nw + nh));
            if (act) {
                const uint64_t t = t0 + c;
                float4 dw, dh;
                dw.x = lr * (e * h[c].x - lam * w[c].x); dw.y = lr * (e * h[c].y - lam * w[c].y);
                dw.z = lr * (e * h[c].z - lam * w[c].z); dw.w = lr * (e * h[c].w - lam * w[c].w);
                dh.x = lr * (e * w[c].x - lam * h[c].x); dh.y = lr * (e * w[c].y - lam * h[c].y);
                dh.z = lr * (e * w[c].z - lam * h[c].z); dh.w = lr * (e * w[c].w - lam * h[c].w);
                upd[(2 * t) * L4 + lane] = dw;
                upd[(2 * t + 1) * L4 + lane] = dh;
            }
        }
    }
    block_loss_out(loss, loss_partial);
}

uint32_t launch_step_mf(ps_store* ps, const uint32_t* d_i, const uint32_t* d_j, const float* d_v, uint64_t n,
                        uint64_t col_key_base, float lr, float lambda, cudaStream_t s) {
    const uint32_t L4 = ps->cfg.row_len / 4;
    const uint32_t grid = step_grid(ps, n);
#define MF_ARGS d_i, d_j, d_v, n, col_key_base, lr, lambda, (const float4*)ps->store, ps->table,                 \
                ps->cfg.slots_per_part, ps->cfg.num_keys, L4, (float4*)ps->upd, ps->loss_partial,              \
                ps->status, ps->epoch
    if (L4 <= 32) PS_LAUNCH(ps, mf_step_small_kernel<4>, grid, 256, s, MF_ARGS);
    else if (L4 <= 64) PS_LAUNCH(ps, mf_step_kernel<2>, grid, 256, s, MF_ARGS);
    else if (L4 <= 128) PS_LAUNCH(ps, mf_step_kernel<4>, grid, 256, s, MF_ARGS);
    else PS_LAUNCH(ps, mf_step_kernel<0>, grid, 256, s, MF_ARGS);
#undef MF_ARGS
    return grid;
}

// ------------------------------------------------------------- ComplEx ----
// Slots of a data point: 0 = subject, 1 = relation, 2 = object, 3 + q = the
// q-th negative entity.  Lane u holds slot u's key and row offset.  Slots that
// repeat an earlier slot's key emit no update (key mark K): their gradient is
// folded into the first slot with that key, so that AdaGrad sees the gradient
// of the data point's loss with respect to each DISTINCT key.
//
// Scores and gradient sums are formed in fp64 from the fp32 rows.  With a zero
// accumulator AdaGrad's step is -lr * g / (|g| + eps), which near g = 0 turns
// rounding noise of g into a visible change of the parameter; fp64 sums keep
// that noise far below the fp32 resolution of the result.  The final AdaGrad
// expression is evaluated in fp32 on the rounded gradient.
// kMaxNeg bounds n_neg at compile time so that a data point's values live in registers: for every block
// of 32 complex dimensions the Re and Im of all its rows are requested together, before any is used.
// kDim / kExactNeg: the complex dimension and "n_neg equals kMaxNeg" known at compile time (0 / false: taken from
// the arguments).  With both fixed the offsets of the four quarters of a row become immediates and the tests on
// the number of negatives fold away; the kernel spends more issue slots on integer bookkeeping than on fp64.
// kGradOnly: the update row of a slot is the GRADIENT of the data point's loss with respect to the slot's key
// (2 d values, Re then Im), and the reduction turns it into the AdaGrad step from the accumulators it finds in the
// target row (kge_reduce_kernel); otherwise the row is the finished pair (step, squared gradient) of 4 d values.
template <int kMaxNeg, int kDim, bool kExactNeg, bool kGradOnly>
__global__ void __launch_bounds__(256, kMaxNeg <= 10 ? 2 : 1)
kge_step_kernel(const uint32_t* __restrict__ ts, const uint32_t* __restrict__ tr, const uint32_t* __restrict__ to,
                const uint32_t* __restrict__ neg_ent, const uint8_t* __restrict__ neg_side, uint64_t n,
                uint32_t n_neg_arg, uint64_t rel_base, uint32_t d_arg, float lr, float eps, const float* __restrict__ store,
                const uint2* __restrict__ table, uint64_t S, uint64_t K, float* __restrict__ upd,
                double* __restrict__ loss_partial, DevStatus* st, unsigned int epoch) {
    const int lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t n_warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    const uint32_t d = kDim ? (uint32_t)kDim : d_arg;
    const uint32_t n_neg = kExactNeg ? (uint32_t)kMaxNeg : n_neg_arg;
    const int n_slots = 3 + (int)n_neg;
    const uint32_t L = 4 * d;
    const unsigned full = 0xffffffffu;
    double loss = 0;
    for (uint64_t t = warp; t < n; t += n_warps) {
        // ---- keys, validity, row offsets, first-slot-with-same-key (lane u holds slot u) ----
        uint64_t key = K;
        int side = 0;
        bool bad = false;
        if (lane < n_slots) {
            if (lane == 1) {
                key = rel_base + tr[t];
                bad = key >= K;
            } else {
                const uint32_t e = lane == 0 ? ts[t] : (lane == 2 ? to[t] : neg_ent[t * n_neg + (lane - 3)]);
                key = e;
                bad = e >= rel_base;
                if (lane >= 3) side = neg_side[t * n_neg + (lane - 3)] != 0;
            }
        }
        if (__any_sync(full, bad)) {
            if (lane == 0) latch_error(st, epoch, PS_ERR_KEY_RANGE);
            continue;
        }
        uint64_t off = 0;
        if (lane < n_slots) off = phys_row(table[key], S) * L;
        int rep = lane;
        for (int z = n_slots - 1; z >= 0; --z) {
            const uint64_t kz = __shfl_sync(full, key, z);
            if (z < lane && kz == key) rep = z;
        }
        const float* Srow = store + __shfl_sync(full, off, 0);
        const float* Rrow = store + __shfl_sync(full, off, 1);
        const float* Orow = store + __shfl_sync(full, off, 2);
        const float* Nrow[kMaxNeg];
#pragma unroll
        for (int q = 0; q < kMaxNeg; ++q) Nrow[q] = store + __shfl_sync(full, off, (3 + q) & 31);
        // bit q: negative q stands in the subject's place / is the first slot with its key
        const unsigned subj_mask = __ballot_sync(full, lane >= 3 && lane < n_slots && side == 0) >> 3;
        const unsigned nrep_mask = __ballot_sync(full, lane >= 3 && lane < n_slots && rep == lane) >> 3;

        // ---- pass A: partial scores of the 1 + n_neg triples over this lane's dimensions ----
        double part[kMaxNeg + 1];
#pragma unroll
        for (int q = 0; q <= kMaxNeg; ++q) part[q] = 0.0;
        for (uint32_t c = lane; c < d; c += 32) {
            const float a_f = Srow[c], b_f = Srow[d + c], cr_f = Rrow[c], ci_f = Rrow[d + c];
            const float e_f = Orow[c], f_f = Orow[d + c];
            float na_f[kMaxNeg], nb_f[kMaxNeg];
#pragma unroll
            for (int q = 0; q < kMaxNeg; ++q) {
                na_f[q] = q < (int)n_neg ? Nrow[q][c] : 0.f;
                nb_f[q] = q < (int)n_neg ? Nrow[q][d + c] : 0.f;
            }
            const double a = a_f, b = b_f, cr = cr_f, ci = ci_f, e = e_f, f = f_f;
            part[0] += cr * (a * e + b * f) + ci * (a * f - b * e);
            // (n, r, o): cr (na e + nb f) + ci (na f - nb e);   (s, r, n): cr (a na + b nb) + ci (a nb - b na)
            const double re_o = cr * e + ci * f, im_o = cr * f - ci * e;        // multiplies (na, nb) for side 0
            const double re_s = cr * a - ci * b, im_s = cr * b + ci * a;        // multiplies (na, nb) for side 1
#pragma unroll
            for (int q = 0; q < kMaxNeg; ++q) {
                const double na = na_f[q], nb = nb_f[q];
                part[q + 1] += ((subj_mask >> q) & 1u) ? (na * re_o + nb * im_o) : (na * re_s + nb * im_s);
            }
        }
        // lane q keeps triple q's score
        double phi_mine = 0;
#pragma unroll
        for (int q = 0; q <= kMaxNeg; ++q) {
            if (q <= (int)n_neg) {
                const double phi = warp_sum_d(part[q]);
                if (lane == q) phi_mine = phi;
            }
        }
        // lane q: loss term and d loss / d phi of triple q (label +1 for the positive, -1 for negatives)
        double coef = 0, loss_q = 0;
        if (lane <= (int)n_neg) {
            const double y = lane == 0 ? 1.0 : -1.0;
            loss_q = softplus_d(-y * phi_mine);
            coef = -y * sigmoid_d(-y * phi_mine);
        }
        loss += warp_sum_d(loss_q);

        // ---- weights with which each entity slot receives the two "negative role" directions ----
        // A negative with side 0 stands in the subject's place: its gradient is coef * dphi/dS(r, o).
        // With side 1 it stands in the object's place: coef * dphi/dO(s, r).  Summed over the
        // negatives whose key's first slot is this lane.
        double wS = 0, wO = 0;
#pragma unroll
        for (int q = 0; q < kMaxNeg; ++q) {
            const int rq = __shfl_sync(full, rep, (3 + q) & 31);
            const double cfq = __shfl_sync(full, coef, (q + 1) & 31);
            if (q < (int)n_neg && rq == lane) {
                if ((subj_mask >> q) & 1u) wS += cfq; else wO += cfq;
            }
        }
        const double cf0 = __shfl_sync(full, coef, 0);
        const int rep_o = __shfl_sync(full, rep, 2);            // 0 if object == subject
        const double wS0 = __shfl_sync(full, wS, 0), wO0 = __shfl_sync(full, wO, 0);
        const double wS2 = __shfl_sync(full, wS, 2), wO2 = __shfl_sync(full, wO, 2);

        // ---- pass B: gradients per block of 32 complex dimensions, AdaGrad, update rows ----
        const uint32_t LU = kGradOnly ? 2 * d : L;        // values per update row
        float* U = upd + (t * n_slots) * LU;
        // -lr g / (sqrt(G + g^2) + eps) with the hardware reciprocal square root and reciprocal (each within
        // 2 ulp, far inside the fp32 tolerance of the result); x = 0 is kept away from 0 * inf
        auto adagrad_out = [&](float* Uu, uint32_t c, double gd_re, double gd_im, float G_re, float G_im) {
            const float g_re = (float)gd_re, g_im = (float)gd_im;
            if (kGradOnly) {
                Uu[c] = g_re;
                Uu[d + c] = g_im;
                return;
            }
            const float g2_re = g_re * g_re, g2_im = g_im * g_im;
            Uu[c] = adagrad_step(g_re, G_re + g2_re, lr, eps);
            Uu[d + c] = adagrad_step(g_im, G_im + g2_im, lr, eps);
            Uu[2 * d + c] = g2_re;
            Uu[3 * d + c] = g2_im;
        };
        for (uint32_t c0 = 0; c0 < d; c0 += 32) {
            const uint32_t c = c0 + lane;
            const bool act = c < d;
            const uint32_t cl = act ? c : 0;                 // idle lanes read (and discard) dimension 0
            // every value this block of dimensions needs, requested before the first use
            const float a_f = Srow[cl], b_f = Srow[d + cl], cr_f = Rrow[cl], ci_f = Rrow[d + cl];
            const float e_f = Orow[cl], f_f = Orow[d + cl];
            float GS_re = 0.f, GS_im = 0.f, GR_re = 0.f, GR_im = 0.f, GO_re = 0.f, GO_im = 0.f;
            if (!kGradOnly) {
                GS_re = Srow[2 * d + cl]; GS_im = Srow[3 * d + cl];
                GR_re = Rrow[2 * d + cl]; GR_im = Rrow[3 * d + cl];
                GO_re = Orow[2 * d + cl]; GO_im = Orow[3 * d + cl];
            }
            float na_f[kMaxNeg], nb_f[kMaxNeg], GN_re[kMaxNeg], GN_im[kMaxNeg];
#pragma unroll
            for (int q = 0; q < kMaxNeg; ++q) {
                const bool live = q < (int)n_neg;
                na_f[q] = live ? Nrow[q][cl] : 0.f;
                nb_f[q] = live ? Nrow[q][d + cl] : 0.f;
                GN_re[q] = (!kGradOnly && ((nrep_mask >> q) & 1u)) ? Nrow[q][2 * d + cl] : 0.f;
                GN_im[q] = (!kGradOnly && ((nrep_mask >> q) & 1u)) ? Nrow[q][3 * d + cl] : 0.f;
            }
            const double a = a_f, b = b_f, cr = cr_f, ci = ci_f, e = e_f, f = f_f;
            // directions that do not depend on the negative
            const double dS_re = cr * e + ci * f, dS_im = cr * f - ci * e;      // d phi / d subject, object = o
            const double dO_re = cr * a - ci * b, dO_im = cr * b + ci * a;      // d phi / d object, subject = s
            double gs_re = cf0 * dS_re, gs_im = cf0 * dS_im;
            double go_re = cf0 * dO_re, go_im = cf0 * dO_im;
            double gr_re = cf0 * (a * e + b * f), gr_im = cf0 * (a * f - b * e);
            // The negatives enter the gradients of subject, relation and object only through their weighted sums:
            // (A0, B0) over those in the subject's place (triples (n, r, o)), (A1, B1) over those in the object's
            // place (triples (s, r, n)).  Two multiply-adds per negative instead of twelve.
            double A0 = 0.0, B0 = 0.0, A1 = 0.0, B1 = 0.0;
#pragma unroll
            for (int q = 0; q < kMaxNeg; ++q) {
                const double na = na_f[q], nb = nb_f[q];
                const double w = __shfl_sync(full, coef, (q + 1) & 31);
                const bool in_subject_place = (subj_mask >> q) & 1u;
                const double w0 = in_subject_place ? w : 0.0, w1 = in_subject_place ? 0.0 : w;
                A0 += w0 * na; B0 += w0 * nb;
                A1 += w1 * na; B1 += w1 * nb;
            }
            gr_re += (A0 * e + B0 * f) + (a * A1 + b * B1); gr_im += (A0 * f - B0 * e) + (a * B1 - b * A1);
            go_re += cr * A0 - ci * B0; go_im += cr * B0 + ci * A0;
            gs_re += cr * A1 + ci * B1; gs_im += cr * B1 - ci * A1;
            // negatives that coincide with the subject or the object
            gs_re += wS0 * dS_re + wO0 * dO_re; gs_im += wS0 * dS_im + wO0 * dO_im;
            go_re += wS2 * dS_re + wO2 * dO_re; go_im += wS2 * dS_im + wO2 * dO_im;
            if (rep_o == 0) { gs_re += go_re; gs_im += go_im; }
            if (act) {
                adagrad_out(U, c, gs_re, gs_im, GS_re, GS_im);
                adagrad_out(U + LU, c, gr_re, gr_im, GR_re, GR_im);
                if (rep_o == 2) adagrad_out(U + 2 * (uint64_t)LU, c, go_re, go_im, GO_re, GO_im);
            }
#pragma unroll
            for (int q = 0; q < kMaxNeg; ++q) {
                const double wSq = __shfl_sync(full, wS, (3 + q) & 31), wOq = __shfl_sync(full, wO, (3 + q) & 31);
                if (act && ((nrep_mask >> q) & 1u))
                    adagrad_out(U + (uint64_t)(3 + q) * LU, c, wSq * dS_re + wOq * dO_re, wSq * dS_im + wOq * dO_im,
                                GN_re[q], GN_im[q]);
            }
        }
    }
    block_loss_out(loss, loss_partial);
}

// Keys of the occurrence slots of each data point; a slot that repeats an earlier slot's key, and every
// slot of a data point with an index out of range, gets the "no key" mark K.
__global__ void __launch_bounds__(256)
kge_keys_kernel(const uint32_t* __restrict__ ts, const uint32_t* __restrict__ tr, const uint32_t* __restrict__ to,
                const uint32_t* __restrict__ neg_ent, uint64_t n, uint32_t n_neg, uint64_t rel_base, uint64_t K,
                uint32_t* __restrict__ keys_out, DevStatus* st, unsigned int epoch) {
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n) return;
    const int n_slots = 3 + (int)n_neg;
    uint64_t key[32];
    key[0] = ts[t];
    key[1] = rel_base + tr[t];
    key[2] = to[t];
    bool bad = key[0] >= rel_base || key[2] >= rel_base || key[1] >= K;
    for (int q = 0; q < (int)n_neg; ++q) {
        key[3 + q] = neg_ent[t * n_neg + q];
        bad |= key[3 + q] >= rel_base;
    }
    if (bad) latch_error(st, epoch, PS_ERR_KEY_RANGE);
    uint32_t* kout = keys_out + t * n_slots;
    for (int u = 0; u < n_slots; ++u) {
        bool first = true;
        for (int z = 0; z < u; ++z) first &= key[z] != key[u];
        kout[u] = (first && !bad) ? (uint32_t)key[u] : (uint32_t)K;
    }
}

uint32_t launch_step_kge(ps_store* ps, const uint32_t* d_s, const uint32_t* d_r, const uint32_t* d_o,
                         const uint32_t* d_neg_ent, const uint8_t* d_neg_side, uint64_t n, uint32_t n_neg,
                         uint64_t rel_key_base, uint32_t dim, float lr, float eps, bool grad_only, cudaStream_t s) {
    const uint32_t grid = step_grid(ps, n);
#define KGE_ARGS d_s, d_r, d_o, d_neg_ent, d_neg_side, n, n_neg, rel_key_base, dim, lr, eps,                     \
                 (const float*)ps->store, ps->table, ps->cfg.slots_per_part, ps->cfg.num_keys, ps->upd,         \
                 ps->loss_partial, ps->status, ps->epoch
#define KGE_LAUNCH(kMaxNeg, kDim, kExact, kGrad)                                                                 \
    do {                                                                                                         \
        if (ps->prof) prof_before(ps, "kge_step_kernel<" #kMaxNeg ">", s);                                       \
        kge_step_kernel<kMaxNeg, kDim, kExact, kGrad><<<grid, 256, 0, s>>>(KGE_ARGS);                            \
        if (ps->prof) prof_after(ps, s);                                                                         \
        ps->launches++;                                                                                          \
    } while (0)
    if (grad_only) {
        if (n_neg == 10 && dim == 100) KGE_LAUNCH(10, 100, true, true);
        else if (n_neg <= 4) KGE_LAUNCH(4, 0, false, true);
        else if (n_neg <= 10) KGE_LAUNCH(10, 0, false, true);
        else KGE_LAUNCH(29, 0, false, true);
    } else {
        if (n_neg <= 4) KGE_LAUNCH(4, 0, false, false);
        else if (n_neg <= 10) KGE_LAUNCH(10, 0, false, false);
        else KGE_LAUNCH(29, 0, false, false);
    }
#undef KGE_LAUNCH
#undef KGE_ARGS
    return grid;
}

void launch_keys_kge(ps_store* ps, const uint32_t* d_s, const uint32_t* d_r, const uint32_t* d_o,
                     const uint32_t* d_neg_ent, uint64_t n, uint32_t n_neg, uint64_t rel_key_base, cudaStream_t s) {
    PS_LAUNCH(ps, kge_keys_kernel, div_up_u32(n, 256), 256, s, d_s, d_r, d_o, d_neg_ent, n, n_neg, rel_key_base,
              ps->cfg.num_keys, ps->keysA, ps->status, ps->epoch);
}

// ---------------------------------------------------------------- SGNS ----
// number of (center, context) pairs of all centers before position p
__device__ __forceinline__ uint64_t sgns_pairs_before(uint64_t p, uint64_t T, uint64_t W) {
    // left contexts: sum over q < p of min(q, W)
    const uint64_t m = p < W ? p : W;
    const uint64_t left = m * (m - (m > 0)) / 2 + (p - m) * W;
    // right contexts: sum over q < p of min(T - 1 - q, W)
    const uint64_t full = T > W ? (p < T - W ? p : T - W) : 0;
    const uint64_t rest = p - full;
    const uint64_t first = T - 1 - full;                    // value at q = full (only used if rest > 0)
    const uint64_t right = full * W + (rest ? rest * first - rest * (rest - 1) / 2 : 0);
    return left + right;
}

// Occurrence slots of center number c of the batch: slot_base = c * (1 + 2W(1 + n_neg));
// slot_base = the center's input vector; then per context j (ascending position) 1 + n_neg output vectors.
// The update of an output vector is a multiple of the center's input vector, the same vector for all of
// the center's slots, so it is not written out per slot: the kernel writes, per center, two source rows
// (2c: the summed update of the input vector; 2c + 1: a copy of the input vector as it was before the
// batch) and one factor per slot (1 for slot 0); the reduction multiplies as it adds.
// A warp takes one center at a time.  The output-vector slots are handled 32 at a time: every lane first
// resolves one slot (word -> key -> table entry -> row address), so those lookups are in flight together;
// the rows are then read four slots at a time, all loads of the four before the first dot product.
// kL4, kWindow, kNeg: row length (float4), window and negatives per context if known at compile time (0: taken
// from the arguments; kNeg < 0: from the argument); divisions by the slots per context and row offsets then fold.
template <int kCh, int kL4, int kWindow, int kNeg>
__global__ void __launch_bounds__(256, 2)
sgns_step_kernel(const uint32_t* __restrict__ tokens, uint64_t tok_first, uint64_t first_pos, uint64_t n_centers,
                 uint64_t T, uint32_t window_arg, const uint32_t* __restrict__ negs, uint32_t n_neg_arg, uint64_t out_base,
                 float lr, const float4* __restrict__ store, const uint2* __restrict__ table, uint64_t S, uint64_t K,
                 uint32_t L4_arg, float4* __restrict__ upd, float* __restrict__ scales, double* __restrict__ loss_partial,
                 DevStatus* st, unsigned int epoch) {
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t n_warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    const uint32_t L4 = kL4 ? (uint32_t)kL4 : L4_arg;
    const uint32_t window = kWindow ? (uint32_t)kWindow : window_arg;
    const uint32_t n_neg = kNeg >= 0 ? (uint32_t)kNeg : n_neg_arg;
    const uint32_t per_ctx = 1 + n_neg;
    const uint64_t slots = 1 + (uint64_t)2 * window * per_ctx;
    const uint64_t pairs0 = sgns_pairs_before(first_pos, T, window);
    constexpr int kQuad = 4;
    double loss = 0;
    for (uint64_t cidx = warp; cidx < n_centers; cidx += n_warps) {
        const uint64_t p = first_pos + cidx;
        const uint64_t lo = p >= window ? p - window : 0;
        const uint64_t hi = p + window < T ? p + window : T - 1;
        const uint64_t z0 = sgns_pairs_before(p, T, window) - pairs0;
        const uint32_t n_left = (uint32_t)(p - lo);
        const uint32_t n_out = (uint32_t)(hi - lo) * per_ctx;   // contexts (the center itself excluded) x (1 + n_neg)
        float4* U = upd + cidx * 2 * L4;
        float* F = scales + cidx * slots;
        const uint32_t wtok = tokens[p - tok_first];
        if (wtok >= out_base) {
            if (lane == 0) latch_error(st, epoch, PS_ERR_KEY_RANGE);
            continue;
        }
        const float4* V = store + phys_row(table[wtok], S) * L4;
        float4 v[kCh], dv[kCh];
#pragma unroll
        for (int c = 0; c < kCh; ++c) {
            const uint32_t f = lane + 32 * c;
            v[c] = f < L4 ? V[f] : make_float4(0.f, 0.f, 0.f, 0.f);
            dv[c] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        float loss_c = 0.f;
        bool bad = false;
        for (uint32_t t0 = 0; t0 < n_out; t0 += 32) {
            // this lane's slot of the round
            const uint32_t t = t0 + lane;
            uint64_t my_row = 0;
            bool my_ok = false;
            if (t < n_out) {
                const uint32_t j = t / per_ctx, i = t - j * per_ctx;
                const uint64_t q = j < n_left ? lo + j : lo + j + 1;            // skip the center itself
                const uint32_t word = i == 0 ? tokens[q - tok_first] : negs[(z0 + j) * n_neg + (i - 1)];
                const uint64_t ku = out_base + word;
                if (ku < K) {
                    my_row = phys_row(table[ku], S);
                    my_ok = true;
                } else {
                    bad = true;
                }
            }
            const unsigned ok_mask = __ballot_sync(full, my_ok);
            const uint32_t in_round = tmin<uint32_t>(32u, n_out - t0);
            float my_scale = 0.f;                                               // factor of this lane's slot
            for (uint32_t b = 0; b < in_round; b += kQuad) {
                float4 u[kQuad][kCh];
                float x[kQuad];
#pragma unroll
                for (int a = 0; a < kQuad; ++a) {
                    const uint64_t r = __shfl_sync(full, my_row, (b + a) & 31);
                    const bool ok = (ok_mask >> (b + a)) & 1u;                  // b + a <= 31; bits past the round are 0
                    const float4* Urow = store + r * L4;
#pragma unroll
                    for (int c = 0; c < kCh; ++c) {
                        const uint32_t f = lane + 32 * c;
                        u[a][c] = (ok && f < L4) ? Urow[f] : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
#pragma unroll
                for (int a = 0; a < kQuad; ++a) {
                    x[a] = 0.f;
#pragma unroll
                    for (int c = 0; c < kCh; ++c)
                        x[a] += v[c].x * u[a][c].x + v[c].y * u[a][c].y + v[c].z * u[a][c].z + v[c].w * u[a][c].w;
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                    for (int a = 0; a < kQuad; ++a) x[a] += __shfl_xor_sync(full, x[a], o);
                }
                // lane a < 4 turns the a-th score of the four into the slot's factor and loss term
                float xa = x[0];
#pragma unroll
                for (int a = 1; a < kQuad; ++a) xa = lane == a ? x[a] : xa;
                float sc_mine = 0.f;
                if (lane < kQuad && ((ok_mask >> (b + lane)) & 1u)) {
                    const bool positive = (t0 + b + lane) % per_ctx == 0;
                    sc_mine = -lr * (sigmoidf(xa) - (positive ? 1.f : 0.f));
                    loss_c += positive ? softplusf(-xa) : softplusf(xa);
                }
#pragma unroll
                for (int a = 0; a < kQuad; ++a) {
                    const float sc = __shfl_sync(full, sc_mine, a);
                    if (!((ok_mask >> (b + a)) & 1u)) continue;
                    if (lane == (int)(b + a)) my_scale = sc;
#pragma unroll
                    for (int c = 0; c < kCh; ++c) {
                        dv[c].x += sc * u[a][c].x; dv[c].y += sc * u[a][c].y;
                        dv[c].z += sc * u[a][c].z; dv[c].w += sc * u[a][c].w;
                    }
                }
            }
            if (my_ok) F[1 + t] = my_scale;
        }
        if (__any_sync(full, bad) && lane == 0) latch_error(st, epoch, PS_ERR_KEY_RANGE);
#pragma unroll
        for (int c = 0; c < kCh; ++c) {
            const uint32_t f = lane + 32 * c;
            if (f < L4) {
                U[f] = dv[c];
                U[L4 + f] = v[c];
            }
        }
        if (lane == 0) F[0] = 1.f;
        loss += (double)loss_c;                             // this lane's share (lanes 0..3 hold the terms)
    }
    block_loss_out(warp_sum_d(loss), loss_partial);
}

// Keys of the occurrence slots of each center: slot 0 the center's input vector, then per context
// 1 + n_neg output vectors; slots of contexts cut off at the stream's ends get the "no key" mark K.
__global__ void __launch_bounds__(256)
sgns_keys_kernel(const uint32_t* __restrict__ tokens, uint64_t tok_first, uint64_t first_pos, uint64_t n_centers,
                 uint64_t T, uint32_t window, const uint32_t* __restrict__ negs, uint32_t n_neg, uint64_t out_base,
                 uint64_t K, uint32_t* __restrict__ keys_out, DevStatus* st, unsigned int epoch) {
    const uint32_t per_ctx = 1 + n_neg;
    const uint64_t slots = 1 + (uint64_t)2 * window * per_ctx;
    const uint64_t x = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= n_centers * slots) return;
    const uint64_t cidx = x / slots, slot = x % slots;
    const uint64_t p = first_pos + cidx;
    uint64_t key = K;
    bool bad = false;
    if (slot == 0) {
        const uint32_t w = tokens[p - tok_first];
        bad = w >= out_base;
        key = w;
    } else {
        const uint64_t lo = p >= window ? p - window : 0;
        const uint64_t hi = p + window < T ? p + window : T - 1;
        const uint64_t j = (slot - 1) / per_ctx, i = (slot - 1) % per_ctx;
        const uint64_t n_left = p - lo;
        const uint64_t q = j < n_left ? lo + j : lo + j + 1;        // skip the center itself
        if (q <= hi) {
            const uint64_t z = sgns_pairs_before(p, T, window) - sgns_pairs_before(first_pos, T, window) + j;
            const uint32_t word = i == 0 ? tokens[q - tok_first] : negs[z * n_neg + (i - 1)];
            key = out_base + word;
            bad = key >= K;
        }
    }
    if (bad) {
        latch_error(st, epoch, PS_ERR_KEY_RANGE);
        key = K;
    }
    keys_out[x] = (uint32_t)key;
}

// the per-slot factors follow the 2 n_centers source rows in the update buffer
float* sgns_scales(ps_store* ps, uint64_t n_centers) { return ps->upd + n_centers * 2 * ps->cfg.row_len; }

uint32_t launch_step_sgns(ps_store* ps, const uint32_t* d_tokens, uint64_t tok_first, uint64_t first_pos,
                          uint64_t n_centers, uint64_t corpus_len, uint32_t window, const uint32_t* d_negs,
                          uint32_t n_neg, uint64_t out_key_base, float lr, cudaStream_t s) {
    const uint32_t L4 = ps->cfg.row_len / 4;
    const uint32_t grid = step_grid(ps, n_centers, 2);      // the kernels are bounded to two blocks per SM
#define SG_ARGS d_tokens, tok_first, first_pos, n_centers, corpus_len, window, d_negs, n_neg, out_key_base, lr,   \
                (const float4*)ps->store, ps->table, ps->cfg.slots_per_part, ps->cfg.num_keys, L4,              \
                (float4*)ps->upd, sgns_scales(ps, n_centers), ps->loss_partial, ps->status, ps->epoch
#define SG_LAUNCH(kCh, kL4, kW, kN)                                                                                  \
    do {                                                                                                             \
        if (ps->prof) prof_before(ps, "sgns_step_kernel<" #kCh ">", s);                                              \
        sgns_step_kernel<kCh, kL4, kW, kN><<<grid, 256, 0, s>>>(SG_ARGS);                                            \
        if (ps->prof) prof_after(ps, s);                                                                             \
        ps->launches++;                                                                                              \
    } while (0)
    if (L4 == 75 && window == 5 && n_neg == 3) SG_LAUNCH(3, 75, 5, 3);     // 300 values, window 5, 3 negatives
    else if (L4 <= 32) SG_LAUNCH(1, 0, 0, -1);
    else if (L4 <= 64) SG_LAUNCH(2, 0, 0, -1);
    else if (L4 <= 96) SG_LAUNCH(3, 0, 0, -1);
    else SG_LAUNCH(4, 0, 0, -1);
#undef SG_LAUNCH
#undef SG_ARGS
    return grid;
}

void launch_keys_sgns(ps_store* ps, const uint32_t* d_tokens, uint64_t tok_first, uint64_t first_pos,
                      uint64_t n_centers, uint64_t corpus_len, uint32_t window, const uint32_t* d_negs, uint32_t n_neg,
                      uint64_t out_key_base, cudaStream_t s) {
    const uint64_t total = n_centers * (1 + (uint64_t)2 * window * (1 + n_neg));
    PS_LAUNCH(ps, sgns_keys_kernel, div_up_u32(total, 256), 256, s, d_tokens, tok_first, first_pos, n_centers,
              corpus_len, window, d_negs, n_neg, out_key_base, ps->cfg.num_keys, ps->keysA, ps->status, ps->epoch);
}

}  // namespace psb
