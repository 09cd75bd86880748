// RESCAL (Section 4.1 of the paper names the model; Table 4: entity dimension d, relation dimension d * d): the
// gradient kernel of one minibatch.  Rows of the store have one length, so a relation's d x d matrix is d keys, one
// per matrix row:  key e < rel_base: entity e, row [x | G];  key rel_base + r d + a: row a of R_r, row [R_r[a][.] | G]
// (G: element-wise AdaGrad accumulators, row_len = 2 d).  Score  phi(s, r, o) = x_s^T R_r x_o.
//
// A data point is a positive triple and its negatives (each replaces the subject or the object).  With c_q the
// derivative of softplus(-y phi_q) with respect to phi_q, the gradients of the data point's loss factor through four
// matrix-vector products of the one matrix R = R_r:
//   u = R x_o,  w = R^T x_s                 phi_pos = x_s . u,  phi of a subject-negative k = x_k . u,  of an
//                                           object-negative k = w . x_k
//   a = c_pos x_s + sum over subject-negatives c_k x_k,   b' = sum over object-negatives c_k x_k,  b = c_pos x_o + b'
//   subject slot: R b      object slot: R^T a      subject-negative k: c_k u      object-negative k: c_k w
//   matrix row alpha:  a[alpha] x_o + x_s[alpha] b'
// Slots that hold the same entity are folded into the first of them before anything is written (AdaGrad is taken on
// the gradient with respect to each DISTINCT key), as the key kernel marks the later ones "no key".
//
// One block of eight warps works on one data point at a time.  Warp w owns the matrix rows w, w + 8, ...: it loads
// them once (a lane holds four consecutive values of each of its rows) and uses them from registers for all four
// matrix-vector products: a row's dot product with a vector is summed over the lanes by shuffles, its contribution to
// a product with the transpose is kept per lane and the eight warps' parts are added in warp order.  The vectors live
// in shared memory in fp64.  Written per occurrence slot (2 + n_neg entity slots, then d matrix rows): the gradient
// row of d values; the ComplEx path's reduction (kge_reduce_kernel: AdaGrad inside the segmented reduction of gradient
// rows) does the rest, a row of [d | d] values being to it what [Re Im | G_Re G_Im] of d / 2 complex dimensions is.
#include "ps_internal.cuh"

namespace psb {

__device__ __forceinline__ double rescal_softplus(double z) { return fmax(z, 0.0) + log1p(exp(-fabs(z))); }
__device__ __forceinline__ double rescal_sigmoid(double z) {
    if (z >= 0.0) return 1.0 / (1.0 + exp(-z));
    const double e = exp(z);
    return e / (1.0 + e);
}

constexpr int kRescalThreads = 256;
constexpr int kRescalMaxNeg = 29;

// shared memory of a block, fp64: the entity slots' vectors, their gradients, u, w, a, b, b', and the warps' parts of
// a product with the transpose
__host__ __device__ inline size_t rescal_smem(uint32_t d, uint32_t n_neg) {
    return ((size_t)2 * (2 + n_neg) + 5 + kRescalThreads / 32) * d * sizeof(double);
}

struct d4r {
    double x, y, z, w;
};

// kRows: matrix rows per warp, at least d / 8 rounded up
template <int kRows>
__global__ void __launch_bounds__(kRescalThreads, 2)
rescal_grad_kernel(const uint32_t* __restrict__ ts, const uint32_t* __restrict__ tr, const uint32_t* __restrict__ to,
                   const uint32_t* __restrict__ neg_ent, const uint8_t* __restrict__ neg_side, uint64_t n,
                   uint32_t n_neg, uint64_t rel_base, uint32_t d, const float* __restrict__ store,
                   const uint2* __restrict__ table, uint64_t S, uint64_t K, float* __restrict__ grad,
                   double* __restrict__ loss_partial) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ uint64_t s_row[2 + kRescalMaxNeg];           // store row of each entity slot
    __shared__ uint32_t s_key[2 + kRescalMaxNeg];
    __shared__ int s_rep[2 + kRescalMaxNeg];                // first slot that holds the same key
    __shared__ double s_coef[1 + kRescalMaxNeg];
    __shared__ double s_loss[1 + kRescalMaxNeg];
    __shared__ int s_bad;
    constexpr int kWarps = kRescalThreads / 32;
    const unsigned full = 0xffffffffu;
    const uint32_t L = 2 * d, d4 = d / 4;
    const uint32_t n_ent = 2 + n_neg, n_slots = n_ent + d;
    double* X = reinterpret_cast<double*>(smem_raw);        // [n_ent][d]
    double* Gs = X + (size_t)n_ent * d;                     // [n_ent][d]: gradient per entity slot
    double* U = Gs + (size_t)n_ent * d;
    double* Wv = U + d;
    double* A = Wv + d;
    double* B = A + d;
    double* Bp = B + d;
    double* Wp = Bp + d;                                    // [kWarps][d]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool col = (uint32_t)lane < d4;                   // this lane holds columns 4 lane .. 4 lane + 3
    double loss = 0;                                        // thread 0's
    // One pass over the warp's rows: dot[a] = row a . v (to out_dot) and this warp's part of sum_a s[a] row a (to Wp).
    auto products = [&](const float4 (&R)[kRows], const double* v, const double* sc, double* out_dot) {
        d4r vv = {0, 0, 0, 0}, part = {0, 0, 0, 0};
        if (col) vv = d4r{v[4 * lane], v[4 * lane + 1], v[4 * lane + 2], v[4 * lane + 3]};
#pragma unroll
        for (int j = 0; j < kRows; ++j) {
            const uint32_t a = warp + kWarps * j;
            if (a >= d) break;                              // (the same for the whole warp)
            const double rx = R[j].x, ry = R[j].y, rz = R[j].z, rw = R[j].w;
            double p = rx * vv.x + ry * vv.y + rz * vv.z + rw * vv.w;
            p = warp_sum_d(p);
            if (lane == 0) out_dot[a] = p;
            const double sa = sc[a];
            part.x += sa * rx; part.y += sa * ry; part.z += sa * rz; part.w += sa * rw;
        }
        if (col) {
            double* wp = Wp + (size_t)warp * d + 4 * lane;
            wp[0] = part.x; wp[1] = part.y; wp[2] = part.z; wp[3] = part.w;
        }
    };
    for (uint64_t t = blockIdx.x; t < n; t += gridDim.x) {
        __syncthreads();                                    // the data point before is written out
        if (tid < (int)n_ent) {
            const uint32_t k = tid == 0 ? ts[t] : (tid == 1 ? to[t] : neg_ent[t * n_neg + (tid - 2)]);
            s_key[tid] = k;
        }
        if (tid == 0) s_bad = 0;
        const uint64_t rk = rel_base + (uint64_t)tr[t] * d; // key of row 0 of the matrix
        // the warp's rows of the matrix: their table entries now, the rows below (zeros beyond the last column)
        uint64_t my_rrow = 0;
        if (lane < kRows && warp + kWarps * lane < d && rk + d <= K) my_rrow = phys_row(table[rk + warp + kWarps * lane], S);
        __syncthreads();
        if (tid < (int)n_ent) {
            if (s_key[tid] >= rel_base) s_bad = 1;
            int rep = tid;
            for (int z = tid - 1; z >= 0; --z)
                if (s_key[z] == s_key[tid]) rep = z;
            s_rep[tid] = rep;
        }
        if (tid == 0 && rk + d > K) s_bad = 1;
        __syncthreads();
        if (s_bad) continue;                                // the key kernel has latched the error; nothing is written
        if (tid < (int)n_ent) s_row[tid] = phys_row(table[s_key[tid]], S);
        float4 R[kRows];
#pragma unroll
        for (int j = 0; j < kRows; ++j) {
            const uint64_t rr = __shfl_sync(full, my_rrow, j);
            R[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (warp + kWarps * j < d && col) R[j] = *reinterpret_cast<const float4*>(store + rr * L + 4 * lane);
        }
        __syncthreads();
        for (uint32_t u = warp; u < n_ent; u += kWarps)
            for (uint32_t c = lane; c < d; c += 32) X[(size_t)u * d + c] = (double)store[s_row[u] * L + c];
        __syncthreads();
        const double* xs = X;                               // slot 0: subject, slot 1: object
        const double* xo = X + d;
        // u = R x_o and the parts of w = R^T x_s
        products(R, xo, xs, U);
        __syncthreads();
        for (uint32_t c = tid; c < d; c += kRescalThreads) {
            double acc = Wp[c];
            for (int w2 = 1; w2 < kWarps; ++w2) acc += Wp[(size_t)w2 * d + c];
            Wv[c] = acc;
        }
        __syncthreads();
        // scores, one warp per triple of the data point (q = 0: the positive)
        for (uint32_t q = warp; q <= n_neg; q += kWarps) {
            const double* lhs = xs;
            const double* rhs = U;                          // x . u: the positive and the subject-negatives
            if (q > 0) {
                if (neg_side[t * n_neg + q - 1] == 0) lhs = X + (size_t)(2 + q - 1) * d;
                else { lhs = Wv; rhs = X + (size_t)(2 + q - 1) * d; }
            }
            double p = 0;
            for (uint32_t c = lane; c < d; c += 32) p += lhs[c] * rhs[c];
            p = warp_sum_d(p);
            if (lane == 0) {
                const double y = q == 0 ? 1.0 : -1.0;
                s_coef[q] = -y * rescal_sigmoid(-y * p);
                s_loss[q] = rescal_softplus(-y * p);        // (added by thread 0 below, in the order of the triples)
            }
        }
        __syncthreads();
        if (tid == 0)
            for (uint32_t q = 0; q <= n_neg; ++q) loss += s_loss[q];
        // a, b', b
        for (uint32_t i = tid; i < 2 * d; i += kRescalThreads) {
            const bool is_a = i < d;
            const uint32_t c = is_a ? i : i - d;
            double acc = 0;
            for (uint32_t q = 1; q <= n_neg; ++q) {
                const bool subj = neg_side[t * n_neg + q - 1] == 0;
                if (subj == is_a) acc += s_coef[q] * X[(size_t)(2 + q - 1) * d + c];
            }
            if (is_a) A[c] = s_coef[0] * xs[c] + acc;
            else { Bp[c] = acc; B[c] = s_coef[0] * xo[c] + acc; }
        }
        __syncthreads();
        // gradients per entity slot: subject R b, the parts of the object's R^T a, negatives c_k u or c_k w
        products(R, B, A, Gs);
        for (uint32_t u = 2 + warp; u < n_ent; u += kWarps) {
            const double ck = s_coef[u - 1];
            const double* from = neg_side[t * n_neg + u - 2] == 0 ? U : Wv;
            for (uint32_t c = lane; c < d; c += 32) Gs[(size_t)u * d + c] = ck * from[c];
        }
        __syncthreads();
        for (uint32_t c = tid; c < d; c += kRescalThreads) {
            double acc = Wp[c];
            for (int w2 = 1; w2 < kWarps; ++w2) acc += Wp[(size_t)w2 * d + c];
            Gs[d + c] = acc;
        }
        __syncthreads();
        // entity gradient rows: slots with the same key folded into the first, in slot order
        float* out = grad + (uint64_t)t * n_slots * d;
        for (uint32_t u = warp; u < n_ent; u += kWarps) {
            if (s_rep[u] != (int)u) continue;
            for (uint32_t c = lane; c < d; c += 32) {
                double g = Gs[(size_t)u * d + c];
                for (uint32_t z = u + 1; z < n_ent; ++z)
                    if (s_rep[z] == (int)u) g += Gs[(size_t)z * d + c];
                out[(size_t)u * d + c] = (float)g;
            }
        }
        // matrix rows: a[alpha] x_o + x_s[alpha] b'
        float* outR = out + (uint64_t)n_ent * d;
        if (col) {
            const d4r o4 = {xo[4 * lane], xo[4 * lane + 1], xo[4 * lane + 2], xo[4 * lane + 3]};
            const d4r b4 = {Bp[4 * lane], Bp[4 * lane + 1], Bp[4 * lane + 2], Bp[4 * lane + 3]};
#pragma unroll
            for (int j = 0; j < kRows; ++j) {
                const uint32_t al = warp + kWarps * j;
                if (al >= d) break;
                const double aa = A[al], sa = xs[al];
                float4 g;
                g.x = (float)(aa * o4.x + sa * b4.x);
                g.y = (float)(aa * o4.y + sa * b4.y);
                g.z = (float)(aa * o4.z + sa * b4.z);
                g.w = (float)(aa * o4.w + sa * b4.w);
                *reinterpret_cast<float4*>(outR + (size_t)al * d + 4 * lane) = g;
            }
        }
    }
    if (tid == 0) loss_partial[blockIdx.x] = loss;
}

// Keys of the occurrence slots: 2 + n_neg entity slots (a slot that repeats an earlier slot's key gets the "no key"
// mark K), then the d rows of the relation's matrix; every slot of a data point with an index out of range gets K.
__global__ void __launch_bounds__(256)
rescal_keys_kernel(const uint32_t* __restrict__ ts, const uint32_t* __restrict__ tr, const uint32_t* __restrict__ to,
                   const uint32_t* __restrict__ neg_ent, uint64_t n, uint32_t n_neg, uint64_t rel_base, uint32_t d,
                   uint64_t K, uint32_t* __restrict__ keys_out, DevStatus* st, unsigned int epoch) {
    const uint64_t idx = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t n_ent = 2 + n_neg, n_slots = n_ent + d;
    if (idx >= n * n_slots) return;
    const uint64_t t = idx / n_slots;
    const uint32_t u = (uint32_t)(idx - t * n_slots);
    const uint64_t rk = rel_base + (uint64_t)tr[t] * d;
    bool bad = ts[t] >= rel_base || to[t] >= rel_base || rk + d > K;
    for (uint32_t q = 0; q < n_neg; ++q) bad |= neg_ent[t * n_neg + q] >= rel_base;
    if (bad) {
        if (u == 0) latch_error(st, epoch, PS_ERR_KEY_RANGE);
        keys_out[idx] = (uint32_t)K;
        return;
    }
    if (u >= n_ent) {
        keys_out[idx] = (uint32_t)(rk + (u - n_ent));
        return;
    }
    auto key_of = [&](uint32_t z) { return z == 0 ? ts[t] : (z == 1 ? to[t] : neg_ent[t * n_neg + (z - 2)]); };
    const uint32_t mine = key_of(u);
    bool first = true;
    for (uint32_t z = 0; z < u; ++z) first &= key_of(z) != mine;
    keys_out[idx] = first ? mine : (uint32_t)K;
}

void launch_keys_rescal(ps_store* ps, const uint32_t* d_s, const uint32_t* d_r, const uint32_t* d_o,
                        const uint32_t* d_neg_ent, uint64_t n, uint32_t n_neg, uint64_t rel_key_base, uint32_t dim,
                        cudaStream_t s) {
    const uint64_t occ = n * (2 + (uint64_t)n_neg + dim);
    PS_LAUNCH(ps, rescal_keys_kernel, div_up_u32(occ, 256), 256, s, d_s, d_r, d_o, d_neg_ent, n, n_neg, rel_key_base,
              dim, ps->cfg.num_keys, ps->keysA, ps->status, ps->epoch);
}

uint32_t launch_grad_rescal(ps_store* ps, const uint32_t* d_s, const uint32_t* d_r, const uint32_t* d_o,
                            const uint32_t* d_neg_ent, const uint8_t* d_neg_side, uint64_t n, uint32_t n_neg,
                            uint64_t rel_key_base, uint32_t dim, cudaStream_t s) {
    const size_t smem = rescal_smem(dim, n_neg);
    // two blocks per SM (registers: the warps hold the matrix), at most one block per data point
    uint64_t g = tmin<uint64_t>(n, (uint64_t)ps->sm_count * 2);
    if (g > kMaxLossBlocks) g = kMaxLossBlocks;
    const uint32_t grid = (uint32_t)g;
#define RESCAL_LAUNCH(kRows)                                                                                        \
    do {                                                                                                            \
        static std::atomic<unsigned long long> smem_set{0};                                                         \
        opt_in_smem((const void*)rescal_grad_kernel<kRows>, rescal_smem(128, kRescalMaxNeg), &smem_set);            \
        if (ps->prof) prof_before(ps, "rescal_grad_kernel<" #kRows ">", s);                                         \
        rescal_grad_kernel<kRows><<<grid, kRescalThreads, smem, s>>>(                                               \
            d_s, d_r, d_o, d_neg_ent, d_neg_side, n, n_neg, rel_key_base, dim, (const float*)ps->store, ps->table,  \
            ps->cfg.slots_per_part, ps->cfg.num_keys, (float*)ps->upd, ps->loss_partial);                          \
    } while (0)
    if (dim <= 32) RESCAL_LAUNCH(4);
    else if (dim <= 64) RESCAL_LAUNCH(8);
    else if (dim <= 104) RESCAL_LAUNCH(13);
    else RESCAL_LAUNCH(16);
#undef RESCAL_LAUNCH
    if (ps->prof) prof_after(ps, s);
    ps->launches++;
    return grid;
}

}  // namespace psb
