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
// One block works on one data point at a time: R in shared memory (fp32, odd row stride), the vectors in fp64.  It
// writes, per occurrence slot (2 + n_neg entity slots, then d matrix rows), the gradient row of d values; the
// ComplEx path's reduction (kge_reduce_kernel: AdaGrad inside the segmented reduction of gradient rows) does the rest,
// a row of [d | d] values being to it what [Re Im | G_Re G_Im] of d / 2 complex dimensions is.
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

// shared memory of a block: R (d rows of d + 1 floats), then fp64: the entity slots' vectors, their gradients,
// u, w, a, b, b'
__host__ __device__ inline size_t rescal_smem(uint32_t d, uint32_t n_neg) {
    const size_t r = ((size_t)d * (d + 1) * sizeof(float) + 15) & ~(size_t)15;
    return r + ((size_t)2 * (2 + n_neg) + 5) * d * sizeof(double);
}

__global__ void __launch_bounds__(kRescalThreads)
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
    __shared__ int s_bad;
    const uint32_t L = 2 * d, ld = d + 1;
    const uint32_t n_ent = 2 + n_neg, n_slots = n_ent + d;
    float* Rm = reinterpret_cast<float*>(smem_raw);
    double* X = reinterpret_cast<double*>(smem_raw + (((size_t)d * ld * sizeof(float) + 15) & ~(size_t)15));   // [n_ent][d]
    double* Gs = X + (size_t)n_ent * d;                     // [n_ent][d]: gradient per entity slot
    double* U = Gs + (size_t)n_ent * d;
    double* Wv = U + d;
    double* A = Wv + d;
    double* B = A + d;
    double* Bp = B + d;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    double loss = 0;                                        // thread 0's
    for (uint64_t t = blockIdx.x; t < n; t += gridDim.x) {
        __syncthreads();                                    // the data point before is written out
        if (tid < (int)n_ent) {
            const uint32_t k = tid == 0 ? ts[t] : (tid == 1 ? to[t] : neg_ent[t * n_neg + (tid - 2)]);
            s_key[tid] = k;
        }
        if (tid == 0) s_bad = 0;
        __syncthreads();
        const uint64_t rk = rel_base + (uint64_t)tr[t] * d; // key of row 0 of the matrix
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
        // the matrix: row a from the store row of key rk + a (one warp per row, in turn)
        for (uint32_t a = warp; a < d; a += kRescalThreads / 32) {
            const float* src = store + phys_row(table[rk + a], S) * L;
            for (uint32_t b2 = lane; b2 < d; b2 += 32) Rm[a * ld + b2] = src[b2];
        }
        __syncthreads();
        for (uint32_t i = tid; i < n_ent * d; i += kRescalThreads) {
            const uint32_t u = i / d, c = i - u * d;
            X[i] = (double)store[s_row[u] * L + c];
        }
        __syncthreads();
        const double* xs = X;                               // slot 0: subject, slot 1: object
        const double* xo = X + d;
        // u = R x_o (thread per row), w = R^T x_s (thread per column)
        for (uint32_t i = tid; i < 2 * d; i += kRescalThreads) {
            double acc = 0;
            if (i < d) {
                for (uint32_t b2 = 0; b2 < d; ++b2) acc += (double)Rm[i * ld + b2] * xo[b2];
                U[i] = acc;
            } else {
                const uint32_t b2 = i - d;
                for (uint32_t a = 0; a < d; ++a) acc += xs[a] * (double)Rm[a * ld + b2];
                Wv[b2] = acc;
            }
        }
        __syncthreads();
        // scores, one warp per triple of the data point (q = 0: the positive)
        for (uint32_t q = warp; q <= n_neg; q += kRescalThreads / 32) {
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
                // (the loss terms are added by thread 0 below, in the order of the triples)
                Gs[q] = rescal_softplus(-y * p);            // parked in the gradient area, which is written after the sync
            }
        }
        __syncthreads();
        if (tid == 0)
            for (uint32_t q = 0; q <= n_neg; ++q) loss += Gs[q];
        __syncthreads();
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
        // gradients per entity slot: subject R b, object R^T a, negatives c_k u or c_k w
        for (uint32_t i = tid; i < n_ent * d; i += kRescalThreads) {
            const uint32_t u = i / d, c = i - u * d;
            double g;
            if (u == 0) {
                g = 0;
                for (uint32_t b2 = 0; b2 < d; ++b2) g += (double)Rm[c * ld + b2] * B[b2];
            } else if (u == 1) {
                g = 0;
                for (uint32_t a = 0; a < d; ++a) g += A[a] * (double)Rm[a * ld + c];
            } else {
                g = s_coef[u - 1] * (neg_side[t * n_neg + u - 2] == 0 ? U[c] : Wv[c]);
            }
            Gs[i] = g;
        }
        __syncthreads();
        // entity gradient rows: slots with the same key folded into the first, in slot order
        float* out = grad + (uint64_t)t * n_slots * d;
        for (uint32_t i = tid; i < n_ent * d; i += kRescalThreads) {
            const uint32_t u = i / d, c = i - u * d;
            if (s_rep[u] != (int)u) continue;
            double g = Gs[i];
            for (uint32_t z = u + 1; z < n_ent; ++z)
                if (s_rep[z] == (int)u) g += Gs[(size_t)z * d + c];
            out[i] = (float)g;
        }
        // matrix rows: a[alpha] x_o + x_s[alpha] b'
        float* outR = out + (uint64_t)n_ent * d;
        for (uint32_t i = tid; i < d * d; i += kRescalThreads) {
            const uint32_t al = i / d, be = i - al * d;
            outR[i] = (float)(A[al] * xo[be] + xs[al] * Bp[be]);
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
    static std::atomic<unsigned long long> smem_set{0};
    const size_t smem = rescal_smem(dim, n_neg);
    opt_in_smem((const void*)rescal_grad_kernel, rescal_smem(128, kRescalMaxNeg), &smem_set);
    // as many blocks as the device holds at this size (shared memory decides), at most one per data point
    const uint32_t per_sm = (uint32_t)tmax<size_t>(1, tmin<size_t>(8, (size_t)(220 * 1024) / (smem + 2048)));
    uint64_t g = tmin<uint64_t>(n, (uint64_t)ps->sm_count * per_sm);
    if (g > kMaxLossBlocks) g = kMaxLossBlocks;
    const uint32_t grid = (uint32_t)g;
    if (ps->prof) prof_before(ps, "rescal_grad_kernel", s);
    rescal_grad_kernel<<<grid, kRescalThreads, smem, s>>>(d_s, d_r, d_o, d_neg_ent, d_neg_side, n, n_neg, rel_key_base,
                                                         dim, (const float*)ps->store, ps->table,
                                                         ps->cfg.slots_per_part, ps->cfg.num_keys, (float*)ps->upd,
                                                         ps->loss_partial);
    if (ps->prof) prof_after(ps, s);
    ps->launches++;
    return grid;
}

}  // namespace psb
