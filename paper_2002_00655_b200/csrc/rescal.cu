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
// One WARP works on one data point at a time, with no block-wide synchronisation (a block of eight warps per data
// point, the matrix in shared memory or in registers, spent its time in a dozen dependent phases: 660-700 us per
// step of 8,192 data points).  Lane l holds elements l, l + 32, l + 64, l + 96 of every vector, in fp64.  A pass over
// the matrix goes row by row, coalesced (a lane reads its columns of the row, the loads of eight rows are issued
// before the first is used) and gives two products at once: the row's dot product with a vector (the lanes' shares go
// through a 32 x 33 tile of the warp and one lane adds a row's shares in lane order) and the product of the transpose
// with another vector (a lane accumulates its columns).  Two passes per data point.
// The gradient of an entity slot is c1 (R b) + c2 (R^T a) + c3 u + c4 w with four numbers per slot, so slots that
// hold the same entity are folded by adding their numbers, and no gradient is stored before it is final.  Written per
// occurrence slot (2 + n_neg entity slots, then d matrix rows): the gradient row of d values; the ComplEx path's
// reduction (kge_reduce_kernel: AdaGrad inside the segmented reduction of gradient rows) does the rest, a row of
// [d | d] values being to it what [Re Im | G_Re G_Im] of d / 2 complex dimensions is.
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
constexpr int kBatch = 8;             // matrix rows whose loads a warp has in flight together

// shared memory of a warp, fp64: x_s and a (read as broadcasts by the lanes), and a 32 x 33 tile
__host__ __device__ inline size_t rescal_smem(uint32_t d) {
    return (size_t)(kRescalThreads / 32) * (2 * d + 32 * 33) * sizeof(double);
}

// kE: elements of a vector per lane, d <= 32 kE
template <int kE>
__global__ void __launch_bounds__(kRescalThreads, 2)
rescal_grad_kernel(const uint32_t* __restrict__ ts, const uint32_t* __restrict__ tr, const uint32_t* __restrict__ to,
                   const uint32_t* __restrict__ neg_ent, const uint8_t* __restrict__ neg_side, uint64_t n,
                   uint32_t n_neg, uint64_t rel_base, uint32_t d, const float* __restrict__ store,
                   const uint2* __restrict__ table, uint64_t S, uint64_t K, float* __restrict__ grad,
                   double* __restrict__ loss_partial) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ double s_wl[kRescalThreads / 32];
    constexpr int kWarps = kRescalThreads / 32;
    const unsigned full = 0xffffffffu;
    const uint32_t L = 2 * d;
    const uint32_t n_ent = 2 + n_neg, n_slots = n_ent + d;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double* sxs = reinterpret_cast<double*>(smem_raw) + (size_t)warp * (2 * d + 32 * 33);
    double* sA = sxs + d;
    double* tile = sA + d;                                  // [32][33]
    const uint64_t n_warps = (uint64_t)gridDim.x * kWarps;
    double loss = 0;                                        // lane 0's
    for (uint64_t t = (uint64_t)blockIdx.x * kWarps + warp; t < n; t += n_warps) {
        // entity slots: subject, object, negatives (lane u holds slot u)
        uint32_t key = 0;
        if (lane < (int)n_ent) key = lane == 0 ? ts[t] : (lane == 1 ? to[t] : neg_ent[t * n_neg + (lane - 2)]);
        const uint32_t side = (lane >= 2 && lane < (int)n_ent) ? neg_side[t * n_neg + (lane - 2)] : 0u;
        const uint64_t rk = rel_base + (uint64_t)tr[t] * d; // key of row 0 of the matrix
        if (__ballot_sync(full, lane < (int)n_ent && key >= rel_base) != 0u || rk + d > K) continue;   // (latched by the key kernel)
        int rep = lane;                                     // first slot that holds the same key
        for (int z = 0; z < (int)n_ent; ++z) {
            const uint32_t kz = __shfl_sync(full, key, z);
            if (lane < (int)n_ent && kz == key && z < rep) rep = z;
        }
        uint64_t erow = 0;
        if (lane < (int)n_ent) erow = phys_row(table[key], S);
        // rows of the matrix this lane owns, and its elements of x_s and x_o
        const float* rowp[kE];
        double xs[kE], xo[kE];
        const float* ps_ = store + __shfl_sync(full, erow, 0) * L;
        const float* po_ = store + __shfl_sync(full, erow, 1) * L;
#pragma unroll
        for (int k = 0; k < kE; ++k) {
            const uint32_t e = lane + 32 * k;
            rowp[k] = store;
            xs[k] = xo[k] = 0;
            if (e < d) {
                rowp[k] = store + phys_row(table[rk + e], S) * L;
                xs[k] = (double)ps_[e];
                xo[k] = (double)po_[e];
            }
        }
        __syncwarp();                                       // the data point before is done with the warp's shared memory
#pragma unroll
        for (int k = 0; k < kE; ++k) {
            const uint32_t e = lane + 32 * k;
            if (e < d) sxs[e] = xs[k];
        }
        __syncwarp();
        // v = R y and z = R^T s in one pass over the matrix, row by row (coalesced: a lane reads its columns of the
        // row).  The lane's columns' share of the row's dot product with y goes to a 32 x 32 tile of the warp, and
        // after 32 rows lane j adds up row j's shares, in lane order.  y: the lanes' elements; s: in shared memory.
        auto products = [&](const double (&y)[kE], const double* ss, double (&v)[kE], double (&z)[kE]) {
#pragma unroll
            for (int k = 0; k < kE; ++k) v[k] = z[k] = 0;
#pragma unroll
            for (int kk = 0; kk < kE; ++kk) {
                const uint32_t a0 = 32u * kk;               // the rows a0 .. a0 + 31 are the lanes' rows number kk
                if (a0 >= d) break;
                const uint32_t cnt = d - a0 < 32u ? d - a0 : 32u;
                // kBatch rows at a time: all their loads are issued before the first is used
                for (uint32_t j0 = 0; j0 < cnt; j0 += kBatch) {
                    const float* ra[kBatch];
                    float r[kBatch][kE];
#pragma unroll
                    for (int i = 0; i < kBatch; ++i) {
                        const uint32_t j = j0 + i < cnt ? j0 + i : cnt - 1;
                        ra[i] = reinterpret_cast<const float*>(__shfl_sync(full, (unsigned long long)rowp[kk], j));
                    }
#pragma unroll
                    for (int i = 0; i < kBatch; ++i)
#pragma unroll
                        for (int k = 0; k < kE; ++k) r[i][k] = (uint32_t)(lane + 32 * k) < d ? __ldg(ra[i] + lane + 32 * k) : 0.f;
#pragma unroll
                    for (int i = 0; i < kBatch; ++i) {
                        if (j0 + i >= cnt) break;
                        const double sa = ss[a0 + j0 + i];
                        double p = 0;
#pragma unroll
                        for (int k = 0; k < kE; ++k) {
                            const double rv = (double)r[i][k];
                            z[k] += sa * rv;
                            p += rv * y[k];
                        }
                        tile[(j0 + i) * 33 + lane] = p;
                    }
                }
                __syncwarp();
                if ((uint32_t)lane < cnt) {
                    double acc = 0;
#pragma unroll 8
                    for (int l = 0; l < 32; ++l) acc += tile[lane * 33 + l];
                    v[kk] = acc;
                }
                __syncwarp();
            }
        };
        double u[kE], w[kE];
        products(xo, sxs, u, w);
        // scores: lane 1 keeps the positive's, lane 2 + q negative q's; then every lane forms its triple's coefficient
        // and loss term (the exponentials once per data point, not once per triple); then a and b'
        double phi_mine = 0;
        {
            double p = 0;
#pragma unroll
            for (int k = 0; k < kE; ++k) p += xs[k] * u[k];
            p = warp_sum_d(p);
            if (lane == 1) phi_mine = p;
        }
        for (uint32_t q = 0; q < n_neg; ++q) {
            const float* pk = store + __shfl_sync(full, erow, 2 + q) * L;
            const bool subj = __shfl_sync(full, side, 2 + q) == 0u;
            double p = 0;
#pragma unroll
            for (int k = 0; k < kE; ++k) {
                const uint32_t e = lane + 32 * k;
                if (e < d) p += (double)pk[e] * (subj ? u[k] : w[k]);
            }
            p = warp_sum_d(p);
            if (lane == (int)(2 + q)) phi_mine = p;
        }
        double my_coef = 0, my_loss = 0;                    // d loss / d phi and the loss term of this lane's triple
        if (lane >= 1 && lane < (int)n_ent) {
            const double y = lane == 1 ? 1.0 : -1.0;
            my_coef = -y * rescal_sigmoid(-y * phi_mine);
            my_loss = rescal_softplus(-y * phi_mine);
        }
        const double lsum = warp_sum_d(my_loss);
        const double c_pos = __shfl_sync(full, my_coef, 1);
        double av[kE], bp[kE];
#pragma unroll
        for (int k = 0; k < kE; ++k) { av[k] = c_pos * xs[k]; bp[k] = 0; }
        for (uint32_t q = 0; q < n_neg; ++q) {
            const float* pk = store + __shfl_sync(full, erow, 2 + q) * L;
            const bool subj = __shfl_sync(full, side, 2 + q) == 0u;
            const double cq = __shfl_sync(full, my_coef, 2 + q);
#pragma unroll
            for (int k = 0; k < kE; ++k) {
                const uint32_t e = lane + 32 * k;
                const double xk = e < d ? (double)pk[e] : 0.0;
                if (subj) av[k] += cq * xk;
                else bp[k] += cq * xk;
            }
        }
        if (lane == 0) loss += lsum;
        double bv[kE];
#pragma unroll
        for (int k = 0; k < kE; ++k) {
            const uint32_t e = lane + 32 * k;
            bv[k] = c_pos * xo[k] + bp[k];
            if (e < d) sA[e] = av[k];
        }
        __syncwarp();
        double gs[kE], go[kE];
        products(bv, sA, gs, go);                           // R b, R^T a
        // the four numbers of every slot, folded into the first slot of its key (lane v: the numbers of slot v)
        double c1 = 0, c2 = 0, c3 = 0, c4 = 0;
        for (int z = 0; z < (int)n_ent; ++z) {
            const int rz = __shfl_sync(full, rep, z);
            const double cz = __shfl_sync(full, my_coef, z);
            const uint32_t sz = __shfl_sync(full, side, z);
            if (rz != lane) continue;
            if (z == 0) c1 += 1.0;
            else if (z == 1) c2 += 1.0;
            else if (sz == 0u) c3 += cz;
            else c4 += cz;
        }
        float* out = grad + (uint64_t)t * n_slots * d;
        for (int v = 0; v < (int)n_ent; ++v) {
            if (__shfl_sync(full, rep, v) != v) continue;   // a later slot of a key: marked "no key", never read
            const double f1 = __shfl_sync(full, c1, v), f2 = __shfl_sync(full, c2, v);
            const double f3 = __shfl_sync(full, c3, v), f4 = __shfl_sync(full, c4, v);
#pragma unroll
            for (int k = 0; k < kE; ++k) {
                const uint32_t e = lane + 32 * k;
                if (e < d) out[(size_t)v * d + e] = (float)(f1 * gs[k] + f2 * go[k] + f3 * u[k] + f4 * w[k]);
            }
        }
        // matrix rows: a[alpha] x_o + x_s[alpha] b', written as float4: x_o and b' go through the tile so that a lane
        // holds four consecutive columns
        float* outR = out + (uint64_t)n_ent * d;
        __syncwarp();
#pragma unroll
        for (int k = 0; k < kE; ++k) {
            const uint32_t e = lane + 32 * k;
            if (e < d) { tile[e] = xo[k]; tile[d + e] = bp[k]; }
        }
        __syncwarp();
        if ((uint32_t)lane < d / 4) {
            const double o0 = tile[4 * lane], o1 = tile[4 * lane + 1], o2 = tile[4 * lane + 2], o3 = tile[4 * lane + 3];
            const double b0 = tile[d + 4 * lane], b1 = tile[d + 4 * lane + 1], b2 = tile[d + 4 * lane + 2], b3 = tile[d + 4 * lane + 3];
#pragma unroll 4
            for (uint32_t al = 0; al < d; ++al) {
                const double aa = sA[al], sa = sxs[al];
                float4 g;
                g.x = (float)(aa * o0 + sa * b0);
                g.y = (float)(aa * o1 + sa * b1);
                g.z = (float)(aa * o2 + sa * b2);
                g.w = (float)(aa * o3 + sa * b3);
                *reinterpret_cast<float4*>(outR + (size_t)al * d + 4 * lane) = g;
            }
        }
    }
    if (lane == 0) s_wl[warp] = loss;
    __syncthreads();
    if (threadIdx.x == 0) {
        double tot = 0;
        for (int i = 0; i < kWarps; ++i) tot += s_wl[i];
        loss_partial[blockIdx.x] = tot;
    }
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
    const size_t smem = rescal_smem(dim);
    (void)n_neg;
    // two blocks per SM, a warp per data point at a time
    uint64_t g = tmin<uint64_t>((n + 7) / 8, (uint64_t)ps->sm_count * 2);
    if (g > kMaxLossBlocks) g = kMaxLossBlocks;
    const uint32_t grid = (uint32_t)g;
#define RESCAL_LAUNCH(kE)                                                                                           \
    do {                                                                                                            \
        static std::atomic<unsigned long long> smem_set{0};                                                         \
        opt_in_smem((const void*)rescal_grad_kernel<kE>, rescal_smem(128), &smem_set);                              \
        if (ps->prof) prof_before(ps, "rescal_grad_kernel<" #kE ">", s);                                            \
        rescal_grad_kernel<kE><<<grid, kRescalThreads, smem, s>>>(                                                  \
            d_s, d_r, d_o, d_neg_ent, d_neg_side, n, n_neg, rel_key_base, dim, (const float*)ps->store, ps->table,  \
            ps->cfg.slots_per_part, ps->cfg.num_keys, (float*)ps->upd, ps->loss_partial);                          \
    } while (0)
    if (dim <= 32) RESCAL_LAUNCH(1);
    else if (dim <= 64) RESCAL_LAUNCH(2);
    else RESCAL_LAUNCH(4);
#undef RESCAL_LAUNCH
    if (ps->prof) prof_after(ps, s);
    ps->launches++;
    return grid;
}

}  // namespace psb
