/*
 * CPU oracle for the parameter-server hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, sequential, deliberately slow C implementation of what the CUDA
 * library computes, written from the paper (Renz-Wieland et al., "Dynamic
 * Parameter Allocation in Parameter Servers", VLDB 2020).  It shares no code,
 * header or table with the CUDA path.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may load it; no product path may.
 *
 * State.  Parameter rows are stored BY KEY (row_len fp32 each), next to a
 * location table key -> (owner, slot) and one free-slot stack per partition.
 * Keeping the values by key makes pull/push oblivious of location by
 * construction, which is the property Section 2.3 demands of a PS with dynamic
 * allocation.
 *
 * Step semantics.  Inside one call every read sees the state from before the
 * call; all update terms of the call are summed per key (fp64, in occurrence
 * order) and added once:  row = (float)((double)row + sum).  This is the
 * cumulative push of Section 2.1 / Table 2 applied to a whole minibatch.
 * Gradient arithmetic is fp64 on the fp32 state.
 *
 * Pins (see tests/, "-m not gpu"): finite differences of the written-out loss
 * for every gradient, complex arithmetic for the ComplEx score, textbook SGD on
 * distinct keys, exact integer sums for push, a planted model whose loss must
 * fall, and an independent dictionary model for pull/push/localize.
 * Parity unpinned by the paper (the paper prints no formula or number for
 * them; they are this repository's stated readings): the free-slot policy of
 * localize, the 1/2 convention and per-occurrence L2 of the MF loss, AdaGrad's
 * eps and per-data-point application, the fixed skip-gram window, and for
 * RESCAL the layout of a relation's matrix as one key per matrix row (the score
 * itself is pinned against the bilinear form written with numpy).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { OPS_OK = 0, OPS_ERR_INVALID_ARG = 1, OPS_ERR_KEY_RANGE = 2, OPS_ERR_WORKER_RANGE = 3,
       OPS_ERR_CAPACITY = 4 };

typedef struct ops_store {
    uint64_t K;          /* number of keys, dense in [0, K) (dense store, Section 3.7) */
    uint32_t L;          /* fp32 values per key */
    uint32_t N;          /* logical workers = partitions */
    uint64_t S;          /* slots per partition */
    float *rows;         /* K x L, by key */
    uint32_t *owner;     /* K */
    uint32_t *slot;      /* K */
    uint32_t *stack;     /* N x S free-slot stacks, bottom at index 0 */
    uint64_t *top;       /* N stack heights */
    /* per-call accumulators */
    int32_t *acc_of;     /* K: index of the key's accumulator in this call, -1 if none */
    uint64_t *touched;   /* keys in first-touch order */
    uint64_t n_touched, cap_touched;
    double *acc;         /* cap_touched x L */
} ops_store;

ops_store *ops_create(uint64_t K, uint32_t L, uint32_t N, uint64_t S) {
    if (K == 0 || L == 0 || N == 0) return NULL;
    uint64_t B = (K + N - 1) / N;
    if (S < B || S > 0xFFFFFFFFull || K > 0xFFFFFFFFull) return NULL;
    ops_store *st = (ops_store *)calloc(1, sizeof(ops_store));
    if (!st) return NULL;
    st->K = K; st->L = L; st->N = N; st->S = S;
    st->rows = (float *)calloc(K * L, sizeof(float));
    st->owner = (uint32_t *)calloc(K, sizeof(uint32_t));
    st->slot = (uint32_t *)calloc(K, sizeof(uint32_t));
    st->stack = (uint32_t *)calloc((uint64_t)N * S, sizeof(uint32_t));
    st->top = (uint64_t *)calloc(N, sizeof(uint64_t));
    st->acc_of = (int32_t *)malloc(K * sizeof(int32_t));
    if (!st->rows || !st->owner || !st->slot || !st->stack || !st->top || !st->acc_of) return NULL;
    for (uint64_t k = 0; k < K; ++k) st->acc_of[k] = -1;
    return st;
}

void ops_destroy(ops_store *st) {
    if (!st) return;
    free(st->rows); free(st->owner); free(st->slot); free(st->stack); free(st->top);
    free(st->acc_of); free(st->touched); free(st->acc); free(st);
}

/* Initial static allocation by range partitioning (Section 3.5: a home node is
 * assigned "using range or hash partitioning"; classic PSs allocate the same
 * way, Section 2.1).  B = ceil(K/N); key k starts at owner k / B, slot k % B.
 * The free stack of partition p then holds S-1, S-2, ..., cnt_p (bottom to
 * top), so that the lowest free slot is popped first. */
void ops_init_range_partition(ops_store *st) {
    uint64_t B = (st->K + st->N - 1) / st->N;
    for (uint64_t k = 0; k < st->K; ++k) {
        st->owner[k] = (uint32_t)(k / B);
        st->slot[k] = (uint32_t)(k % B);
    }
    for (uint32_t p = 0; p < st->N; ++p) {
        uint64_t first = (uint64_t)p * B;
        uint64_t cnt = first >= st->K ? 0 : (st->K - first < B ? st->K - first : B);
        uint64_t t = 0;
        for (uint64_t s = st->S; s-- > cnt;) st->stack[(uint64_t)p * st->S + t++] = (uint32_t)s;
        st->top[p] = t;
    }
}

static int keys_in_range(const ops_store *st, const uint64_t *keys, uint64_t n) {
    for (uint64_t t = 0; t < n; ++t)
        if (keys[t] >= st->K) return 0;
    return 1;
}

int ops_set_rows(ops_store *st, const uint64_t *keys, uint64_t n, const float *vals) {
    if (!keys_in_range(st, keys, n)) return OPS_ERR_KEY_RANGE;
    for (uint64_t t = 0; t < n; ++t)
        memcpy(st->rows + keys[t] * st->L, vals + t * st->L, st->L * sizeof(float));
    return OPS_OK;
}

/* pull (Table 2): out[t] = current value of keys[t], one row per occurrence. */
int ops_pull(ops_store *st, const uint64_t *keys, uint64_t n, float *out) {
    if (!keys_in_range(st, keys, n)) return OPS_ERR_KEY_RANGE;
    for (uint64_t t = 0; t < n; ++t)
        memcpy(out + t * st->L, st->rows + keys[t] * st->L, st->L * sizeof(float));
    return OPS_OK;
}

/* ---- per-call accumulation: the cumulative push of Section 2.1 ---- */
static double *acc_row(ops_store *st, uint64_t key) {
    int32_t a = st->acc_of[key];
    if (a < 0) {
        if (st->n_touched == st->cap_touched) {
            uint64_t cap = st->cap_touched ? st->cap_touched * 2 : 1024;
            st->touched = (uint64_t *)realloc(st->touched, cap * sizeof(uint64_t));
            st->acc = (double *)realloc(st->acc, cap * st->L * sizeof(double));
            st->cap_touched = cap;
        }
        a = (int32_t)st->n_touched++;
        st->acc_of[key] = a;
        st->touched[a] = key;
        memset(st->acc + (uint64_t)a * st->L, 0, st->L * sizeof(double));
    }
    return st->acc + (uint64_t)a * st->L;
}

static void apply_acc(ops_store *st) {
    for (uint64_t a = 0; a < st->n_touched; ++a) {
        uint64_t key = st->touched[a];
        float *row = st->rows + key * st->L;
        const double *sum = st->acc + a * st->L;
        for (uint32_t c = 0; c < st->L; ++c) row[c] = (float)((double)row[c] + sum[c]);
        st->acc_of[key] = -1;
    }
    st->n_touched = 0;
}

/* push (Table 2, cumulative): row(k) += sum of the call's updates for k. */
int ops_push(ops_store *st, const uint64_t *keys, uint64_t n, const float *upd) {
    if (!keys_in_range(st, keys, n)) return OPS_ERR_KEY_RANGE;
    for (uint64_t t = 0; t < n; ++t) {
        double *a = acc_row(st, keys[t]);
        for (uint32_t c = 0; c < st->L; ++c) a[c] += (double)upd[t * st->L + c];
    }
    apply_acc(st);
    return OPS_OK;
}

static int cmp_u64(const void *a, const void *b) {
    uint64_t x = *(const uint64_t *)a, y = *(const uint64_t *)b;
    return x < y ? -1 : x > y;
}

/* localize (Section 3.1 API, Section 3.2 relocation): every distinct requested
 * key that worker w does not own moves to w's partition; the location table is
 * rewritten; the value travels with the key.  End state of the three-message
 * protocol of Figure 4, with no in-flight window.  Slot policy (the paper has
 * none; this repository's definition): distinct keys ascending; the m-th moved
 * key takes the m-th slot from the top of w's free stack; afterwards the
 * vacated slots are pushed onto their old owners' stacks in ascending key
 * order.  If w has too few free slots the call changes nothing. */
int ops_localize(ops_store *st, uint32_t w, const uint64_t *keys, uint64_t n) {
    if (w >= st->N) return OPS_ERR_WORKER_RANGE;
    if (!keys_in_range(st, keys, n)) return OPS_ERR_KEY_RANGE;
    if (n == 0) return OPS_OK;
    uint64_t *d = (uint64_t *)malloc(n * sizeof(uint64_t));
    memcpy(d, keys, n * sizeof(uint64_t));
    qsort(d, n, sizeof(uint64_t), cmp_u64);
    uint64_t m = 0;
    for (uint64_t t = 0; t < n; ++t) {
        if (t > 0 && d[t] == d[t - 1]) continue;        /* duplicates collapse */
        if (st->owner[d[t]] == w) continue;             /* already local: nothing to do */
        d[m++] = d[t];
    }
    if (m > st->top[w]) { free(d); return OPS_ERR_CAPACITY; }
    uint32_t *stack_w = st->stack + (uint64_t)w * st->S;
    uint64_t top_w = st->top[w];
    st->top[w] = top_w - m;
    for (uint64_t q = 0; q < m; ++q) {                  /* vacate, ascending key order */
        uint64_t k = d[q];
        uint32_t p = st->owner[k];
        st->stack[(uint64_t)p * st->S + st->top[p]++] = st->slot[k];
    }
    for (uint64_t q = 0; q < m; ++q) {                  /* occupy and rewrite the table */
        uint64_t k = d[q];
        st->owner[k] = w;
        st->slot[k] = stack_w[top_w - 1 - q];
    }
    free(d);
    return OPS_OK;
}

int ops_get_location(ops_store *st, const uint64_t *keys, uint64_t n, uint32_t *owner, uint32_t *slot) {
    if (!keys_in_range(st, keys, n)) return OPS_ERR_KEY_RANGE;
    for (uint64_t t = 0; t < n; ++t) { owner[t] = st->owner[keys[t]]; slot[t] = st->slot[keys[t]]; }
    return OPS_OK;
}

/* raw views for the tests */
float *ops_rows(ops_store *st) { return st->rows; }
uint32_t *ops_owner(ops_store *st) { return st->owner; }
uint32_t *ops_slot(ops_store *st) { return st->slot; }
uint32_t *ops_stack(ops_store *st) { return st->stack; }
uint64_t *ops_top(ops_store *st) { return st->top; }

/* numerically stable log(1 + exp(z)) */
static double softplus(double z) { return (z > 0 ? z : 0) + log1p(exp(-fabs(z))); }
static double sigmoid(double z) { return z >= 0 ? 1.0 / (1.0 + exp(-z)) : exp(z) / (1.0 + exp(z)); }

/* Matrix factorization by SGD (task of Section 4.1; the paper prints no
 * formula).  Key i < col_key_base is row factor w_i, key col_key_base + j is
 * column factor h_j.  Per observed cell (i, j, v), at the pre-batch w, h:
 *   e = v - <w, h>
 *   loss = e^2 / 2 + lambda / 2 * (|w|^2 + |h|^2)
 *   w += lr * (e * h - lambda * w),  h += lr * (e * w - lambda * h)
 * i.e. one plain gradient step on that loss; the L2 term counts once per
 * occurrence of a key. */
int ops_step_mf(ops_store *st, const uint32_t *ci, const uint32_t *cj, const float *cv, uint64_t n,
                uint64_t col_key_base, float lr_f, float lambda_f, double *loss_accum) {
    const uint32_t L = st->L;
    const double lr = lr_f, lam = lambda_f;
    for (uint64_t t = 0; t < n; ++t)
        if (ci[t] >= col_key_base || col_key_base + cj[t] >= st->K) return OPS_ERR_KEY_RANGE;
    double loss = 0;
    for (uint64_t t = 0; t < n; ++t) {
        uint64_t kw = ci[t], kh = col_key_base + cj[t];
        const float *w = st->rows + kw * L, *h = st->rows + kh * L;
        double dot = 0, nw = 0, nh = 0;
        for (uint32_t c = 0; c < L; ++c) {
            dot += (double)w[c] * h[c];
            nw += (double)w[c] * w[c];
            nh += (double)h[c] * h[c];
        }
        double e = (double)cv[t] - dot;
        loss += 0.5 * e * e + 0.5 * lam * (nw + nh);
        double *aw = acc_row(st, kw);
        for (uint32_t c = 0; c < L; ++c) aw[c] += lr * (e * h[c] - lam * w[c]);
        double *ah = acc_row(st, kh);       /* may move st->acc: take it after aw is done */
        for (uint32_t c = 0; c < L; ++c) ah[c] += lr * (e * w[c] - lam * h[c]);
    }
    apply_acc(st);
    if (loss_accum) *loss_accum += loss;
    return OPS_OK;
}

/* ComplEx with AdaGrad and negative sampling (Section 4.1, Appendix A: "SGD with
 * AdaGrad and negative sampling", "AdaGrad metadata in the PS", learning rate
 * 0.1).  Key e < rel_key_base is an entity, key rel_key_base + r a relation.
 * A row is [Re(0..d) | Im(0..d) | G_Re(0..d) | G_Im(0..d)], d = dim, G the
 * element-wise AdaGrad accumulators.
 * Score of (s, r, o):  phi = Re( sum_d  e_s[d] * w_r[d] * conj(e_o[d]) ).
 * A data point is a positive triple and its n_neg negatives, each of which
 * replaces the subject (side 0) or the object (side 1) by neg_ent.  Its loss is
 * sum over the 1 + n_neg triples of softplus(-y * phi), y = +1 / -1.  For every
 * DISTINCT key of the data point, g = d loss / d theta at the pre-batch theta:
 *   dG = g * g,   dtheta = -lr * g / (sqrt(G + g * g) + eps)
 * with the pre-batch G; (dtheta, dG) are pushed additively. */
int ops_step_kge(ops_store *st, const uint32_t *ts, const uint32_t *tr, const uint32_t *to,
                 const uint32_t *neg_ent, const uint8_t *neg_side, uint64_t n, uint32_t n_neg,
                 uint64_t rel_key_base, uint32_t dim, float lr_f, float eps_f, double *loss_accum) {
    const uint32_t L = st->L, d = dim;
    if (L != 4 * d) return OPS_ERR_INVALID_ARG;
    const double lr = lr_f, eps = eps_f;
    for (uint64_t t = 0; t < n; ++t) {
        if (ts[t] >= rel_key_base || to[t] >= rel_key_base || rel_key_base + tr[t] >= st->K)
            return OPS_ERR_KEY_RANGE;
        for (uint32_t q = 0; q < n_neg; ++q)
            if (neg_ent[t * n_neg + q] >= rel_key_base) return OPS_ERR_KEY_RANGE;
    }
    const uint32_t n_slots = 3 + n_neg;             /* s, r, o, negatives */
    uint64_t *key = (uint64_t *)malloc(n_slots * sizeof(uint64_t));
    uint32_t *rep = (uint32_t *)malloc(n_slots * sizeof(uint32_t));
    double *g = (double *)malloc((uint64_t)n_slots * 2 * d * sizeof(double));
    double loss = 0;
    for (uint64_t t = 0; t < n; ++t) {
        key[0] = ts[t]; key[1] = rel_key_base + tr[t]; key[2] = to[t];
        for (uint32_t q = 0; q < n_neg; ++q) key[3 + q] = neg_ent[t * n_neg + q];
        for (uint32_t u = 0; u < n_slots; ++u) {    /* first slot holding the same key */
            rep[u] = u;
            for (uint32_t z = 0; z < u; ++z)
                if (key[z] == key[u]) { rep[u] = z; break; }
        }
        memset(g, 0, (uint64_t)n_slots * 2 * d * sizeof(double));
        for (uint32_t q = 0; q <= n_neg; ++q) {     /* q = 0: the positive triple */
            uint32_t us = 0, uo = 2;
            double y = 1.0;
            if (q > 0) {
                y = -1.0;
                if (neg_side[t * n_neg + q - 1] == 0) us = 3 + q - 1; else uo = 3 + q - 1;
            }
            const float *S = st->rows + key[us] * L, *R = st->rows + key[1] * L, *O = st->rows + key[uo] * L;
            double phi = 0;
            for (uint32_t c = 0; c < d; ++c) {
                double a = S[c], b = S[d + c], cr = R[c], ci = R[d + c], e = O[c], f = O[d + c];
                phi += cr * (a * e + b * f) + ci * (a * f - b * e);
            }
            loss += softplus(-y * phi);
            double coef = -y * sigmoid(-y * phi);   /* d loss / d phi */
            double *gs = g + (uint64_t)rep[us] * 2 * d, *gr = g + (uint64_t)rep[1] * 2 * d,
                   *go = g + (uint64_t)rep[uo] * 2 * d;
            for (uint32_t c = 0; c < d; ++c) {
                double a = S[c], b = S[d + c], cr = R[c], ci = R[d + c], e = O[c], f = O[d + c];
                /* each += reads only pre-batch values, so aliasing gs == go is fine */
                gs[c] += coef * (cr * e + ci * f);
                gs[d + c] += coef * (cr * f - ci * e);
                gr[c] += coef * (a * e + b * f);
                gr[d + c] += coef * (a * f - b * e);
                go[c] += coef * (cr * a - ci * b);
                go[d + c] += coef * (cr * b + ci * a);
            }
        }
        for (uint32_t u = 0; u < n_slots; ++u) {
            if (rep[u] != u) continue;
            const float *G = st->rows + key[u] * L + 2 * d;
            const double *gu = g + (uint64_t)u * 2 * d;
            double *a = acc_row(st, key[u]);
            for (uint32_t c = 0; c < 2 * d; ++c) {
                double g2 = gu[c] * gu[c];
                a[c] += -lr * gu[c] / (sqrt((double)G[c] + g2) + eps);
                a[2 * d + c] += g2;
            }
        }
    }
    free(key); free(rep); free(g);
    apply_acc(st);
    if (loss_accum) *loss_accum += loss;
    return OPS_OK;
}

/* RESCAL with AdaGrad and negative sampling (Section 4.1 names the model; Table 4 gives entity dimension d = 100
 * and relation dimension d * d = 10,000; training as for ComplEx, Appendix A).  All rows of the store have one
 * length, so a relation's d x d matrix is held as d keys, one per matrix row:
 *   key e < rel_key_base                    entity e,        row [x(0..d) | G(0..d)]
 *   key rel_key_base + r * d + a            row a of R_r,    row [R_r[a][0..d) | G(0..d)]
 * with G the element-wise AdaGrad accumulators (L = 2 d).
 * Score of (s, r, o):  phi = x_s^T R_r x_o = sum_a sum_b x_s[a] R_r[a][b] x_o[b].
 * Data points, negatives, loss softplus(-y phi), and the AdaGrad step per DISTINCT key of a data point from
 * pre-batch (theta, G) are those of ops_step_kge; the d matrix-row keys of a data point are distinct by
 * construction, entity keys may repeat among subject, object and negatives. */
int ops_step_rescal(ops_store *st, const uint32_t *ts, const uint32_t *tr, const uint32_t *to,
                    const uint32_t *neg_ent, const uint8_t *neg_side, uint64_t n, uint32_t n_neg,
                    uint64_t rel_key_base, uint32_t dim, float lr_f, float eps_f, double *loss_accum) {
    const uint32_t L = st->L, d = dim;
    if (L != 2 * d) return OPS_ERR_INVALID_ARG;
    const double lr = lr_f, eps = eps_f;
    for (uint64_t t = 0; t < n; ++t) {
        if (ts[t] >= rel_key_base || to[t] >= rel_key_base || rel_key_base + ((uint64_t)tr[t] + 1) * d > st->K)
            return OPS_ERR_KEY_RANGE;
        for (uint32_t q = 0; q < n_neg; ++q)
            if (neg_ent[t * n_neg + q] >= rel_key_base) return OPS_ERR_KEY_RANGE;
    }
    const uint32_t n_slots = 2 + n_neg;             /* s, o, negatives: the entity keys of a data point */
    uint64_t *key = (uint64_t *)malloc(n_slots * sizeof(uint64_t));
    uint32_t *rep = (uint32_t *)malloc(n_slots * sizeof(uint32_t));
    double *g = (double *)malloc((uint64_t)n_slots * d * sizeof(double));
    double *gR = (double *)malloc((uint64_t)d * d * sizeof(double));
    double loss = 0;
    for (uint64_t t = 0; t < n; ++t) {
        key[0] = ts[t]; key[1] = to[t];
        for (uint32_t q = 0; q < n_neg; ++q) key[2 + q] = neg_ent[t * n_neg + q];
        for (uint32_t u = 0; u < n_slots; ++u) {    /* first slot holding the same key */
            rep[u] = u;
            for (uint32_t z = 0; z < u; ++z)
                if (key[z] == key[u]) { rep[u] = z; break; }
        }
        const uint64_t rk = rel_key_base + (uint64_t)tr[t] * d;     /* key of row 0 of R_r */
        memset(g, 0, (uint64_t)n_slots * d * sizeof(double));
        memset(gR, 0, (uint64_t)d * d * sizeof(double));
        for (uint32_t q = 0; q <= n_neg; ++q) {     /* q = 0: the positive triple */
            uint32_t us = 0, uo = 1;
            double y = 1.0;
            if (q > 0) {
                y = -1.0;
                if (neg_side[t * n_neg + q - 1] == 0) us = 2 + q - 1; else uo = 2 + q - 1;
            }
            const float *S = st->rows + key[us] * L, *O = st->rows + key[uo] * L;
            double phi = 0;
            for (uint32_t a = 0; a < d; ++a) {
                const float *Ra = st->rows + (rk + a) * L;
                double ro = 0;
                for (uint32_t b = 0; b < d; ++b) ro += (double)Ra[b] * O[b];
                phi += (double)S[a] * ro;
            }
            loss += softplus(-y * phi);
            double coef = -y * sigmoid(-y * phi);   /* d loss / d phi */
            double *gs = g + (uint64_t)rep[us] * d, *go = g + (uint64_t)rep[uo] * d;
            for (uint32_t a = 0; a < d; ++a) {
                const float *Ra = st->rows + (rk + a) * L;
                for (uint32_t b = 0; b < d; ++b) {
                    /* each += reads only pre-batch values, so aliasing gs == go is fine */
                    gs[a] += coef * (double)Ra[b] * O[b];
                    go[b] += coef * (double)S[a] * Ra[b];
                    gR[(uint64_t)a * d + b] += coef * (double)S[a] * O[b];
                }
            }
        }
        for (uint32_t u = 0; u < n_slots; ++u) {
            if (rep[u] != u) continue;
            const float *G = st->rows + key[u] * L + d;
            const double *gu = g + (uint64_t)u * d;
            double *acc = acc_row(st, key[u]);
            for (uint32_t c = 0; c < d; ++c) {
                double g2 = gu[c] * gu[c];
                acc[c] += -lr * gu[c] / (sqrt((double)G[c] + g2) + eps);
                acc[d + c] += g2;
            }
        }
        for (uint32_t a = 0; a < d; ++a) {
            const float *G = st->rows + (rk + a) * L + d;
            const double *gu = gR + (uint64_t)a * d;
            double *acc = acc_row(st, rk + a);
            for (uint32_t c = 0; c < d; ++c) {
                double g2 = gu[c] * gu[c];
                acc[c] += -lr * gu[c] / (sqrt((double)G[c] + g2) + eps);
                acc[d + c] += g2;
            }
        }
    }
    free(key); free(rep); free(g); free(gR);
    apply_acc(st);
    if (loss_accum) *loss_accum += loss;
    return OPS_OK;
}

/* Skip-gram with negative sampling (Section 4.1, Appendix A: window 5, negative
 * sampling).  Key w < out_key_base is the input vector v_w, key out_key_base + w
 * the output vector u_w.  Centers are the stream positions
 * [first_pos, first_pos + n_centers); the contexts of position p are the
 * positions q != p with |q - p| <= window inside [0, corpus_len).  Pairs are
 * numbered in (p ascending, q ascending) order from 0 at the batch's first
 * pair; pair z uses negs[z * n_neg .. z * n_neg + n_neg).  For each pair and
 * each target (u, y) in {(u_context, 1), (u_negative, 0)...}, at pre-batch
 * values:  x = <v, u>,  g = sigmoid(x) - y,
 *   loss += -y log sigmoid(x) - (1 - y) log sigmoid(-x)
 *   u += -lr * g * v,   v += -lr * g * u. */
int ops_step_sgns(ops_store *st, const uint32_t *tokens, uint64_t first_pos, uint64_t n_centers,
                  uint64_t corpus_len, uint32_t window, const uint32_t *negs, uint32_t n_neg,
                  uint64_t out_key_base, float lr_f, double *loss_accum) {
    const uint32_t L = st->L;
    const double lr = lr_f;
    if (first_pos + n_centers > corpus_len) return OPS_ERR_INVALID_ARG;
    uint64_t z = 0;
    for (uint64_t p = first_pos; p < first_pos + n_centers; ++p) {     /* validate first */
        uint64_t lo = p >= window ? p - window : 0;
        uint64_t hi = p + window < corpus_len ? p + window : corpus_len - 1;
        if (tokens[p] >= out_key_base) return OPS_ERR_KEY_RANGE;
        for (uint64_t q = lo; q <= hi; ++q) {
            if (q == p) continue;
            if (out_key_base + tokens[q] >= st->K) return OPS_ERR_KEY_RANGE;
            for (uint32_t i = 0; i < n_neg; ++i)
                if (out_key_base + negs[z * n_neg + i] >= st->K) return OPS_ERR_KEY_RANGE;
            ++z;
        }
    }
    double loss = 0;
    z = 0;
    for (uint64_t p = first_pos; p < first_pos + n_centers; ++p) {
        uint64_t lo = p >= window ? p - window : 0;
        uint64_t hi = p + window < corpus_len ? p + window : corpus_len - 1;
        uint64_t kv = tokens[p];
        const float *v = st->rows + kv * L;
        for (uint64_t q = lo; q <= hi; ++q) {
            if (q == p) continue;
            for (uint32_t i = 0; i <= n_neg; ++i) {        /* i = 0: the true context */
                uint64_t ku = out_key_base + (i == 0 ? tokens[q] : negs[z * n_neg + i - 1]);
                double y = i == 0 ? 1.0 : 0.0;
                const float *u = st->rows + ku * L;
                double x = 0;
                for (uint32_t c = 0; c < L; ++c) x += (double)v[c] * u[c];
                double gcoef = sigmoid(x) - y;
                loss += y > 0.5 ? softplus(-x) : softplus(x);
                double *au = acc_row(st, ku);
                for (uint32_t c = 0; c < L; ++c) au[c] += -lr * gcoef * v[c];
                double *av = acc_row(st, kv);
                for (uint32_t c = 0; c < L; ++c) av[c] += -lr * gcoef * u[c];
            }
            ++z;
        }
    }
    apply_acc(st);
    if (loss_accum) *loss_accum += loss;
    return OPS_OK;
}
