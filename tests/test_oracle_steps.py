"""Pins for the oracle's three training steps (tasks of Section 4.1 / Appendix A).

Each gradient is checked against central finite differences of a loss that is
written out here independently (numpy fp64; complex numbers for ComplEx), plus
special cases that reduce to textbook results.  The oracle's step applies
theta += -lr * g, so with lr = 1 the gradient is read off the state change.
"""
import numpy as np
import pytest

from oracle import OracleStore
from synth import workloads as W


def central_diff(fn, x, h=1e-6):
    g = np.zeros_like(x)
    flat, gf = x.reshape(-1), g.reshape(-1)
    for i in range(flat.size):
        old = flat[i]
        flat[i] = old + h
        fp = fn(x)
        flat[i] = old - h
        fm = fn(x)
        flat[i] = old
        gf[i] = (fp - fm) / (2 * h)
    return g


# ------------------------------------------------------------------ MF ----
def mf_loss(theta, cells, R, lam):
    tot = 0.0
    for i, j, v in cells:
        w, h = theta[i], theta[R + j]
        e = v - w @ h
        tot += 0.5 * e * e + 0.5 * lam * (w @ w + h @ h)
    return tot


def mf_store(R, Cc, L, seed=0):
    rng = np.random.default_rng(seed)
    st = OracleStore(R + Cc, L, 1)
    st.set_rows(np.arange(R + Cc), rng.normal(0, 0.5, size=(R + Cc, L)).astype(np.float32))
    return st


def test_mf_gradient_matches_finite_differences_with_duplicates():
    R, Cc, L, lam = 3, 2, 4, np.float32(0.05)
    st = mf_store(R, Cc, L)
    theta0 = st.rows.astype(np.float64).copy()
    cells = [(0, 1, 0.7), (0, 1, -0.2), (2, 0, 1.5), (0, 0, 0.3), (1, 1, 0.0)]
    i, j, v = (np.array(c) for c in zip(*cells))
    st.step_mf(i, j, v.astype(np.float32), R, 1.0, lam)
    cells32 = [(a, b, float(np.float32(c))) for a, b, c in cells]
    g_fd = central_diff(lambda th: mf_loss(th, cells32, R, float(lam)), theta0.copy())
    g_oracle = -(st.rows.astype(np.float64) - theta0)
    assert np.allclose(g_oracle, g_fd, rtol=0, atol=3e-7)
    assert np.isclose(st.loss[0], mf_loss(theta0, cells32, R, float(lam)), rtol=1e-12)


def test_mf_single_cell_is_textbook_sgd():
    st = mf_store(2, 2, 3, seed=3)
    w, h = st.rows[1].astype(np.float64), st.rows[2 + 0].astype(np.float64)
    lr, lam, v = np.float32(0.01), np.float32(0.05), np.float32(0.9)
    st.step_mf([1], [0], [v], 2, lr, lam)
    e = float(v) - w @ h
    assert (st.rows[1] == (w + float(lr) * (e * h - float(lam) * w)).astype(np.float32)).all()
    assert (st.rows[2] == (h + float(lr) * (e * w - float(lam) * h)).astype(np.float32)).all()


def test_mf_exact_fit_without_regulariser_is_a_fixed_point():
    st = OracleStore(2, 2, 1)
    st.set_rows([0, 1], np.array([[0.5, 2.0], [4.0, 0.25]], np.float32))      # <w,h> = 2.5 exactly
    before = st.rows.copy()
    st.step_mf([0], [0], [np.float32(2.5)], 1, 0.1, 0.0)
    assert (st.rows == before).all() and st.loss[0] == 0.0


def test_mf_distinct_key_batch_equals_sequential_sgd():
    R = Cc = 16
    a, b = mf_store(R, Cc, 5, seed=7), mf_store(R, Cc, 5, seed=7)
    perm_i, perm_j = np.random.default_rng(1).permutation(R), np.random.default_rng(2).permutation(Cc)
    v = np.random.default_rng(3).normal(size=R).astype(np.float32)
    a.step_mf(perm_i, perm_j, v, R, 0.01, 0.05)
    for t in reversed(range(R)):                               # any order
        b.step_mf(perm_i[t:t + 1], perm_j[t:t + 1], v[t:t + 1], R, 0.01, 0.05)
    assert (a.rows == b.rows).all()
    assert np.isclose(a.loss[0], b.loss[0], rtol=1e-13)


def test_mf_planted_model_loss_falls():
    """Planted rank-8 model, uniform cells, the tiny configuration: the epoch loss must fall."""
    cfg = W.MF_TINY
    st = OracleStore(cfg.num_keys, cfg.rank, 1)
    st.set_rows(np.arange(cfg.num_keys), W.mf_init_rows(cfg, 0, cfg.num_keys, "cpu"))
    planted = W.mf_planted(cfg, "cpu")
    i, j, v = W.mf_cells(cfg, planted, 0, cfg.n_cells, "cpu")
    losses = []
    for _ in range(30):
        st.loss[0] = 0
        for b in range(cfg.n_batches):
            s, c = cfg.batch_range(b)
            st.step_mf(i[s:s + c], j[s:s + c], v[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam)
        losses.append(st.loss[0])
    assert np.isfinite(losses).all()
    assert all(b < a for a, b in zip(losses, losses[1:])), losses
    assert losses[-1] < 0.3 * losses[0], losses


# ------------------------------------------------------------- ComplEx ----
def kge_rows(E, Rn, d, seed=0, G=None):
    rng = np.random.default_rng(seed)
    emb = rng.normal(0, 0.6, size=(E + Rn, 2 * d))
    acc = np.zeros_like(emb) if G is None else rng.uniform(0, G, size=emb.shape)
    return np.concatenate([emb, acc], axis=1).astype(np.float32)


def cplx(theta, k, d):
    return theta[k, :d] + 1j * theta[k, d:2 * d]


def kge_dp_loss(theta, E, d, s, r, o, negs, sides):
    """softplus(-y phi) summed over the positive and its negatives; phi via complex arithmetic."""
    def phi(a, b):
        return np.real(np.sum(cplx(theta, a, d) * cplx(theta, E + r, d) * np.conj(cplx(theta, b, d))))
    tot = np.logaddexp(0, -phi(s, o))
    for n, side in zip(negs, sides):
        tot += np.logaddexp(0, phi(n, o) if side == 0 else phi(s, n))
    return tot


def kge_run(rows, E, d, s, r, o, negs, sides, lr=0.1, eps=1e-8):
    st = OracleStore(rows.shape[0], 4 * d, 1)
    st.set_rows(np.arange(rows.shape[0]), rows)
    st.step_kge([s], [r], [o], np.array(negs, np.uint32).reshape(1, -1), np.array(sides, np.uint8).reshape(1, -1),
                E, d, lr, eps)
    return st


def test_complex_score_equals_complex_triple_product_and_special_cases():
    E, Rn, d = 4, 2, 6
    rows = kge_rows(E, Rn, d, seed=5)

    def score(rows, s, r, o):
        st = kge_run(rows, E, d, s, r, o, [], [])
        return -np.log(np.expm1(st.loss[0]))                   # loss = softplus(-phi)

    th = rows.astype(np.float64)
    want = np.real(np.sum(cplx(th, 0, d) * cplx(th, E + 1, d) * np.conj(cplx(th, 2, d))))
    assert np.isclose(score(rows, 0, 1, 2), want, rtol=1e-10)
    real = rows.copy(); real[:, d:2 * d] = 0                   # all imaginary parts zero: tri-linear product
    assert np.isclose(score(real, 0, 1, 2), np.sum(th[0, :d] * th[E + 1, :d] * th[2, :d]), rtol=1e-10)
    rr = rows.copy(); rr[E + 1, d:2 * d] = 0                   # real relation: symmetric
    assert np.isclose(score(rr, 0, 1, 2), score(rr, 2, 1, 0), rtol=1e-10)
    ri = rows.copy(); ri[E + 1, :d] = 0                        # imaginary relation: antisymmetric
    assert np.isclose(score(ri, 0, 1, 2), -score(ri, 2, 1, 0), rtol=1e-10)


@pytest.mark.parametrize("case", ["distinct", "s_eq_o", "neg_eq_s", "neg_eq_o", "neg_repeat", "everything"])
def test_complex_gradient_per_distinct_key_matches_finite_differences(case):
    E, Rn, d = 8, 2, 3
    s, r, o = 1, 1, 2
    negs, sides = [3, 4, 5, 6], [0, 1, 1, 0]
    if case == "s_eq_o": o = s
    if case == "neg_eq_s": negs[1] = s                         # (s, r, s)
    if case == "neg_eq_o": negs[0] = o                         # (o, r, o)
    if case == "neg_repeat": negs[2] = negs[1] = 7; sides[2] = 0
    if case == "everything": o = s; negs = [s, s, 3, 3]; sides = [0, 1, 0, 1]
    rows = kge_rows(E, Rn, d, seed=11)                         # G = 0
    th0 = rows.astype(np.float64)
    st = kge_run(rows, E, d, s, r, o, negs, sides)
    emb = th0[:, :2 * d].copy()

    def loss_of(e):
        th = th0.copy(); th[:, :2 * d] = e
        return kge_dp_loss(th, E, d, s, r, o, negs, sides)

    g_fd = central_diff(loss_of, emb)
    dG = st.rows[:, 2 * d:].astype(np.float64)                 # G was 0: dG = g * g
    dtheta = st.rows[:, :2 * d].astype(np.float64) - emb
    assert np.allclose(dG, g_fd ** 2, rtol=2e-5, atol=1e-12)
    assert np.isclose(st.loss[0], loss_of(emb), rtol=1e-12)
    big = np.abs(g_fd) > 1e-4
    assert (np.sign(dtheta[big]) == -np.sign(g_fd[big])).all()
    assert np.allclose(np.abs(dtheta[big]), 0.1, rtol=1e-5)    # G = 0: |dtheta| = lr |g| / (|g| + eps)
    touched = np.zeros(E + Rn, bool); touched[[s, o, E + r] + negs] = True
    assert (st.rows[~touched] == rows[~touched]).all()


def test_adagrad_uses_prebatch_accumulator_and_never_decreases_it():
    E, Rn, d = 6, 1, 4
    rows = kge_rows(E, Rn, d, seed=2, G=0.5)
    th0 = rows.astype(np.float64)
    s, r, o, negs, sides = 0, 0, 1, [2, 3], [0, 1]
    st = kge_run(rows, E, d, s, r, o, negs, sides, lr=0.1, eps=1e-8)
    emb = th0[:, :2 * d].copy()

    def loss_of(e):
        th = th0.copy(); th[:, :2 * d] = e
        return kge_dp_loss(th, E, d, s, r, o, negs, sides)

    g = central_diff(loss_of, emb)
    G0 = th0[:, 2 * d:]
    assert np.allclose(st.rows[:, 2 * d:], G0 + g * g, rtol=1e-6)
    assert (st.rows[:, 2 * d:] >= rows[:, 2 * d:]).all()
    want = emb - np.float64(np.float32(0.1)) * g / (np.sqrt(G0 + g * g) + np.float64(np.float32(1e-8)))
    assert np.allclose(st.rows[:, :2 * d], want, rtol=1e-6, atol=1e-7)


def test_kge_batch_sums_per_data_point_pushes():
    """Two data points sharing keys: the batch equals the sum of their separate pushes from the same state."""
    E, Rn, d = 6, 2, 3
    rows = kge_rows(E, Rn, d, seed=4, G=0.3)
    a = kge_run(rows, E, d, 0, 0, 1, [2, 3], [0, 1])
    b = kge_run(rows, E, d, 1, 0, 0, [2, 5], [1, 1])
    st = OracleStore(E + Rn, 4 * d, 1)
    st.set_rows(np.arange(E + Rn), rows)
    st.step_kge([0, 1], [0, 0], [1, 0], np.array([[2, 3], [2, 5]], np.uint32), np.array([[0, 1], [1, 1]], np.uint8),
                E, d, 0.1, 1e-8)
    want = rows.astype(np.float64) + (a.rows.astype(np.float64) - rows) + (b.rows.astype(np.float64) - rows)
    assert np.allclose(st.rows, want, rtol=0, atol=2e-7)
    assert np.isclose(st.loss[0], a.loss[0] + b.loss[0], rtol=1e-13)


# ---------------------------------------------------------------- SGNS ----
def sgns_loss(theta, V, tokens, first, n, window, negs, n_neg):
    T, tot, z = len(tokens), 0.0, 0
    for p in range(first, first + n):
        v = theta[tokens[p]]
        for q in range(max(0, p - window), min(T - 1, p + window) + 1):
            if q == p:
                continue
            tot += np.logaddexp(0, -(v @ theta[V + tokens[q]]))
            for i in range(n_neg):
                tot += np.logaddexp(0, v @ theta[V + negs[z * n_neg + i]])
            z += 1
    return tot


def test_sgns_gradient_matches_finite_differences():
    V, L, window, n_neg = 5, 3, 2, 2
    rng = np.random.default_rng(0)
    tokens = rng.integers(0, V, size=9)
    first, n = 1, 7                                            # both clipped ends appear across the two calls below
    cfg = W.scaled(W.SGNS_TINY, vocab=V, n_tokens=9, window=window, n_neg=n_neg)
    n_pairs = cfg.pairs_before(first + n) - cfg.pairs_before(first)
    negs = rng.integers(0, V, size=n_pairs * n_neg)
    rows = rng.normal(0, 0.7, size=(2 * V, L)).astype(np.float32)
    st = OracleStore(2 * V, L, 1)
    st.set_rows(np.arange(2 * V), rows)
    st.step_sgns(tokens, first, n, window, negs, n_neg, V, 1.0)
    th0 = rows.astype(np.float64)
    g_fd = central_diff(lambda th: sgns_loss(th, V, tokens, first, n, window, negs, n_neg), th0.copy())
    assert np.allclose(-(st.rows.astype(np.float64) - th0), g_fd, rtol=0, atol=1e-6)
    assert np.isclose(st.loss[0], sgns_loss(th0, V, tokens, first, n, window, negs, n_neg), rtol=1e-12)


def test_sgns_pair_count_and_window_clipping():
    V, L = 4, 2
    tokens = np.array([0, 1, 2, 3, 0, 1])
    rows = np.zeros((2 * V, L), np.float32)                    # x = 0 everywhere: loss = log 2 per scored target
    for first, n, window in [(0, 6, 5), (0, 6, 1), (2, 2, 2), (5, 1, 3)]:
        cfg = W.scaled(W.SGNS_TINY, vocab=V, n_tokens=6, window=window, n_neg=3)
        pairs = cfg.pairs_before(first + n) - cfg.pairs_before(first)
        brute = sum(1 for p in range(first, first + n) for q in range(6) if q != p and abs(q - p) <= window)
        assert pairs == brute
        st = OracleStore(2 * V, L, 1)
        st.set_rows(np.arange(2 * V), rows)
        st.step_sgns(tokens, first, n, window, np.zeros(pairs * 3, np.uint32), 3, V, 0.025)
        assert np.isclose(st.loss[0], pairs * 4 * np.log(2.0), rtol=1e-13)


def test_sgns_single_pair_without_negatives_is_a_logistic_regression_step():
    V, L, lr = 3, 4, np.float32(0.025)
    rows = np.random.default_rng(5).normal(size=(2 * V, L)).astype(np.float32)
    st = OracleStore(2 * V, L, 1)
    st.set_rows(np.arange(2 * V), rows)
    tokens = np.array([2, 1])
    st.step_sgns(tokens, 0, 1, 1, np.zeros(0, np.uint32), 0, V, lr)     # center 2, context 1
    v, u = rows[2].astype(np.float64), rows[V + 1].astype(np.float64)
    g = 1 / (1 + np.exp(-(v @ u))) - 1
    assert (st.rows[2] == (v - float(lr) * g * u).astype(np.float32)).all()
    assert (st.rows[V + 1] == (u - float(lr) * g * v).astype(np.float32)).all()


def test_sgns_zero_output_vectors_first_batch():
    """Output vectors zero: dv = 0 exactly; a word's output vector moves by lr/2 * sum of the centers' v
    over its occurrences as a context minus lr/2 * the same over its occurrences as a negative."""
    cfg = W.scaled(W.SGNS_TINY, vocab=50, n_tokens=400, dim=6, batch=400)
    V, L = cfg.vocab, cfg.dim
    rows = W.sgns_init_rows(cfg, 0, 2 * V, "cpu").numpy()
    assert (rows[V:] == 0).all() and np.abs(rows[:V]).max() <= 0.5 / L
    tokens = W.sgns_tokens(cfg, 0, cfg.n_tokens, "cpu").numpy()
    negs = W.sgns_negatives(cfg, 0, cfg.n_tokens, "cpu").numpy()
    st = OracleStore(2 * V, L, 1)
    st.set_rows(np.arange(2 * V), rows)
    st.step_sgns(tokens, 0, cfg.n_tokens, cfg.window, negs, cfg.n_neg, V, cfg.lr)
    assert (st.rows[:V] == rows[:V]).all()
    want = np.zeros((V, L))
    z = 0
    for p in range(cfg.n_tokens):
        for q in range(max(0, p - 5), min(cfg.n_tokens - 1, p + 5) + 1):
            if q == p:
                continue
            want[tokens[q]] += 0.5 * rows[tokens[p]]
            for i in range(3):
                want[negs[z * 3 + i]] -= 0.5 * rows[tokens[p]]
            z += 1
    assert np.allclose(st.rows[V:], float(np.float32(cfg.lr)) * want, rtol=0, atol=3e-8)
