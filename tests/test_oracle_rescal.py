"""Pins of the oracle's RESCAL step (Section 4.1 names the model; the score is Nickel et al.'s bilinear form
x_s^T R_r x_o).  The score against a matrix product written here with numpy, special relations (identity, zero but
one entry, transpose), the gradient per DISTINCT key against central differences of a loss written out here (merge
cases included), AdaGrad with a non-zero pre-batch accumulator, additivity over data points.  None of these calls
the oracle to produce its own expected value."""
import numpy as np
import pytest

from oracle import OracleStore


def central_diff(fn, x, h=1e-6):
    g = np.zeros_like(x)
    it = np.nditer(x, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        xp = x.copy(); xp[i] += h
        xm = x.copy(); xm[i] -= h
        g[i] = (fn(xp) - fn(xm)) / (2 * h)
    return g


def rescal_rows(E, Rn, d, seed=0, G=None):
    """E entity rows and Rn * d matrix-row rows of [d values | d accumulators]."""
    rng = np.random.default_rng(seed)
    emb = rng.normal(0, 0.6, size=(E + Rn * d, d))
    acc = np.zeros_like(emb) if G is None else rng.uniform(0, G, size=emb.shape)
    return np.concatenate([emb, acc], axis=1).astype(np.float32)


def rel(theta, E, d, r):
    return theta[E + r * d:E + (r + 1) * d, :d]                 # row a of the block = row a of R_r


def rescal_dp_loss(theta, E, d, s, r, o, negs, sides):
    def phi(a, b):
        return theta[a, :d] @ rel(theta, E, d, r) @ theta[b, :d]
    tot = np.logaddexp(0, -phi(s, o))
    for n, side in zip(negs, sides):
        tot += np.logaddexp(0, phi(n, o) if side == 0 else phi(s, n))
    return tot


def rescal_run(rows, E, d, s, r, o, negs, sides, lr=0.1, eps=1e-8):
    st = OracleStore(rows.shape[0], 2 * d, 1)
    st.set_rows(np.arange(rows.shape[0]), rows)
    st.step_rescal([s], [r], [o], np.array(negs, np.uint32).reshape(1, -1), np.array(sides, np.uint8).reshape(1, -1),
                   E, d, lr, eps)
    return st


def test_rescal_score_is_the_bilinear_form_and_special_relations():
    E, Rn, d = 4, 2, 5
    rows = rescal_rows(E, Rn, d, seed=5)

    def score(rows, s, r, o):
        st = rescal_run(rows, E, d, s, r, o, [], [])
        return -np.log(np.expm1(st.loss[0]))                   # loss = softplus(-phi)

    th = rows.astype(np.float64)
    assert np.isclose(score(rows, 0, 1, 2), th[0, :d] @ rel(th, E, d, 1) @ th[2, :d], rtol=1e-10)
    assert not np.isclose(score(rows, 0, 1, 2), score(rows, 2, 1, 0))       # a general R is not symmetric
    assert not np.isclose(score(rows, 0, 1, 2), score(rows, 0, 0, 2))       # ... and the relation matters
    eye = rows.copy(); eye[E + d:E + 2 * d, :d] = np.eye(d)    # identity: the dot product of the entities
    assert np.isclose(score(eye, 0, 1, 2), th[0, :d] @ th[2, :d], rtol=1e-10)
    one = rows.copy(); one[E + d:E + 2 * d, :d] = 0; one[E + d + 1, 3] = 2.0    # R[1][3] = 2 only: row index = subject side
    assert np.isclose(score(one, 0, 1, 2), 2.0 * th[0, 1] * th[2, 3], rtol=1e-10)
    tr = rows.copy(); tr[E + d:E + 2 * d, :d] = rel(th, E, d, 1).T.astype(np.float32)   # transposed: roles swapped
    assert np.isclose(score(tr, 2, 1, 0), score(rows, 0, 1, 2), rtol=1e-10)


@pytest.mark.parametrize("case", ["distinct", "s_eq_o", "neg_eq_s", "neg_eq_o", "neg_repeat", "everything"])
def test_rescal_gradient_per_distinct_key_matches_finite_differences(case):
    E, Rn, d = 8, 2, 3
    s, r, o = 1, 1, 2
    negs, sides = [3, 4, 5, 6], [0, 1, 1, 0]
    if case == "s_eq_o": o = s
    if case == "neg_eq_s": negs[1] = s                         # (s, r, s)
    if case == "neg_eq_o": negs[0] = o                         # (o, r, o)
    if case == "neg_repeat": negs[2] = negs[1] = 7; sides[2] = 0
    if case == "everything": o = s; negs = [s, s, 3, 3]; sides = [0, 1, 0, 1]
    rows = rescal_rows(E, Rn, d, seed=11)                      # G = 0
    th0 = rows.astype(np.float64)
    st = rescal_run(rows, E, d, s, r, o, negs, sides)
    emb = th0[:, :d].copy()

    def loss_of(e):
        th = th0.copy(); th[:, :d] = e
        return rescal_dp_loss(th, E, d, s, r, o, negs, sides)

    g_fd = central_diff(loss_of, emb)
    dG = st.rows[:, d:].astype(np.float64)                     # G was 0: dG = g * g
    dtheta = st.rows[:, :d].astype(np.float64) - emb
    assert np.allclose(dG, g_fd ** 2, rtol=2e-5, atol=1e-12)
    assert np.isclose(st.loss[0], loss_of(emb), rtol=1e-12)
    big = np.abs(g_fd) > 1e-4
    assert (np.sign(dtheta[big]) == -np.sign(g_fd[big])).all()
    assert np.allclose(np.abs(dtheta[big]), 0.1, rtol=1e-5)    # G = 0: |dtheta| = lr |g| / (|g| + eps)
    touched = np.zeros(E + Rn * d, bool)
    touched[[s, o] + negs] = True
    touched[E + r * d:E + (r + 1) * d] = True
    assert (st.rows[~touched] == rows[~touched]).all()         # the other relation's matrix among them
    assert (g_fd[E + r * d:E + (r + 1) * d] != 0).all()        # every row of R_r gets a gradient


def test_rescal_adagrad_uses_the_prebatch_accumulator():
    E, Rn, d = 6, 1, 4
    rows = rescal_rows(E, Rn, d, seed=2, G=0.5)
    th0 = rows.astype(np.float64)
    s, r, o, negs, sides = 0, 0, 1, [2, 3], [0, 1]
    st = rescal_run(rows, E, d, s, r, o, negs, sides, lr=0.1, eps=1e-8)
    emb = th0[:, :d].copy()

    def loss_of(e):
        th = th0.copy(); th[:, :d] = e
        return rescal_dp_loss(th, E, d, s, r, o, negs, sides)

    g = central_diff(loss_of, emb)
    G0 = th0[:, d:]
    assert np.allclose(st.rows[:, d:], G0 + g * g, rtol=1e-6)
    assert (st.rows[:, d:] >= rows[:, d:]).all()
    want = emb - np.float64(np.float32(0.1)) * g / (np.sqrt(G0 + g * g) + np.float64(np.float32(1e-8)))
    assert np.allclose(st.rows[:, :d], want, rtol=1e-6, atol=1e-7)


def test_rescal_batch_sums_per_data_point_pushes():
    """Two data points sharing entities and the relation: the batch equals the sum of their separate pushes."""
    E, Rn, d = 6, 2, 3
    rows = rescal_rows(E, Rn, d, seed=4, G=0.3)
    a = rescal_run(rows, E, d, 0, 0, 1, [2, 3], [0, 1])
    b = rescal_run(rows, E, d, 1, 0, 0, [2, 5], [1, 1])
    st = OracleStore(E + Rn * d, 2 * d, 1)
    st.set_rows(np.arange(E + Rn * d), rows)
    st.step_rescal([0, 1], [0, 0], [1, 0], np.array([[2, 3], [2, 5]], np.uint32), np.array([[0, 1], [1, 1]], np.uint8),
                   E, d, 0.1, 1e-8)
    want = rows.astype(np.float64) + (a.rows.astype(np.float64) - rows) + (b.rows.astype(np.float64) - rows)
    assert np.allclose(st.rows, want, rtol=0, atol=2e-7)
    assert np.isclose(st.loss[0], a.loss[0] + b.loss[0], rtol=1e-13)


def test_rescal_rejects_keys_out_of_range_and_a_wrong_row_length():
    E, Rn, d = 5, 2, 3
    rows = rescal_rows(E, Rn, d)
    st = OracleStore(E + Rn * d, 2 * d, 1)
    st.set_rows(np.arange(E + Rn * d), rows)
    none = (np.zeros((1, 0), np.uint32), np.zeros((1, 0), np.uint8))
    for s, r, o in ((E, 0, 1), (0, 0, E), (0, Rn, 1)):         # subject / object in the relations' range; relation past the end
        with pytest.raises(Exception):
            st.step_rescal([s], [r], [o], *none, E, d, 0.1, 1e-8)
    with pytest.raises(Exception):
        st.step_rescal([0], [0], [1], np.array([[E]], np.uint32), np.array([[0]], np.uint8), E, d, 0.1, 1e-8)
    assert (st.rows == rows).all()
    with pytest.raises(Exception):
        st.step_rescal([0], [0], [1], *none, E, d + 1, 0.1, 1e-8)
