"""Pins of the oracle's sparse-map front end and of its parameter-blocking schedule (no GPU)."""
import itertools

import numpy as np

from oracle import ABSENT, KeyMapFull, OracleKeyMap, OracleStore, dsgd


# ---------------------------------------------------------------- sparse map ----
def test_keymap_hands_out_dense_keys_in_order_of_first_appearance():
    km = OracleKeyMap(10)
    got = km.insert([2**63 + 5, 7, 2**63 + 5, 123456789012345, 7, 0])
    assert got.tolist() == [0, 1, 0, 2, 1, 3]
    assert km.insert([0, 99, 7]).tolist() == [3, 4, 1]          # known keys keep theirs, the new one is next
    assert len(km) == 5
    assert km.lookup([99, 1, 2**63 + 5]).tolist() == [4, int(ABSENT), 0]


def test_keymap_against_brute_force_list_index():
    rng = np.random.default_rng(0)
    km = OracleKeyMap(400)
    order = []                                                  # brute force: the list of distinct keys as they appeared
    for _ in range(20):
        keys = rng.integers(0, 300, size=50).astype(np.uint64) * np.uint64(0x9E3779B97F4A7C15)
        got = km.insert(keys)
        for k in keys.tolist():
            if k not in order:
                order.append(k)
        assert got.tolist() == [order.index(k) for k in keys.tolist()]
    assert sorted(km.lookup(np.array(order, dtype=np.uint64)).tolist()) == list(range(len(order)))   # a bijection onto 0..D-1


def test_keymap_full_call_adds_nothing():
    km = OracleKeyMap(3)
    km.insert([10, 20])
    try:
        km.insert([20, 30, 40])
        raise AssertionError("expected KeyMapFull")
    except KeyMapFull:
        pass
    assert len(km) == 2 and km.lookup([30, 40]).tolist() == [int(ABSENT)] * 2
    assert km.insert([30]).tolist() == [2]


def test_store_behind_a_keymap_is_a_store_with_renamed_keys():
    """pull/push through the map on sparse keys = pull/push on the dense store with the keys renamed."""
    rng = np.random.default_rng(1)
    sparse = rng.integers(0, 2**62, size=40).astype(np.uint64)
    km = OracleKeyMap(64)
    a = OracleStore(64, 4, 2, 40)
    calls = [rng.choice(sparse, size=25) for _ in range(6)]
    upds = [rng.integers(-3, 4, size=(25, 4)).astype(np.float32) for _ in range(6)]
    total = {}
    for keys, upd in zip(calls, upds):
        a.push(km.insert(keys), upd)
        for k, u in zip(keys.tolist(), upd):
            total[k] = total.get(k, 0) + u.astype(np.float64)
    for k, t in total.items():
        assert (a.pull(km.lookup([k]))[0] == t.astype(np.float32)).all()


# ------------------------------------------------------- parameter blocking ----
def test_strata_partition_the_cells_and_share_no_parameter_within_a_subepoch():
    rng = np.random.default_rng(2)
    rows, cols, N = 37, 23, 4
    i, j = rng.integers(0, rows, size=500), rng.integers(0, cols, size=500)
    st = dsgd.strata(i, j, rows, cols, N)
    allidx = np.sort(np.concatenate(list(st.values())))
    assert (allidx == np.arange(500)).all()                     # every cell in exactly one stratum
    for s in range(N):
        for w1, w2 in itertools.combinations(range(N), 2):
            a, b = st[(s, w1)], st[(s, w2)]
            assert not set(i[a]) & set(i[b]) and not set(j[a]) & set(j[b])     # disjoint rows and columns
        assert sorted((w + s) % N for w in range(N)) == list(range(N))          # every column block used once


def test_blocked_epoch_equals_plain_steps_over_the_same_cell_order_and_localizes_every_block():
    """The schedule changes WHERE parameters live and the ORDER of the cells, nothing else: the parameters after a
    blocked epoch equal those of plain minibatch steps over the cells in stratum order (location transparency),
    and after subepoch s worker w owns column block (w + s) mod N."""
    rng = np.random.default_rng(3)
    rows, cols, N, L, batch = 24, 16, 4, 5, 7
    K = rows + cols
    i, j = rng.integers(0, rows, size=300), rng.integers(0, cols, size=300)
    v = rng.normal(size=300).astype(np.float32)
    init = rng.normal(0, 0.3, size=(K, L)).astype(np.float32)
    a, b = OracleStore(K, L, N, K), OracleStore(K, L, N, K)
    a.set_rows(np.arange(K), init)
    b.set_rows(np.arange(K), init)
    dsgd.run_epoch(a, i, j, v, rows, cols, N, batch, 0.05, 0.01)
    st = dsgd.strata(i, j, rows, cols, N)
    for s in range(N):
        for w in range(N):
            idx = st[(s, w)]
            for t in range(0, len(idx), batch):
                part = idx[t:t + batch]
                b.step_mf(i[part], j[part], v[part], rows, 0.05, 0.01)
    assert (a.rows == b.rows).all() and a.loss[0] == b.loss[0]
    size = -(-cols // N)
    s = N - 1
    for w in range(N):
        blk = (w + s) % N
        keys = rows + np.arange(blk * size, min((blk + 1) * size, cols))
        assert (a.owner[keys] == w).all()
    assert (a.owner[:rows] == np.arange(rows) // (-(-rows // N))).all()          # row block w lives with worker w
