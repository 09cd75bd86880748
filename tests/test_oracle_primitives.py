"""Pins for the oracle's pull / push / localize (Table 2, Sections 2.1, 3.1, 3.2).

The checks use what the paper and arithmetic fix: values that can be recomputed
without the store, exact integer sums, the single-owner invariant, the
"requester owns the key afterwards" rule, arrival-order conflict resolution,
and an independent model that physically moves rows between per-worker lists.
"""
import itertools

import numpy as np
import pytest

from oracle import OracleStore
from oracle.ps_oracle import OracleError


def f_row(keys, L):
    """An exact function of (key, column): recomputable without the store."""
    keys = np.asarray(keys, dtype=np.int64)
    return ((keys[:, None] * 31 + np.arange(L)[None, :] * 7) % 1021).astype(np.float32)


def make(K=37, L=5, N=3, S=None):
    st = OracleStore(K, L, N, S)
    st.set_rows(np.arange(K), f_row(np.arange(K), L))
    return st


def test_range_partition_closed_form():
    st = OracleStore(10, 2, 3, 6)
    B = 4
    assert (st.owner == np.arange(10) // B).all()
    assert (st.slot == np.arange(10) % B).all()
    assert st.top.tolist() == [2, 2, 4]
    # lowest free slot on top of each stack
    for p, cnt in enumerate([4, 4, 2]):
        assert st.stack[p, st.top[p] - 1] == cnt
        assert sorted(st.stack[p, :st.top[p]].tolist()) == list(range(cnt, 6))


def test_pull_returns_row_per_occurrence():
    st = make()
    keys = np.array([3, 3, 36, 0, 17, 3])
    assert (st.pull(keys) == f_row(keys, 5)).all()
    assert st.pull([]).shape == (0, 5)


def test_push_is_cumulative_and_exact_on_integers():
    rng = np.random.default_rng(1)
    st = make(K=50, L=4, N=2)
    keys = rng.integers(0, 6, size=4000)                     # heavy duplication
    upd = rng.integers(-8, 9, size=(4000, 4)).astype(np.float32)
    before = st.rows.copy()
    st.push(keys, upd)
    want = before.astype(np.int64)
    np.add.at(want, keys, upd.astype(np.int64))
    assert (st.rows == want.astype(np.float32)).all()        # no lost update, order-free


def test_push_sums_in_double_then_rounds_once():
    st = OracleStore(2, 1, 1)
    st.set_rows([0], np.array([1.0], np.float32))
    tiny = np.float32(2.0 ** -25)                            # half an ulp of 1.0f: lost if added one by one
    st.push([0] * 4, np.full((4, 1), tiny, np.float32))
    assert st.rows[0, 0] == np.float32(1.0 + 4 * 2.0 ** -25)


def test_key_range_error_changes_nothing():
    st = make()
    before = st.rows.copy()
    with pytest.raises(OracleError) as e:
        st.push([1, 37], np.ones((2, 5), np.float32))
    assert e.value.code == 2
    assert (st.rows == before).all()
    with pytest.raises(OracleError):
        st.localize(3, [1])


def check_invariants(st):
    """A key lives at exactly one (owner, slot); occupied + free = capacity (Section 3.2: no replicas)."""
    phys = st.owner.astype(np.int64) * st.S + st.slot
    assert len(np.unique(phys)) == st.K
    assert (st.slot < st.S).all() and (st.owner < st.N).all()
    for p in range(st.N):
        free = st.stack[p, :st.top[p]].astype(np.int64)
        occ = st.slot[st.owner == p].astype(np.int64)
        assert len(np.unique(free)) == len(free)
        assert not np.intersect1d(free, occ).size
        assert len(free) + len(occ) == st.S


def test_localize_requester_owns_and_values_travel():
    st = make(K=40, L=3, N=4, S=20)
    owner0, slot0 = st.owner.copy(), st.slot.copy()
    keys = np.array([39, 5, 5, 11, 22, 0])
    st.localize(1, keys)
    assert (st.owner[keys] == 1).all()
    untouched = np.setdiff1d(np.arange(40), keys)
    assert (st.owner[untouched] == owner0[untouched]).all() and (st.slot[untouched] == slot0[untouched]).all()
    assert st.owner[11] == 1 and st.slot[11] == slot0[11]     # was already local: entry unchanged
    assert (st.pull(np.arange(40)) == f_row(np.arange(40), 3)).all()
    check_invariants(st)
    snap = (st.owner.copy(), st.slot.copy(), st.stack.copy(), st.top.copy())
    st.localize(1, keys)                                       # second identical call: no-op
    for a, b in zip(snap, (st.owner, st.slot, st.stack, st.top)):
        assert (a == b).all()


def test_localize_conflict_resolves_in_call_order():
    st = make(K=12, L=2, N=3, S=8)
    st.localize(1, [0, 1])
    st.localize(2, [1])
    assert st.owner[0] == 1 and st.owner[1] == 2
    check_invariants(st)


def test_localize_slot_policy_lowest_free_first_then_lifo():
    st = OracleStore(8, 1, 2, 6)                               # partitions of 4, two spare slots each
    st.localize(0, [6, 4])                                     # ascending: key 4 -> slot 4, key 6 -> slot 5
    assert (st.slot[4], st.slot[6]) == (4, 5)
    assert st.top[0] == 0 and st.stack[1, :st.top[1]].tolist() == [5, 4, 0, 2]
    st.localize(1, [4])                                        # takes the slot freed last (2)
    assert (st.owner[4], st.slot[4]) == (1, 2)
    assert st.stack[0, :st.top[0]].tolist() == [4]


def test_localize_capacity_failure_is_atomic():
    st = OracleStore(8, 1, 2, 5)
    snap = (st.owner.copy(), st.slot.copy(), st.stack.copy(), st.top.copy())
    with pytest.raises(OracleError) as e:
        st.localize(0, [4, 5, 6])                              # one spare slot only
    assert e.value.code == 4
    for a, b in zip(snap, (st.owner, st.slot, st.stack, st.top)):
        assert (a == b).all()
    st.localize(0, [4, 4, 4])                                  # duplicates collapse: fits
    assert st.owner[4] == 0


class ListModel:
    """Independent model: each worker holds a physical list of slots with (key, value) in them."""

    def __init__(self, K, L, N, S):
        B = -(-K // N)
        self.cells = [[None] * S for _ in range(N)]
        self.free = [[] for _ in range(N)]
        for k in range(K):
            self.cells[k // B][k % B] = (k, f_row([k], L)[0].astype(np.float64))
        for p in range(N):
            self.free[p] = [s for s in range(S - 1, -1, -1) if self.cells[p][s] is None]

    def find(self, k):
        for p, cs in enumerate(self.cells):
            for s, c in enumerate(cs):
                if c is not None and c[0] == k:
                    return p, s
        raise KeyError(k)

    def localize(self, w, keys):
        moved = [k for k in sorted(set(keys)) if self.find(k)[0] != w]
        if len(moved) > len(self.free[w]):
            return False
        new = [self.free[w].pop() for _ in moved]
        for k, ns in zip(moved, new):
            p, s = self.find(k)
            self.cells[w][ns] = self.cells[p][s]
            self.cells[p][s] = None
            self.free[p].append(s)
        return True

    def push(self, keys, upd):
        tot = {}
        for k, u in zip(keys, upd):
            tot[k] = tot.get(k, 0) + u.astype(np.float64)
        for k, u in tot.items():
            p, s = self.find(k)
            self.cells[p][s] = (k, np.float32(self.cells[p][s][1] + u).astype(np.float64))


def compare(st, model):
    for k in range(st.K):
        p, s = model.find(k)
        assert (st.owner[k], st.slot[k]) == (p, s)
        assert (st.rows[k] == model.cells[p][s][1].astype(np.float32)).all()
    for p in range(st.N):
        assert st.stack[p, :st.top[p]].tolist() == model.free[p]


@pytest.mark.parametrize("seed", range(6))
def test_random_call_sequences_match_list_model(seed):
    rng = np.random.default_rng(seed)
    K, L, N, S = 16, 2, 3, 9
    st, model = make(K, L, N, S), ListModel(K, L, N, S)
    for _ in range(40):
        op = rng.integers(0, 3)
        keys = rng.integers(0, K, size=rng.integers(0, 7))
        if op == 0:
            w = int(rng.integers(0, N))
            ok = model.localize(w, keys.tolist())
            if ok:
                st.localize(w, keys)
            else:
                with pytest.raises(OracleError):
                    st.localize(w, keys)
        elif op == 1:
            upd = rng.integers(-3, 4, size=(len(keys), L)).astype(np.float32)
            model.push(keys.tolist(), upd)
            st.push(keys, upd)
        else:
            got = st.pull(keys)
            for t, k in enumerate(keys):
                p, s = model.find(k)
                assert (got[t] == model.cells[p][s][1].astype(np.float32)).all()
        compare(st, model)
        check_invariants(st)


def test_all_short_localize_sequences_match_list_model():
    K, L, N, S = 4, 1, 2, 3
    calls = [(w, ks) for w in range(N) for ks in ([0], [3], [0, 1], [1, 2], [0, 1, 2, 3])]
    for seq in itertools.product(calls, repeat=3):
        st, model = make(K, L, N, S), ListModel(K, L, N, S)
        for w, ks in seq:
            if model.localize(w, ks):
                st.localize(w, ks)
            else:
                with pytest.raises(OracleError):
                    st.localize(w, ks)
        compare(st, model)
