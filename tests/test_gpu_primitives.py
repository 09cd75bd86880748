"""GPU parity: pull, push, localize through the C-ABI against the CPU oracle (Table 2, Sections 3.1-3.2)."""
import numpy as np
import pytest
import torch

from tests.util import assert_close, compare_state, dev, make_pair

pytestmark = pytest.mark.gpu


def f_row(keys, L):
    keys = np.asarray(keys, dtype=np.int64)
    return ((keys[:, None] * 31 + np.arange(L)[None, :] * 7) % 1021).astype(np.float32)


@pytest.mark.parametrize("K,L,N,n", [(5000, 100, 1, 4099), (3001, 128, 7, 10007), (640, 8, 3, 33), (900, 300, 2, 1),
                                      (2000, 400, 5, 2500), (700, 516, 1, 777), (300, 1028, 2, 500),
                                      (40, 16000, 2, 100)])     # the last: a ComplEx-4000 row (Table 3: 8000 values + AdaGrad)
def test_pull_is_bit_exact(K, L, N, n):
    g, o = make_pair(K, L, N, rows=f_row(np.arange(K), L))
    keys = np.random.default_rng(n).integers(0, K, size=n)
    keys[: min(n, 5)] = K - 1                                   # duplicates and the last key
    got = g.pull(dev(keys)).cpu().numpy()
    g.sync()
    assert (got == o.pull(keys)).all()
    assert (got == f_row(keys, L)).all()                        # recomputable without any store
    assert g.pull(dev(np.zeros(0, np.int64))).shape == (0, L)


@pytest.mark.parametrize("L", [4, 100, 128, 300, 1028])
def test_push_integer_updates_are_exact_and_order_free(L):
    K, n = 3000, 20011
    g, o = make_pair(K, L, 4, rows=f_row(np.arange(K), L), max_batch_keys=n)
    rng = np.random.default_rng(L)
    keys = rng.integers(0, K, size=n)
    keys[rng.random(n) < 0.3] = 17                              # one segment spanning hundreds of tiles
    keys[rng.random(n) < 0.05] = 2999
    upd = rng.integers(-4, 5, size=(n, L)).astype(np.float32)
    g.push(dev(keys), dev(upd))
    g.sync()
    o.push(keys, upd)
    compare_state(g, o, exact_rows=True, what="push")
    perm = rng.permutation(n)                                   # same multiset, another order: same sums
    g.push(dev(keys[perm]), dev(upd[perm]))
    g.sync()
    o.push(keys, upd)
    compare_state(g, o, exact_rows=True, what="push permuted")


@pytest.mark.parametrize("K,L,n,hot", [(4000, 100, 9001, 0.2), (1000, 128, 65, 0.0), (50000, 128, 60000, 0.1),
                                         (300, 400, 4000, 0.5), (64, 8, 31, 0.9), (64, 8, 32, 1.0),
                                         (60, 16000, 300, 0.3)])
def test_push_matches_oracle(K, L, n, hot):
    g, o = make_pair(K, L, 3, max_batch_keys=n)
    rng = np.random.default_rng(n)
    keys = rng.integers(0, K, size=n)
    keys[rng.random(n) < hot] = K // 2
    upd = rng.normal(size=(n, L)).astype(np.float32)
    for _ in range(2):
        g.push(dev(keys), dev(upd))
        o.push(keys, upd)
    g.sync()
    compare_state(g, o, what="push")


def test_push_by_atomic_adds_is_exact_on_integers_and_refuses_bad_keys():
    """The measured alternative to the sorted push: no order of adds is promised, so only integer-valued updates
    (exact in any order) are compared bit for bit; a call with a key out of range must still change nothing."""
    import paper_2002_00655_b200 as ps
    K, L, n = 3000, 100, 20_000
    g, o = make_pair(K, L, 3, rows=f_row(np.arange(K), L), max_batch_keys=64)      # the call is larger than the workspace's batch
    ps.ps_set_push_mode(g.h, ps.PS_PUSH_ATOMIC)
    rng = np.random.default_rng(3)
    keys = (rng.zipf(1.2, size=n) - 1) % K
    upd = rng.integers(-3, 4, size=(n, L)).astype(np.float32)
    g.push(dev(keys), dev(upd))
    g.sync()
    o.push(keys, upd)
    compare_state(g, o, exact_rows=True, what="atomic push")
    keys[n // 2] = K
    g.push(dev(keys), dev(upd))
    assert g.sync(check=False) == ps.PS_ERR_KEY_RANGE
    compare_state(g, o, exact_rows=True, what="atomic push with a bad key")
    ps.ps_set_push_mode(g.h, ps.PS_PUSH_SORTED)
    small = rng.normal(size=(50, L)).astype(np.float32)
    g.push(dev(keys[:50]), dev(small))
    g.sync()
    o.push(keys[:50], small)
    compare_state(g, o, what="sorted push afterwards")


def test_a_wait_that_runs_out_is_reported_and_the_handle_stays_usable():
    """Device-side waits are bounded.  The self-test call lets two blocks wait at the sort's grid barrier for an
    arrival that never comes: they give up, ps_sync reports PS_ERR_CUDA and re-arms the barrier (which was left
    mid-count), and the calls after it work as if nothing had happened, the sort in the same buffer set included."""
    import paper_2002_00655_b200 as ps
    K, L = 2000, 16
    g, o = make_pair(K, L, 2, K, max_batch_keys=4096)
    rng = np.random.default_rng(12)
    for round_ in range(2):
        ps.ps_selftest_barrier_timeout(g.h)
        assert g.sync(check=False) == ps.PS_ERR_CUDA
        assert g.sync(check=False) == ps.PS_OK                  # reported once
        for _ in range(5):                                      # every buffer set comes round again
            keys = rng.integers(0, K, size=3000)
            upd = rng.integers(-2, 3, size=(3000, L)).astype(np.float32)
            g.push(dev(keys), dev(upd))
            o.push(keys, upd)
        g.localize(1, dev(keys[:500]))
        o.localize(1, keys[:500])
        g.sync()
        compare_state(g, o, exact_rows=True, what=f"after the wait ran out, round {round_}")


def test_push_and_pull_reject_bad_keys_without_touching_the_store():
    import paper_2002_00655_b200 as ps
    K, L = 500, 12
    g, o = make_pair(K, L, 2)
    keys = np.array([1, 2, K, 3])
    g.push(dev(keys), dev(np.ones((4, L), np.float32)))
    assert g.sync(check=False) == ps.PS_ERR_KEY_RANGE
    assert g.sync(check=False) == ps.PS_OK                      # reading the error clears it
    compare_state(g, o, exact_rows=True, what="rejected push")
    out = g.pull(dev(keys)).cpu().numpy()
    assert g.sync(check=False) == ps.PS_ERR_KEY_RANGE
    assert (out[2] == 0).all() and (out[[0, 1, 3]] == o.pull([1, 2, 3])).all()
    with pytest.raises(ps.PSError) as e:                        # more occurrences than the workspace was sized for
        g.push(dev(np.zeros(g.max_batch_keys + 1, np.int64)), dev(np.zeros((g.max_batch_keys + 1, L), np.float32)))
    assert e.value.code == ps.PS_ERR_WORKSPACE
    with pytest.raises(ps.PSError) as e:
        g.localize(2, dev(keys[:2]))
    assert e.value.code == ps.PS_ERR_WORKER_RANGE


@pytest.mark.parametrize("K,L,N,slack,n,seed", [(5000, 16, 4, 1.5, 700, 0), (20000, 128, 8, 1.25, 6000, 1),
                                                 (1000, 4, 64, 2.0, 300, 2), (3000, 100, 3, 1.3, 2048, 3),
                                                 (120, 16000, 3, 1.5, 90, 4), (6000, 8, 1500, 2.0, 900, 5),
                                                 (4000, 32, 300, 2.0, 1200, 6), (500, 1024, 5, 1.5, 300, 7)])
def test_localize_sequences_are_bit_exact(K, L, N, slack, n, seed):
    S = int(np.ceil(slack * -(-K // N)))
    g, o = make_pair(K, L, N, S, max_batch_keys=n)
    rng = np.random.default_rng(seed)
    from oracle.ps_oracle import OracleError
    import paper_2002_00655_b200 as ps
    moved = 0
    for it in range(14):
        w = int(rng.integers(0, N))
        m = int(rng.integers(1, n + 1))
        keys = (rng.zipf(1.3, size=m) - 1) % K if it % 2 else rng.integers(0, K, size=m)
        before = o.owner.copy()
        g.localize(w, dev(keys))
        code = g.sync(check=False)
        try:
            o.localize(w, keys)
            assert code == ps.PS_OK
            moved += int((before != o.owner).sum())
        except OracleError as e:
            assert e.code == 4 and code == ps.PS_ERR_CAPACITY
        compare_state(g, o, exact_rows=True, what=f"localize call {it}")
        if it == 5:                                             # an identical second call changes nothing
            g.localize(w, dev(keys))
            assert g.sync(check=False) == code
            compare_state(g, o, exact_rows=True, what="repeated localize")
        upd = rng.integers(-2, 3, size=(m, L)).astype(np.float32)
        g.push(dev(keys), dev(upd))                             # push through the new locations
        o.push(keys, upd)
    g.sync()
    compare_state(g, o, exact_rows=True, what="after pushes")
    assert ps.ps_rows_moved(g.h) == moved
    owner, slot = o.get_location(np.arange(K))
    d_owner = torch.empty(K, dtype=torch.int32, device="cuda")
    d_slot = torch.empty(K, dtype=torch.int32, device="cuda")
    ps.ps_get_location(g.h, dev(np.arange(K)), d_owner, d_slot)
    g.sync()
    assert (d_owner.cpu().numpy().view(np.uint32) == owner).all() and (d_slot.cpu().numpy().view(np.uint32) == slot).all()


def test_localize_capacity_failure_and_bad_key_leave_everything_unchanged():
    import paper_2002_00655_b200 as ps
    K, L, N = 64, 4, 4
    g, o = make_pair(K, L, N, 18)                               # 16 keys per partition, 2 spare slots
    g.localize(0, dev(np.array([20, 21, 22, 40])))
    assert g.sync(check=False) == ps.PS_ERR_CAPACITY
    compare_state(g, o, exact_rows=True, what="over capacity")
    g.localize(0, dev(np.array([20, 20, 40, 40, 5])))           # duplicates collapse, key 5 is already local: fits
    g.sync()
    o.localize(0, [20, 20, 40, 40, 5])
    compare_state(g, o, exact_rows=True, what="at capacity")
    g.localize(1, dev(np.array([3, K + 7])))
    assert g.sync(check=False) == ps.PS_ERR_KEY_RANGE
    compare_state(g, o, exact_rows=True, what="bad key")


def test_stress_twin_pull_push_localize_loop():
    """The pull / push / localize stress loop on a scaled-down twin, every batch checked against the oracle."""
    from synth import workloads as W
    cfg = W.STRESS_TINY
    rows = W.stress_init_rows(cfg, 0, cfg.num_keys, "cpu")
    g, o = make_pair(cfg.num_keys, cfg.row_len, cfg.workers, cfg.slots_per_part, rows=rows, max_batch_keys=cfg.batch)
    for b in range(cfg.n_batches):
        keys = W.stress_keys(cfg, b, "cpu")
        upd = W.stress_updates(cfg, b, "cpu")
        got = g.pull(keys.cuda())
        g.sync()
        assert (got.cpu().numpy() == g.export(table=False)[0].numpy()[keys.numpy()]).all()   # pulled = stored, bit for bit
        g.push(keys.cuda(), upd.cuda())
        o.push(keys, upd)
        g.localize(cfg.requester(b), keys[:cfg.localize_count].cuda())
        o.localize(cfg.requester(b), keys[:cfg.localize_count])
        g.sync()
        compare_state(g, o, what=f"stress batch {b}")


def test_push_of_a_batch_that_gives_every_sort_block_several_tiles():
    """700k occurrences: more than one tile per block of the one-launch sort on any GPU, hot and cold keys."""
    K, L, n = 300_000, 4, 700_001
    g, o = make_pair(K, L, 5, K, rows=f_row(np.arange(K), L), max_batch_keys=n)      # any partition can hold every key
    rng = np.random.default_rng(7)
    keys = rng.integers(0, K, size=n)
    keys[rng.random(n) < 0.2] = 123_456                          # one key a fifth of the batch
    keys[rng.random(n) < 0.01] = K - 1
    upd = rng.integers(-3, 4, size=(n, L)).astype(np.float32)    # integer-valued: sums are exact in any order
    g.push(dev(keys), dev(upd))
    g.sync()
    o.push(keys, upd)
    compare_state(g, o, exact_rows=True, what="large push")
    g.localize(3, dev(keys[:250_000]))                           # a large localize sorts the same way
    g.sync()
    o.localize(3, keys[:250_000])
    compare_state(g, o, exact_rows=True, what="large localize")


@pytest.mark.parametrize("n", [1, 31, 32, 33, 255, 256, 257, 2047, 2048, 2049, 4095, 4097, 6145])
def test_push_sizes_around_the_sort_and_reduction_tile_borders(n):
    K, L = 777, 8
    g, o = make_pair(K, L, 2, rows=f_row(np.arange(K), L), max_batch_keys=8192)
    rng = np.random.default_rng(n)
    keys = rng.integers(0, K, size=n)
    keys[::3] = 5                                                # a segment through every tile
    upd = rng.integers(-3, 4, size=(n, L)).astype(np.float32)
    g.push(dev(keys), dev(upd))
    g.sync()
    o.push(keys, upd)
    compare_state(g, o, exact_rows=True, what=f"push of {n}")


def test_localize_of_a_million_keys_in_one_call():
    """2^20 keys in one call, mostly distinct (every block of the one-launch relocation has a span of several
    tiles), then one key more; a store of more than 1024 partitions refuses calls beyond 2^20 keys."""
    import paper_2002_00655_b200 as ps
    K, L, N, n = 2_500_000, 4, 2, 1 << 20
    g, o = make_pair(K, L, N, K, rows=f_row(np.arange(K), L), max_batch_keys=n + 1)
    rng = np.random.default_rng(21)
    keys = rng.integers(0, K, size=n)
    keys[:1000] = K - 1
    g.localize(1, dev(keys))
    g.sync()
    o.localize(1, keys)
    compare_state(g, o, exact_rows=True, what="localize of 2^20 keys")
    assert ps.ps_rows_moved(g.h) > 300_000
    more = np.concatenate([keys, keys[:1]])
    g.localize(0, dev(more))
    g.sync()
    o.localize(0, more)
    compare_state(g, o, exact_rows=True, what="localize of 2^20 + 1 keys")
    wide, _ = make_pair(4000, 4, 2000, 4, max_batch_keys=n + 1)  # the path that sorts by old owner scans in shared memory
    with pytest.raises(ps.PSError) as e:
        wide.localize(0, dev(np.concatenate([keys, keys[:1]]) % 4000))
    assert e.value.code == ps.PS_ERR_UNSUPPORTED
