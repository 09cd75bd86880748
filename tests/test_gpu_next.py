"""GPU parity of the sparse-map front end (ps_keymap_*) and of the parameter-blocking epoch (ps_dsgd_epoch_mf)."""
import numpy as np
import pytest
import torch

import paper_2002_00655_b200 as ps
from oracle import ABSENT, KeyMapFull, OracleKeyMap, OracleStore, dsgd
from synth import workloads as W
from tests.util import assert_close, close, compare_state, dev, make_pair

pytestmark = pytest.mark.gpu


def u64(a):
    return torch.from_numpy(np.asarray(a, dtype=np.uint64).view(np.int64)).cuda()


def as_u64(t):
    return t.cpu().numpy().view(np.uint64)


@pytest.mark.parametrize("capacity,n,universe,seed", [(5000, 3000, 4000, 0), (200_000, 70_001, 150_000, 1), (64, 300, 50, 2)])
def test_keymap_dense_keys_match_the_oracle_bit_for_bit(capacity, n, universe, seed):
    rng = np.random.default_rng(seed)
    names = rng.integers(0, 2**64 - 1, size=universe, dtype=np.uint64)          # the sparse keys in use
    g, o = ps.KeyMap(capacity, max_batch_keys=n), OracleKeyMap(capacity)
    for call in range(6):
        pick = (rng.zipf(1.2, size=n) - 1) % universe if call % 2 else rng.integers(0, universe, size=n)
        keys = names[pick]
        got = g.insert(u64(keys))
        code, size = g.sync()
        assert code == ps.PS_OK
        assert (as_u64(got) == o.insert(keys)).all(), f"insert call {call}"
        assert size == len(o)
    probe = np.concatenate([names[:100], rng.integers(0, 2**64 - 1, size=100, dtype=np.uint64)])
    assert (as_u64(g.lookup(u64(probe))) == o.lookup(probe)).all()


def test_keymap_full_and_reserved_key_add_nothing():
    g, o = ps.KeyMap(100, max_batch_keys=4096), OracleKeyMap(100)
    first = np.arange(1000, 1090, dtype=np.uint64) * np.uint64(2654435761)
    assert (as_u64(g.insert(u64(first))) == o.insert(first)).all()
    over = np.concatenate([first[:5], np.arange(5000, 5030, dtype=np.uint64)])  # 30 new keys, room for 10
    out = g.insert(u64(over))
    code, size = g.sync()
    assert code == ps.PS_ERR_CAPACITY and size == 90 and (as_u64(out) == ABSENT).all()
    try:
        o.insert(over)
        raise AssertionError("the oracle should refuse the call too")
    except KeyMapFull:
        pass
    assert (as_u64(g.lookup(u64(over))) == o.lookup(over)).all()                # none of the 30 stayed behind
    bad = np.array([7, 2**64 - 1, 8], dtype=np.uint64)                          # the reserved key
    g.insert(u64(bad))
    code, size = g.sync()
    assert code == ps.PS_ERR_KEY_RANGE and size == 90
    assert (as_u64(g.lookup(u64(bad))) == ABSENT).all()
    fit = np.arange(5000, 5010, dtype=np.uint64)
    assert (as_u64(g.insert(u64(fit))) == o.insert(fit)).all()
    assert g.sync() == (ps.PS_OK, 100)


def test_store_behind_a_keymap_serves_sparse_keys():
    """push, localize and pull through the map against the oracle's map in front of the oracle's store."""
    rng = np.random.default_rng(4)
    cap, L, N = 6000, 16, 4
    names = rng.integers(0, 2**63, size=5000, dtype=np.uint64)
    g, o = make_pair(cap, L, N, cap, max_batch_keys=4096)
    gm, om = ps.KeyMap(cap, max_batch_keys=4096), OracleKeyMap(cap)
    for it in range(8):
        keys = names[(rng.zipf(1.3, size=4000) - 1) % len(names)]
        upd = rng.integers(-2, 3, size=(4000, L)).astype(np.float32)
        d = gm.insert(u64(keys))
        g.push(d, dev(upd))
        o.push(om.insert(keys), upd)
        g.localize(it % N, d[:700])
        o.localize(it % N, om.lookup(keys[:700]))
    g.sync()
    assert gm.sync()[0] == ps.PS_OK
    compare_state(g, o, exact_rows=True, what="store behind a key map")
    probe = np.array(om.sparse_of[:300], dtype=np.uint64)       # keys that were inserted
    got = g.pull(gm.lookup(u64(probe))).cpu().numpy()
    assert (got == o.pull(om.lookup(probe))).all()


@pytest.mark.parametrize("rows,cols,N,L,n,batch,max_keys", [(4000, 1000, 4, 32, 20_000, 512, 1024), (900, 700, 8, 100, 9_000, 300, 600),
                                                           (50_000, 3_000, 8, 100, 60_000, 2048, 4096)])
def test_parameter_blocking_epoch_matches_the_oracle_schedule(rows, cols, N, L, n, batch, max_keys):
    cfg = W.MFConfig("t", rows, cols, L, n, batch, 0.002, 0.05, 0.1, 0.5, 1.1)
    K = rows + cols
    init = W.mf_init_rows(cfg, 0, K, "cpu")
    i, j, v = W.mf_cells(cfg, W.mf_planted(cfg, "cpu"), 0, n, "cpu")
    S = 2 * (-(-K // N))
    g, o = make_pair(K, L, N, S, rows=init, max_batch_keys=max(max_keys, 2 * batch))   # blocks larger than one relocation call
    ps.ps_set_pipelining(g.h, True)
    si, sj, sv, off = W.mf_stratify(i, j, v, rows, cols, N)
    ps.ps_dsgd_epoch_mf(g.h, si.cuda(), sj.cuda(), sv.cuda(), off, rows, cols, batch, cfg.lr, cfg.lam, g.loss)
    dsgd.run_epoch(o, i.numpy(), j.numpy(), v.numpy(), rows, cols, N, batch, cfg.lr, cfg.lam)
    g.sync()
    compare_state(g, o, what="parameter-blocking epoch")
    assert close(float(g.loss.cpu()[0]), o.loss[0])
    # the strata of the regrouped arrays are the oracle's, cell for cell
    st = dsgd.strata(i.numpy(), j.numpy(), rows, cols, N)
    for s in range(N):
        for w in range(N):
            lo, hi = int(off[s * N + w]), int(off[s * N + w + 1])
            assert (si[lo:hi].numpy() == i.numpy()[st[(s, w)]]).all() and (sj[lo:hi].numpy() == j.numpy()[st[(s, w)]]).all()
