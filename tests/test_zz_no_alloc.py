"""ps_push_static, the push for callers that may not allocate, against ps_push.

The entry point exists for embedders that cannot call cudaMalloc when they need
a push (all GPU memory already in the host application's pool, a fixed memory
budget, a loop that cannot take an allocation's device-wide synchronisation).
It keeps its scratch in a static device array, so the things to check are: the
result equals ps_push's, a second call right after the first is as good as the
first (the array keeps the first call's leftovers), and its limits are
enforced.  Collected last on purpose.
"""
import numpy as np
import pytest
import torch

import paper_2002_00655_b200 as ps
from tests.util import close, dev, make_pair

pytestmark = pytest.mark.gpu


def test_push_static_matches_push_on_two_calls_in_a_row():
    K, L, N, S = 6000, 100, 4, 2000
    a, _ = make_pair(K, L, N, S, max_batch_keys=1 << 14, seed=5)
    b, o = make_pair(K, L, N, S, max_batch_keys=1 << 14, seed=5)
    moved = np.arange(0, 900, 3)
    b.localize(2, dev(moved))                                   # a table that is not the initial one
    a.localize(2, dev(moved))
    o.localize(2, moved)
    a.sync(); b.sync()
    # the first use of a kernel loads its code onto the device (lazy module loading), which is not the call's doing:
    # one push of a zero row first, so that the checks below see the entry point alone
    assert ps.ps_push_static(b.store, b.table, K, L, S, dev(np.zeros(1, np.int64)), dev(np.zeros((1, L), np.float32))) == ps.PS_OK
    rng = np.random.default_rng(9)
    for n in (ps.PS_PUSH_STATIC_MAX_KEYS, 4097):       # the maximum size, then a ragged one
        keys = rng.integers(0, K, size=n)
        keys[rng.random(n) < 0.25] = 4321                       # a segment that spans many tiles
        upd = rng.normal(size=(n, L)).astype(np.float32)
        d_keys, d_upd = dev(keys), dev(upd)                     # every input exists before the call that may not allocate
        a.push(d_keys, d_upd)
        a.sync()
        torch.cuda.synchronize()
        free_before, held_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        code = ps.ps_push_static(b.store, b.table, K, L, S, d_keys, d_upd)
        assert code == ps.PS_OK
        # the property the entry point exists for: the call took no device memory, from the driver or from torch
        assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == held_before
        o.push(keys, upd)
        ra, rb = a.export(table=False)[0].numpy(), b.export(table=False)[0].numpy()
        assert close(ra, rb).all()
        assert (ra == rb).all()                                 # same kernels, same order of sums
        assert close(rb, o.rows).all()                          # ... and both are the oracle's push


def test_push_static_after_a_failed_call_of_the_maximum_size():
    """A call that fails on the device leaves the shared array full of its leftovers (sorted keys, the list of
    border-crossing segments, parked partial sums); the next call must not see any of it."""
    K, L, N, S = 5000, 64, 2, 2500
    a, _ = make_pair(K, L, N, S, max_batch_keys=1 << 14, seed=6)
    b, _ = make_pair(K, L, N, S, max_batch_keys=1 << 14, seed=6)
    rng = np.random.default_rng(10)
    n = ps.PS_PUSH_STATIC_MAX_KEYS
    keys = rng.integers(0, K, size=n)
    keys[rng.random(n) < 0.3] = 77                              # long segments: many parked partials
    keys[n // 2] = K                                            # one key out of range: the whole call is a no-op
    before = b.export(table=False)[0].numpy().copy()
    code = ps.ps_push_static(b.store, b.table, K, L, S, dev(keys), dev(rng.normal(size=(n, L)).astype(np.float32)))
    assert code == ps.PS_ERR_KEY_RANGE
    assert (b.export(table=False)[0].numpy() == before).all()
    n = 3001                                                    # ragged
    keys = rng.integers(0, K, size=n)
    keys[rng.random(n) < 0.3] = 77
    upd = rng.normal(size=(n, L)).astype(np.float32)
    assert ps.ps_push_static(b.store, b.table, K, L, S, dev(keys), dev(upd)) == ps.PS_OK
    a.push(dev(keys), dev(upd))
    a.sync()
    assert (a.export(table=False)[0].numpy() == b.export(table=False)[0].numpy()).all()


def test_push_static_enforces_its_limits_and_reports_bad_keys():
    K, L = 500, 8
    g, o = make_pair(K, L)
    before = g.export(table=False)[0].numpy().copy()
    big = ps.PS_PUSH_STATIC_MAX_KEYS + 1
    code = ps.ps_push_static(g.store, g.table, K, L, g.S, dev(np.zeros(big, np.int64)), dev(np.zeros((big, L), np.float32)))
    assert code == ps.PS_ERR_WORKSPACE
    wide_len = ps.PS_PUSH_STATIC_MAX_ROW_LEN + 4
    wide = torch.zeros(4 * wide_len, dtype=torch.float32, device="cuda")
    code = ps.ps_push_static(wide, g.table, 4, wide_len, 4, dev(np.zeros(1, np.int64)),
                             dev(np.zeros((1, wide_len), np.float32)))
    assert code == ps.PS_ERR_UNSUPPORTED
    code = ps.ps_push_static(g.store, g.table, K, L, g.S, dev(np.array([3, K, 5])), dev(np.ones((3, L), np.float32)))
    assert code == ps.PS_ERR_KEY_RANGE
    assert (g.export(table=False)[0].numpy() == before).all()
    code = ps.ps_push_static(g.store, g.table, K, L, g.S, dev(np.array([3, 3, 5])), dev(np.ones((3, L), np.float32)))
    assert code == ps.PS_OK                                     # the failed call left nothing behind
    o.push([3, 3, 5], np.ones((3, L), np.float32))
    assert (g.export(table=False)[0].numpy() == o.rows).all()
