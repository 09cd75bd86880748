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
    b, _ = make_pair(K, L, N, S, max_batch_keys=1 << 14, seed=5)
    b.localize(2, dev(np.arange(0, 900, 3)))                    # a table that is not the initial one
    a.localize(2, dev(np.arange(0, 900, 3)))
    a.sync(); b.sync()
    rng = np.random.default_rng(9)
    for n in (ps.PS_PUSH_STATIC_MAX_KEYS, 4097):       # the maximum size, then a ragged one
        keys = rng.integers(0, K, size=n)
        keys[rng.random(n) < 0.25] = 4321                       # a segment that spans many tiles
        upd = rng.normal(size=(n, L)).astype(np.float32)
        a.push(dev(keys), dev(upd))
        a.sync()
        code = ps.ps_push_static(b.store, b.table, K, L, S, dev(keys), dev(upd))
        assert code == ps.PS_OK
        ra, rb = a.export(table=False)[0].numpy(), b.export(table=False)[0].numpy()
        assert close(ra, rb).all()
        assert (ra == rb).all()                                 # same kernels, same order of sums


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
