"""Helpers shared by the GPU parity tests: a CUDA store and an oracle store with the same contents."""
import numpy as np
import torch

from oracle import OracleStore

RTOL, ATOL = 1e-5, 1e-6     # |gpu - cpu| <= RTOL * max(|gpu|, |cpu|) + ATOL  (fp32 parameters, epoch loss)


def close(a, b, rtol=RTOL, atol=ATOL):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return np.abs(a - b) <= rtol * np.maximum(np.abs(a), np.abs(b)) + atol


def assert_close(a, b, what="", rtol=RTOL, atol=ATOL):
    ok = close(a, b, rtol, atol)
    if not ok.all():
        a64, b64 = np.asarray(a, np.float64), np.asarray(b, np.float64)
        bad = np.argwhere(~ok)
        i = tuple(bad[0])
        raise AssertionError(f"{what}: {len(bad)} of {ok.size} values differ; first at {i}: gpu={a64[i]!r} cpu={b64[i]!r}")


def make_pair(K, L, N=1, S=None, rows=None, max_batch_keys=1 << 16, seed=0):
    """(gpu Store, OracleStore) holding identical rows (random N(0, 0.5) unless given)."""
    import paper_2002_00655_b200 as ps
    if rows is None:
        rows = torch.from_numpy(np.random.default_rng(seed).normal(0, 0.5, size=(K, L)).astype(np.float32))
    elif isinstance(rows, np.ndarray):
        rows = torch.from_numpy(rows)
    g = ps.Store(K, L, N, S, max_batch_keys=max_batch_keys)
    g.set_all_rows(rows)
    o = OracleStore(K, L, N, S)
    o.set_rows(np.arange(K), rows.numpy())
    return g, o


def dev(a, dtype=None):
    t = torch.as_tensor(np.ascontiguousarray(a)) if not torch.is_tensor(a) else a
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda().contiguous()


def compare_state(g, o, exact_rows=False, what=""):
    """Location table, free lists bit-exact; rows exact or within tolerance."""
    rows, owner, slot = g.export()
    assert (owner.numpy().view(np.uint32) == o.owner).all(), f"{what}: owner table differs"
    assert (slot.numpy().view(np.uint32) == o.slot).all(), f"{what}: slot table differs"
    stacks, tops = g.export_freelists()
    assert (tops.numpy().view(np.uint64) == o.top).all(), f"{what}: stack heights differ"
    st = stacks.numpy().view(np.uint32)
    for p in range(o.N):
        assert (st[p, :o.top[p]] == o.stack[p, :o.top[p]]).all(), f"{what}: free stack {p} differs"
    if exact_rows:
        assert (rows.numpy() == o.rows).all(), f"{what}: rows differ"
    else:
        assert_close(rows.numpy(), o.rows, f"{what}: rows")
    return rows
