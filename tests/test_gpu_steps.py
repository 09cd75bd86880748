"""GPU parity: the three fused training steps through the C-ABI against the CPU oracle.

Two modes: single-step (the oracle's pre-step state is loaded into the GPU store,
one step runs on both, every row is compared) and free-running (both sides train
side by side; rows, tables and the epoch loss are compared at the end).
"""
import numpy as np
import pytest
import torch

import paper_2002_00655_b200 as ps
from synth import workloads as W
from tests.util import assert_close, close, compare_state, dev, make_pair

pytestmark = pytest.mark.gpu


def loss_of(g):
    return float(g.loss.cpu()[0])


# ------------------------------------------------------------------ MF ----
def mf_data(cfg):
    planted = W.mf_planted(cfg, "cpu")
    return W.mf_cells(cfg, planted, 0, cfg.n_cells, "cpu")


MF_PATHS = [ps.PS_MF_SYMMETRIC, ps.PS_MF_BY_COLUMN]      # both sets of kernels on every small case (auto picks by size)


@pytest.mark.parametrize("path", MF_PATHS)
def test_mf_tiny_epoch_free_running_and_localize_transparency(path):
    cfg = W.MF_TINY
    rows = W.mf_init_rows(cfg, 0, cfg.num_keys, "cpu")
    i, j, v = mf_data(cfg)
    g, o = make_pair(cfg.num_keys, cfg.rank, rows=rows, max_batch_keys=2 * cfg.batch)
    g2, _ = make_pair(cfg.num_keys, cfg.rank, 8, cfg.num_keys, rows=rows,
                      max_batch_keys=2 * cfg.batch)           # same run with relocations in between
    ps.ps_set_mf_path(g.h, path)
    ps.ps_set_mf_path(g2.h, path)
    di, dj, dv = i.cuda(), j.cuda(), v.cuda()
    rng = np.random.default_rng(0)
    for b in range(cfg.n_batches):
        s, c = cfg.batch_range(b)
        ps.ps_step_mf(g.h, di[s:s + c], dj[s:s + c], dv[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam, g.loss)
        ps.ps_step_mf(g2.h, di[s:s + c], dj[s:s + c], dv[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam, g2.loss)
        g2.localize(int(rng.integers(0, 8)), dev(rng.integers(0, cfg.num_keys, size=150)))
        o.step_mf(i[s:s + c], j[s:s + c], v[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam)
    g.sync()
    g2.sync()
    compare_state(g, o, what="mf_tiny epoch")
    assert close(loss_of(g), o.loss[0]), (loss_of(g), o.loss[0])
    r1, r2 = g.export(table=False)[0], g2.export(table=False)[0]
    assert (r1 == r2).all(), "relocations changed the parameters (location transparency, Section 2.3)"
    assert loss_of(g) == loss_of(g2)
    assert ps.ps_rows_moved(g2.h) > 1000


@pytest.mark.parametrize("R,Cc,L,n,zipf", [(3000, 500, 100, 5000, 1.1), (400, 300, 8, 1024, None), (1000, 50, 128, 2047, 1.1),
                                           (200, 200, 260, 999, None), (90, 70, 640, 300, 1.1),
                                           (200_000, 300, 100, 6000, 1.1), (50_000, 40, 64, 3000, 1.3),
                                           (7, 5000, 24, 1500, None)])
@pytest.mark.parametrize("path", MF_PATHS)
def test_mf_single_steps(R, Cc, L, n, zipf, path):
    cfg = W.MFConfig("t", R, Cc, L, 4 * n, n, 0.002, 0.05, 0.1, 0.5, zipf)
    rows = W.mf_init_rows(cfg, 0, cfg.num_keys, "cpu")
    i, j, v = mf_data(cfg)
    g, o = make_pair(cfg.num_keys, L, rows=rows, max_batch_keys=2 * n)
    ps.ps_set_mf_path(g.h, path)
    for b in range(cfg.n_batches):
        s, c = cfg.batch_range(b)
        if b == cfg.n_batches - 1:
            c = c - 37                                           # ragged last batch
        g.set_all_rows(torch.from_numpy(o.rows.copy()))         # oracle's pre-step state
        g.loss.zero_(); o.loss[0] = 0
        ps.ps_step_mf(g.h, i[s:s + c].cuda(), j[s:s + c].cuda(), v[s:s + c].cuda(), cfg.col_key_base, cfg.lr, cfg.lam, g.loss)
        o.step_mf(i[s:s + c], j[s:s + c], v[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam)
        g.sync()
        compare_state(g, o, what=f"mf step {b}")
        assert close(loss_of(g), o.loss[0]), (loss_of(g), o.loss[0])


def _random_mf_shapes(count, seed):
    """Seeded shapes: few to many rows and columns (so that row keys repeat a lot, a little, or never), ranks that
    are and are not multiples of 32 values, batches that end inside a tile."""
    r = np.random.RandomState(seed)
    out = []
    for _ in range(count):
        R = int(round(10 ** r.uniform(0.5, 4.7)))
        Cc = int(round(10 ** r.uniform(0.3, 3.7)))
        L = 4 * int(r.randint(1, 33))
        n = int(r.randint(1, 4000))
        zipf = None if r.rand() < 0.4 else float(r.uniform(1.05, 1.5))
        out.append((R, Cc, L, n, zipf))
    return out


@pytest.mark.parametrize("path", [ps.PS_MF_SYMMETRIC, ps.PS_MF_SYMMETRIC_ROW_COPIES, ps.PS_MF_BY_COLUMN])
def test_mf_seeded_random_shapes(path):
    """One step each on two dozen seeded shapes, every row against the oracle; the symmetric form both with the
    four-row TMA gather and with one bulk copy per row."""
    for R, Cc, L, n, zipf in _random_mf_shapes(24, 20260101):
        cfg = W.MFConfig("t", R, Cc, L, n, n, 0.002, 0.05, 0.1, 0.5, zipf)
        rows = W.mf_init_rows(cfg, 0, cfg.num_keys, "cpu")
        i, j, v = mf_data(cfg)
        g, o = make_pair(cfg.num_keys, L, rows=rows, max_batch_keys=2 * n)
        ps.ps_set_mf_path(g.h, path)
        g.loss.zero_(); o.loss[0] = 0
        ps.ps_step_mf(g.h, i.cuda(), j.cuda(), v.cuda(), cfg.col_key_base, cfg.lr, cfg.lam, g.loss)
        o.step_mf(i, j, v, cfg.col_key_base, cfg.lr, cfg.lam)
        g.sync()
        compare_state(g, o, what=f"mf {R}x{Cc} rank {L} batch {n} zipf {zipf}")
        assert close(loss_of(g), o.loss[0]), (R, Cc, L, n, zipf, loss_of(g), o.loss[0])


def test_mf_bad_index_makes_the_step_a_no_op():
    g, o = make_pair(100, 8)
    i = dev(np.array([1, 2, 60, 3]), torch.int32)               # 60 >= col_key_base
    j = dev(np.array([1, 2, 3, 4]), torch.int32)
    ps.ps_step_mf(g.h, i, j, dev(np.ones(4, np.float32)), 50, 0.1, 0.0, g.loss)
    assert g.sync(check=False) == ps.PS_ERR_KEY_RANGE
    compare_state(g, o, exact_rows=True, what="bad mf step")
    assert loss_of(g) == 0.0


# ------------------------------------------------------------- ComplEx ----
def kge_run(cfg, steps, single_step, first=0):
    rows = W.kge_init_rows(cfg, 0, cfg.num_keys, "cpu")
    g, o = make_pair(cfg.num_keys, cfg.row_len, rows=rows, max_batch_keys=(3 + cfg.n_neg) * cfg.batch)
    for b in range(first, first + steps):
        s0, c = cfg.batch_range(b)
        s, r, t, neg, side = W.kge_triples(cfg, s0, c, "cpu")
        if single_step:
            g.set_all_rows(torch.from_numpy(o.rows.copy()))
            g.loss.zero_(); o.loss[0] = 0
        ps.ps_step_kge(g.h, s.cuda(), r.cuda(), t.cuda(), neg.cuda(), side.cuda(), cfg.n_neg, cfg.rel_key_base,
                       cfg.dim, cfg.lr, cfg.eps, g.loss)
        o.step_kge(s, r, t, neg, side, cfg.rel_key_base, cfg.dim, cfg.lr, cfg.eps)
        g.sync()
        if single_step:
            compare_state(g, o, what=f"kge step {b}")
            assert close(loss_of(g), o.loss[0]), (loss_of(g), o.loss[0])
    return g, o


def test_kge_tiny_epoch_single_steps():
    cfg = W.KGE_TINY                                            # 2,000 Zipf entities: s = o and negative = s/o do occur
    s, r, t, neg, side = W.kge_triples(cfg, 0, cfg.n_triples, "cpu")
    assert (s == t).any() and ((neg == s[:, None]) | (neg == t[:, None])).any()
    kge_run(cfg, cfg.n_batches, single_step=True)


def test_kge_free_running():
    """Eight steps without re-synchronising the two sides.  A first AdaGrad step on a gradient component
    near zero, -lr g / (|g| + eps), magnifies the fp32 rounding differences the two sides carry over from
    earlier steps, so a few values in ten thousand may leave the single-step tolerance; they must stay
    rare and small, and the loss must agree."""
    cfg = W.KGE_TINY
    g, o = kge_run(cfg, 8, single_step=False)
    rows = g.export(table=False)[0].numpy()
    ok = close(rows, o.rows)
    assert (~ok).mean() <= 1e-4, (~ok).sum()
    assert np.abs(rows.astype(np.float64) - o.rows).max() <= 1e-3
    assert close(loss_of(g), o.loss[0])


# (33 and 130: an odd dimension and one above 128 take the path with finished update rows, the others gradient rows)
@pytest.mark.parametrize("dim,n_neg,batch,ents", [(100, 10, 700, 5000), (32, 1, 333, 40), (36, 29, 64, 9), (4, 0, 100, 30),
                                                  (33, 3, 200, 50), (130, 2, 90, 25), (4000, 2, 24, 20)])
def test_kge_shapes_and_heavy_key_collisions(dim, n_neg, batch, ents):
    cfg = W.scaled(W.KGE_TINY, entities=ents, relations=5, dim=dim, n_neg=n_neg, batch=batch, n_triples=3 * batch - 11)
    kge_run(cfg, cfg.n_batches, single_step=True)


def test_kge_seeded_random_shapes():
    """Single steps on a dozen seeded shapes: few entities (heavy key collisions inside a data point and across the
    batch) to many, dimensions on both sides of 128 and odd ones, zero to many negatives, ragged last batches."""
    r = np.random.RandomState(20260102)
    for _ in range(12):
        dim = int(r.choice([4, 12, 32, 33, 50, 64, 100, 128, 130, 200]))
        n_neg = int(r.randint(0, 13))
        batch = int(r.randint(1, 400))
        ents = int(round(10 ** r.uniform(0.7, 3.5)))
        cfg = W.scaled(W.KGE_TINY, entities=ents, relations=int(r.randint(1, 9)), dim=dim, n_neg=n_neg, batch=batch,
                       n_triples=2 * batch - int(r.randint(0, batch)))
        kge_run(cfg, cfg.n_batches, single_step=True)


# ---------------------------------------------------------------- SGNS ----
def sgns_run(cfg, batches, single_step, random_init):
    if random_init:
        rows = torch.from_numpy(np.random.default_rng(3).normal(0, 0.3, size=(cfg.num_keys, cfg.dim)).astype(np.float32))
    else:
        rows = W.sgns_init_rows(cfg, 0, cfg.num_keys, "cpu")
    tokens = W.sgns_tokens(cfg, 0, cfg.n_tokens, "cpu")
    occ = cfg.batch * (1 + 2 * cfg.window * (1 + cfg.n_neg))
    g, o = make_pair(cfg.num_keys, cfg.dim, rows=rows, max_batch_keys=occ)
    d_tok = tokens.cuda()
    for b in batches:
        first, n = cfg.batch_range(b)
        negs = W.sgns_negatives(cfg, first, n, "cpu")
        if single_step:
            g.set_all_rows(torch.from_numpy(o.rows.copy()))
            g.loss.zero_(); o.loss[0] = 0
        ps.ps_step_sgns(g.h, d_tok, first, n, cfg.window, negs.cuda(), cfg.n_neg, cfg.out_key_base, cfg.lr, g.loss)
        o.step_sgns(tokens, first, n, cfg.window, negs, cfg.n_neg, cfg.out_key_base, cfg.lr)
        g.sync()
        if single_step:
            compare_state(g, o, what=f"sgns step {b}")
            assert close(loss_of(g), o.loss[0]), (loss_of(g), o.loss[0])
    return g, o


def test_sgns_tiny_single_steps_cover_both_stream_ends():
    cfg = W.SGNS_TINY
    sgns_run(cfg, [0, 1, 17, cfg.n_batches - 1], single_step=True, random_init=True)


def test_sgns_tiny_free_running_from_the_standard_init():
    cfg = W.SGNS_TINY
    g, o = sgns_run(cfg, range(10), single_step=False, random_init=False)
    compare_state(g, o, what="sgns free-running")
    assert close(loss_of(g), o.loss[0])


@pytest.mark.parametrize("dim,window,n_neg,batch,T", [(300, 5, 3, 200, 650), (8, 2, 0, 64, 130), (128, 1, 5, 100, 100),
                                                      (512, 3, 2, 40, 41)])
def test_sgns_shapes(dim, window, n_neg, batch, T):
    cfg = W.scaled(W.SGNS_TINY, vocab=500, n_tokens=T, dim=dim, window=window, n_neg=n_neg, batch=batch)
    sgns_run(cfg, range(cfg.n_batches), single_step=True, random_init=True)


def test_sgns_seeded_random_shapes():
    """Single steps on a dozen seeded shapes: vector lengths on both sides of a warp's 128 values, windows of 1 to 6,
    zero to six negatives, token streams that end inside a batch (clipped windows at both ends).  First and last batch
    of each stream, from the random initial vectors: with a vocabulary of a few dozen words the summed pushes of a
    batch leave the range in which fp32 dot products agree with fp64 ones to 1e-5 within a step or two."""
    r = np.random.RandomState(20260103)
    for _ in range(12):
        dim = 4 * int(r.randint(1, 100))
        window = int(r.randint(1, 7))
        n_neg = int(r.randint(0, 7))
        batch = int(r.randint(1, 200))
        T = batch + int(r.randint(1, 2 * batch + 2))
        cfg = W.scaled(W.SGNS_TINY, vocab=int(round(10 ** r.uniform(1.7, 3.0))), n_tokens=T, dim=dim, window=window,
                       n_neg=n_neg, batch=batch)
        for b in sorted({0, cfg.n_batches - 1}):
            sgns_run(cfg, [b], single_step=True, random_init=True)


# ------------------------------------------------------- host variants ----
def test_host_batch_variants_match_the_device_calls():
    cfg = W.MF_TINY
    rows = W.mf_init_rows(cfg, 0, cfg.num_keys, "cpu")
    i, j, v = mf_data(cfg)
    a, _ = make_pair(cfg.num_keys, cfg.rank, rows=rows, max_batch_keys=2 * cfg.batch)
    b, _ = make_pair(cfg.num_keys, cfg.rank, rows=rows, max_batch_keys=2 * cfg.batch)
    h_loss = torch.zeros(1, dtype=torch.float64).pin_memory()
    for s in range(0, 5 * cfg.batch, cfg.batch):
        sl = slice(s, s + cfg.batch)
        ps.ps_step_mf(a.h, i[sl].cuda(), j[sl].cuda(), v[sl].cuda(), cfg.col_key_base, cfg.lr, cfg.lam, a.loss)
        ps.ps_step_mf_host(b.h, i[sl].pin_memory(), j[sl].pin_memory(), v[sl].pin_memory(), cfg.col_key_base, cfg.lr,
                           cfg.lam, b.loss, h_loss)
        a.sync()
        assert h_loss[0] == loss_of(a)
    assert (a.export(table=False)[0] == b.export(table=False)[0]).all()

    kc = W.KGE_TINY
    rows = W.kge_init_rows(kc, 0, kc.num_keys, "cpu")
    a, _ = make_pair(kc.num_keys, kc.row_len, rows=rows, max_batch_keys=13 * kc.batch)
    b, _ = make_pair(kc.num_keys, kc.row_len, rows=rows, max_batch_keys=13 * kc.batch)
    s, r, t, neg, side = W.kge_triples(kc, 0, kc.batch, "cpu")
    ps.ps_step_kge(a.h, s.cuda(), r.cuda(), t.cuda(), neg.cuda(), side.cuda(), kc.n_neg, kc.rel_key_base, kc.dim, kc.lr, kc.eps, a.loss)
    ps.ps_step_kge_host(b.h, s, r, t, neg.contiguous(), side.contiguous(), kc.n_neg, kc.rel_key_base, kc.dim, kc.lr, kc.eps, b.loss, h_loss)
    a.sync()
    assert h_loss[0] == loss_of(a) and (a.export(table=False)[0] == b.export(table=False)[0]).all()

    sc = W.SGNS_TINY
    rows = torch.from_numpy(np.random.default_rng(1).normal(0, 0.3, size=(sc.num_keys, sc.dim)).astype(np.float32))
    occ = sc.batch * (1 + 2 * sc.window * (1 + sc.n_neg))
    a, _ = make_pair(sc.num_keys, sc.dim, rows=rows, max_batch_keys=occ)
    b, _ = make_pair(sc.num_keys, sc.dim, rows=rows, max_batch_keys=occ)
    tokens = W.sgns_tokens(sc, 0, sc.n_tokens, "cpu")
    first, n = sc.batch_range(3)
    negs = W.sgns_negatives(sc, first, n, "cpu")
    ps.ps_step_sgns(a.h, tokens.cuda(), first, n, sc.window, negs.cuda(), sc.n_neg, sc.out_key_base, sc.lr, a.loss)
    lo, hi = first - sc.window, first + n + sc.window
    ps.ps_step_sgns_host(b.h, tokens[lo:hi].contiguous(), lo, first, n, sc.n_tokens, sc.window, negs, sc.n_neg,
                         sc.out_key_base, sc.lr, b.loss, h_loss)
    a.sync()
    assert h_loss[0] == loss_of(a) and (a.export(table=False)[0] == b.export(table=False)[0]).all()


# ---------------------------------------------------------- pipelining ----
@pytest.mark.parametrize("path", MF_PATHS)
def test_pipelined_mode_gives_identical_results(path):
    """ps_set_pipelining lets the key sort of step t+1 run beside step t's kernels; nothing may change."""
    cfg = W.scaled(W.MF_TINY, rows=3000, cols=400, rank=100, n_cells=40 * 2048, batch=2048, col_zipf=1.1, lr=0.0005)
    rows = W.mf_init_rows(cfg, 0, cfg.num_keys, "cpu")
    i, j, v = mf_data(cfg)
    di, dj, dv = i.cuda(), j.cuda(), v.cuda()
    out = []
    for pipelined in (False, True):
        g, _ = make_pair(cfg.num_keys, cfg.rank, 4, cfg.num_keys, rows=rows, max_batch_keys=2 * cfg.batch)
        ps.ps_set_pipelining(g.h, pipelined)
        ps.ps_set_mf_path(g.h, path)
        torch.cuda.synchronize()
        rng = np.random.default_rng(1)
        for b in range(cfg.n_batches):
            s, c = cfg.batch_range(b)
            ps.ps_step_mf(g.h, di[s:s + c], dj[s:s + c], dv[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam, g.loss)
            if b % 7 == 3:
                g.localize(int(rng.integers(0, 4)), dev(rng.integers(0, cfg.num_keys, size=500)))
            if b % 11 == 5:
                keys = rng.integers(0, cfg.num_keys, size=700)
                g.push(dev(keys), dev((0.01 * rng.normal(size=(700, cfg.rank))).astype(np.float32)))
        g.sync()
        out.append((g.export()[0].numpy(), loss_of(g)))
    assert (out[0][0] == out[1][0]).all() and out[0][1] == out[1][1]
    assert np.isfinite(out[0][1])


@pytest.mark.parametrize("path", MF_PATHS)
def test_mf_pipelined_steps_with_relocations_in_between(path):
    """In pipelined mode the key sort of a step starts early and reads the location table (it writes the row
    addresses the gradient kernel uses): a localize between two steps must still be seen by the next step."""
    cfg = W.MFConfig("t", 2000, 300, 100, 6 * 1500, 1500, 0.002, 0.05, 0.1, 0.5, 1.1)
    rows = W.mf_init_rows(cfg, 0, cfg.num_keys, "cpu")
    i, j, v = mf_data(cfg)
    g, o = make_pair(cfg.num_keys, cfg.rank, 6, cfg.num_keys, rows=rows, max_batch_keys=2 * cfg.batch)
    ps.ps_set_pipelining(g.h, True)
    ps.ps_set_mf_path(g.h, path)
    di, dj, dv = i.cuda(), j.cuda(), v.cuda()
    torch.cuda.synchronize()
    rng = np.random.default_rng(3)
    for b in range(cfg.n_batches):
        s, c = cfg.batch_range(b)
        ps.ps_step_mf(g.h, di[s:s + c], dj[s:s + c], dv[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam, g.loss)
        o.step_mf(i[s:s + c], j[s:s + c], v[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam)
        # the keys of the NEXT batch move to another partition before it runs
        nxt = np.concatenate([i[s + c:s + 2 * c].numpy().astype(np.int64),
                              cfg.col_key_base + j[s + c:s + 2 * c].numpy().astype(np.int64)])
        if len(nxt):
            w = int(rng.integers(0, 6))
            g.localize(w, dev(nxt))
            o.localize(w, nxt)
    g.sync()
    compare_state(g, o, what="pipelined mf with relocations")
    assert close(loss_of(g), o.loss[0]), (loss_of(g), o.loss[0])


@pytest.mark.parametrize("path", MF_PATHS)
@pytest.mark.parametrize("graph", [False, True])
def test_two_pipelined_mf_steps_right_after_a_large_localize(graph, path):
    """MF steps sort on two internal streams in turn.  After a call that rewrites the location table BOTH streams
    must wait for it before a sort that reads the table: here a localize of 100,000 keys (long enough to be still
    running when the second step's sort could start) is followed by two steps whose cells all use moved keys."""
    cfg = W.MFConfig("t", 120_000, 4_000, 32, 3 * 4096, 4096, 0.002, 0.05, 0.1, 0.5, 1.1)
    rows = W.mf_init_rows(cfg, 0, cfg.num_keys, "cpu")
    i, j, v = mf_data(cfg)
    g, o = make_pair(cfg.num_keys, cfg.rank, 4, cfg.num_keys, rows=rows, max_batch_keys=1 << 17)
    ps.ps_set_pipelining(g.h, True)
    ps.ps_set_mf_path(g.h, path)
    di, dj, dv = i.cuda(), j.cuda(), v.cuda()
    moved = np.concatenate([np.arange(0, 96_000), cfg.col_key_base + np.arange(0, 4_000)]).astype(np.int64)
    d_moved = dev(moved)

    def steps(lo, hi):
        for b in range(lo, hi):
            s, c = cfg.batch_range(b)
            ps.ps_step_mf(g.h, di[s:s + c], dj[s:s + c], dv[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam, g.loss)

    steps(0, 1)                                                  # both internal streams have been used before
    torch.cuda.synchronize()
    if graph:
        cg = torch.cuda.CUDAGraph()
        with torch.cuda.graph(cg):
            g.localize(3, d_moved)
            steps(1, 3)
        cg.replay()
    else:
        g.localize(3, d_moved)
        steps(1, 3)
    g.sync()
    s, c = cfg.batch_range(0)
    o.step_mf(i[s:s + c], j[s:s + c], v[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam)
    o.localize(3, moved)
    for b in range(1, 3):
        s, c = cfg.batch_range(b)
        o.step_mf(i[s:s + c], j[s:s + c], v[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam)
    compare_state(g, o, what="two pipelined steps after a large localize")
    assert close(loss_of(g), o.loss[0])


def test_overlapped_host_batches_give_identical_results():
    """ps_set_host_overlap: batches are copied on the library's copy stream while earlier steps run and the
    calls do not wait; parameters and every step's loss must equal those of the device-batch calls."""
    cfg = W.scaled(W.MF_TINY, rows=3000, cols=400, rank=100, n_cells=24 * 2048, batch=2048, col_zipf=1.1, lr=0.0005)
    rows = W.mf_init_rows(cfg, 0, cfg.num_keys, "cpu")
    i, j, v = mf_data(cfg)
    hi, hj, hv = i.pin_memory(), j.pin_memory(), v.pin_memory()
    a, _ = make_pair(cfg.num_keys, cfg.rank, rows=rows, max_batch_keys=2 * cfg.batch)
    losses = []
    for b in range(cfg.n_batches):
        s, c = cfg.batch_range(b)
        ps.ps_step_mf(a.h, i[s:s + c].cuda(), j[s:s + c].cuda(), v[s:s + c].cuda(), cfg.col_key_base, cfg.lr, cfg.lam, a.loss)
        a.sync()
        losses.append(loss_of(a))
    want = a.export(table=False)[0]
    for pipelined in (False, True):
        g, _ = make_pair(cfg.num_keys, cfg.rank, rows=rows, max_batch_keys=2 * cfg.batch)
        ps.ps_set_pipelining(g.h, pipelined)
        ps.ps_set_host_overlap(g.h, True)
        h_loss = torch.zeros(cfg.n_batches, dtype=torch.float64).pin_memory()
        for b in range(cfg.n_batches):
            s, c = cfg.batch_range(b)
            ps.ps_step_mf_host(g.h, hi[s:s + c], hj[s:s + c], hv[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam, g.loss,
                               h_loss[b:b + 1])
        g.sync()
        assert (h_loss.numpy() == np.array(losses)).all()
        assert (g.export(table=False)[0] == want).all()
        ps.ps_set_host_overlap(g.h, False)                      # back to calls that wait
        s, c = cfg.batch_range(0)
        ps.ps_step_mf_host(g.h, hi[s:s + c], hj[s:s + c], hv[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam, g.loss, h_loss[0:1])
        assert h_loss[0] == loss_of(g)


@pytest.mark.parametrize("path", MF_PATHS)
def test_steps_captured_into_a_graph_give_the_same_results_as_eager_calls(path):
    """The timed configuration: pipelined steps captured into one CUDA graph (the internal streams join the
    capture), replayed with one launch.  Eager calls before and after the capture use the same handle."""
    cfg = W.scaled(W.MF_TINY, rows=3000, cols=400, rank=100, n_cells=24 * 2048, batch=2048, col_zipf=1.1, lr=0.0005)
    rows = W.mf_init_rows(cfg, 0, cfg.num_keys, "cpu")
    i, j, v = mf_data(cfg)
    di, dj, dv = i.cuda(), j.cuda(), v.cuda()
    loc_keys = dev(np.random.default_rng(2).integers(0, cfg.num_keys, size=400))

    def run(g, b):
        s, c = cfg.batch_range(b)
        ps.ps_step_mf(g.h, di[s:s + c], dj[s:s + c], dv[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam, g.loss)
        if b % 5 == 2:
            g.localize(b % 4, loc_keys)                          # rewrites the table the next step's sort reads

    eager, _ = make_pair(cfg.num_keys, cfg.rank, 4, cfg.num_keys, rows=rows, max_batch_keys=2 * cfg.batch)
    graphed, o = make_pair(cfg.num_keys, cfg.rank, 4, cfg.num_keys, rows=rows, max_batch_keys=2 * cfg.batch)
    for g in (eager, graphed):
        ps.ps_set_pipelining(g.h, True)
        ps.ps_set_mf_path(g.h, path)
    for b in range(cfg.n_batches):
        run(eager, b)
    eager.sync()
    for b in range(3):                                           # eager calls, then a capture, then eager calls again
        run(graphed, b)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for b in range(3, cfg.n_batches - 2):
            run(graphed, b)
    graph.replay()
    torch.cuda.synchronize()
    for b in range(cfg.n_batches - 2, cfg.n_batches):
        run(graphed, b)
    graphed.sync()
    r_e, r_g = eager.export(), graphed.export()
    assert all((x == y).all() for x, y in zip(r_e, r_g)), "graph replay differs from eager calls"
    assert loss_of(eager) == loss_of(graphed)
    for b in range(cfg.n_batches):                               # and both agree with the oracle
        s, c = cfg.batch_range(b)
        o.step_mf(i[s:s + c], j[s:s + c], v[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam)
        if b % 5 == 2:
            o.localize(b % 4, loc_keys.cpu().numpy())
    compare_state(graphed, o, what="graph-captured MF steps")
    assert close(loss_of(graphed), o.loss[0])

    kc = W.KGE_TINY                                              # a step with a gradient kernel beside the sort
    rows = W.kge_init_rows(kc, 0, kc.num_keys, "cpu")
    a, _ = make_pair(kc.num_keys, kc.row_len, rows=rows, max_batch_keys=13 * kc.batch)
    b2, _ = make_pair(kc.num_keys, kc.row_len, rows=rows, max_batch_keys=13 * kc.batch)
    d = [t.cuda() for t in W.kge_triples(kc, 0, 6 * kc.batch, "cpu")]

    def krun(g, k):
        sl = slice(k * kc.batch, (k + 1) * kc.batch)
        ps.ps_step_kge(g.h, *(t[sl] for t in d), kc.n_neg, kc.rel_key_base, kc.dim, kc.lr, kc.eps, g.loss)

    for g in (a, b2):
        ps.ps_set_pipelining(g.h, True)
    for k in range(6):
        krun(a, k)
    a.sync()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for k in range(6):
            krun(b2, k)
    graph.replay()
    b2.sync()
    assert (a.export(table=False)[0] == b2.export(table=False)[0]).all() and loss_of(a) == loss_of(b2)
