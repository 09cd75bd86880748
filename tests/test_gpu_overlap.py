"""Pre-localization beside a running call (ps_localize_beside): the keys of the next batch are relocated on a second
stream while the current batch is processed.  The result must be exactly that of the same calls made one after the
other on one stream, which in turn is the oracle's sequential order."""
import numpy as np
import pytest
import torch

import paper_2002_00655_b200 as ps
from synth import workloads as W
from tests.util import close, compare_state, dev, make_pair

pytestmark = pytest.mark.gpu


def same_state(a, b, what):
    ra, rb = a.export(), b.export()
    assert all((x == y).all() for x, y in zip(ra, rb)), f"{what}: rows or table differ"
    sa, ta = a.export_freelists()
    sb, tb = b.export_freelists()
    assert (ta == tb).all(), f"{what}: stack heights differ"
    for p in range(a.N):
        assert (sa[p, :ta[p]] == sb[p, :tb[p]]).all(), f"{what}: free stack {p} differs"


@pytest.mark.parametrize("pipelined", [False, True])
def test_push_loop_with_the_next_batch_localized_beside_the_push(pipelined):
    cfg = W.scaled(W.STRESS_TINY, num_keys=300_000, workers=8, batch=40_000, n_batches=10, localize_count=8_000, slack=1.5)
    rows = W.stress_init_rows(cfg, 0, cfg.num_keys, "cpu")
    ref, o = make_pair(cfg.num_keys, cfg.row_len, cfg.workers, cfg.slots_per_part, rows=rows, max_batch_keys=cfg.batch)
    g, _ = make_pair(cfg.num_keys, cfg.row_len, cfg.workers, cfg.slots_per_part, rows=rows, max_batch_keys=cfg.batch)
    for s in (ref, g):
        ps.ps_set_pipelining(s.h, pipelined)
    keys = [W.stress_keys(cfg, b, "cuda") for b in range(cfg.n_batches + 1)]
    upd = W.stress_updates(cfg, 0, "cuda")
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    for b in range(cfg.n_batches):
        nxt = keys[b + 1][:cfg.localize_count]
        ref.push(keys[b], upd)
        ref.localize(cfg.requester(b), nxt)
        g.push(keys[b], upd)
        ps.ps_localize_beside(g.h, cfg.requester(b), nxt, side)
        o.push(keys[b].cpu().numpy(), upd.cpu().numpy())
        o.localize(cfg.requester(b), nxt.cpu().numpy())
        if b % 4 == 1:                                          # a call that sorts nothing in between: the next relocation has nothing to run beside
            out = g.pull(keys[b][:100])
            ref.pull(keys[b][:100])
            ps.ps_localize_beside(g.h, (b + 3) % cfg.workers, keys[b][:500], side)
            ref.localize((b + 3) % cfg.workers, keys[b][:500])
            o.localize((b + 3) % cfg.workers, keys[b][:500].cpu().numpy())
    ref.sync()
    g.sync()
    same_state(ref, g, "relocations beside the pushes")
    compare_state(g, o, what="relocations beside the pushes, against the oracle")
    sr, sg = ps.ps_localize_stats(ref.h), ps.ps_localize_stats(g.h)
    assert sr["moved"] == sg["moved"] == ps.ps_rows_moved(g.h) and sr["moved"] > 10_000
    assert sr["requested"] == sg["requested"] and sr["already_local"] == sg["already_local"]
    assert sr["moved_again"] == sg["moved_again"] > 0
    assert sr["deferred"] == 0 and 0 < sg["deferred"] < sg["moved"]      # keys of the next batch that the running push also touches


@pytest.mark.parametrize("path", [ps.PS_MF_SYMMETRIC, ps.PS_MF_BY_COLUMN])
def test_mf_steps_with_the_next_batch_localized_beside_the_step(path):
    cfg = W.MFConfig("t", 60_000, 3_000, 100, 8 * 4096, 4096, 0.002, 0.05, 0.1, 0.5, 1.1)
    rows = W.mf_init_rows(cfg, 0, cfg.num_keys, "cpu")
    planted = W.mf_planted(cfg, "cpu")
    i, j, v = W.mf_cells(cfg, planted, 0, cfg.n_cells, "cpu")
    plain, o = make_pair(cfg.num_keys, cfg.rank, 8, cfg.num_keys, rows=rows, max_batch_keys=2 * cfg.batch)    # no relocations at all
    g, _ = make_pair(cfg.num_keys, cfg.rank, 8, cfg.num_keys, rows=rows, max_batch_keys=2 * cfg.batch)
    for s in (plain, g):
        ps.ps_set_pipelining(s.h, True)
        ps.ps_set_mf_path(s.h, path)
    di, dj, dv = i.cuda(), j.cuda(), v.cuda()
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    for b in range(cfg.n_batches):
        s, c = cfg.batch_range(b)
        ps.ps_step_mf(plain.h, di[s:s + c], dj[s:s + c], dv[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam, plain.loss)
        ps.ps_step_mf(g.h, di[s:s + c], dj[s:s + c], dv[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam, g.loss)
        o.step_mf(i[s:s + c], j[s:s + c], v[s:s + c], cfg.col_key_base, cfg.lr, cfg.lam)
        if b + 1 < cfg.n_batches:                               # the next batch's keys move to worker (b + 1) mod 8 meanwhile
            s2, c2 = cfg.batch_range(b + 1)
            nxt = torch.cat([di[s2:s2 + c2].to(torch.int64), cfg.col_key_base + dj[s2:s2 + c2].to(torch.int64)])
            ps.ps_localize_beside(g.h, (b + 1) % 8, nxt, side)
            o.localize((b + 1) % 8, nxt.cpu().numpy())
    plain.sync()
    g.sync()
    assert (plain.export(table=False)[0] == g.export(table=False)[0]).all(), "relocations changed the parameters"
    assert float(plain.loss.cpu()[0]) == float(g.loss.cpu()[0])
    compare_state(g, o, what="mf with pre-localization")
    assert close(float(g.loss.cpu()[0]), o.loss[0])
    st = ps.ps_localize_stats(g.h)
    assert st["deferred"] > 0 and st["moved"] > st["deferred"]
