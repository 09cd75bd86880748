"""GPU parity of the RESCAL step (ps_step_rescal) against the CPU oracle: single steps from the oracle's state, a few
steps free-running with relocations in between, error cases."""
import numpy as np
import pytest
import torch

import paper_2002_00655_b200 as ps
from synth import workloads as W
from tests.util import close, compare_state, dev, make_pair

pytestmark = pytest.mark.gpu


def loss_of(g):
    return float(g.loss.cpu()[0])


def rescal_rows(E, Rn, d, seed, G):
    """E entity rows, Rn * d matrix-row rows: [d values N(0, 0.3) | d accumulators uniform in [0, G)]."""
    rng = np.random.default_rng(seed)
    K = E + Rn * d
    emb = rng.normal(0, 0.3, size=(K, d))
    acc = rng.uniform(0, G, size=(K, d)) if G else np.zeros((K, d))
    return torch.from_numpy(np.concatenate([emb, acc], axis=1).astype(np.float32))


def rescal_run(d, n_neg, batch, ents, rels, steps, single_step, G=0.0, workers=1, relocate=False):
    cfg = W.scaled(W.KGE_TINY, entities=ents, relations=rels, dim=4, n_neg=n_neg, batch=batch,
                   n_triples=steps * batch - (7 if steps * batch > 7 else 0))
    K = ents + rels * d
    rows = rescal_rows(ents, rels, d, 5, G)
    g, o = make_pair(K, 2 * d, workers, K if workers > 1 else None, rows=rows, max_batch_keys=(2 + n_neg + d) * batch)
    rng = np.random.default_rng(1)
    for b in range(cfg.n_batches):
        s0, c = cfg.batch_range(b)
        s, r, t, neg, side = W.kge_triples(cfg, s0, c, "cpu")
        if single_step:
            g.set_all_rows(torch.from_numpy(o.rows.copy()))
            g.loss.zero_(); o.loss[0] = 0
        ps.ps_step_rescal(g.h, s.cuda(), r.cuda(), t.cuda(), neg.cuda(), side.cuda(), n_neg, ents, d, 0.1, 1e-8, g.loss)
        o.step_rescal(s, r, t, neg, side, ents, d, 0.1, 1e-8)
        if relocate:
            keys = rng.integers(0, K, size=200)
            w = int(rng.integers(0, workers))
            g.localize(w, dev(keys))
            o.localize(w, keys)
        g.sync()
        if single_step:
            compare_state(g, o, what=f"rescal step {b}")
            assert close(loss_of(g), o.loss[0]), (loss_of(g), o.loss[0])
    return g, o


# (dimension, negatives, batch, entities, relations): the paper's dimension 100 with 10 negatives; tiny and maximal
# dimensions; no negatives; many negatives over nine entities (slots of a data point share keys all the time)
@pytest.mark.parametrize("d,n_neg,batch,ents,rels", [(100, 10, 96, 3000, 20), (8, 1, 333, 40, 3), (36, 29, 64, 9, 2),
                                                    (4, 0, 100, 30, 1), (128, 3, 50, 50, 4)])
@pytest.mark.parametrize("G", [0.0, 0.5])
def test_rescal_single_steps(d, n_neg, batch, ents, rels, G):
    rescal_run(d, n_neg, batch, ents, rels, steps=3, single_step=True, G=G)


def test_rescal_seeded_random_shapes():
    """Single steps on a dozen seeded shapes: every fourth dimension up to 128, zero to 29 negatives, few to many
    entities (slots of a data point that share a key), one to nine relations."""
    r = np.random.RandomState(20260104)
    for _ in range(12):
        d = 4 * int(r.randint(1, 33))
        n_neg = int(r.randint(0, 30))
        batch = int(r.randint(1, 120))
        ents = int(round(10 ** r.uniform(0.7, 3.3)))
        rescal_run(d, n_neg, batch, ents, int(r.randint(1, 10)), steps=2, single_step=True, G=float(r.choice([0.0, 0.3])))


def test_rescal_free_running_with_relocations():
    """Four steps without re-synchronising the two sides, keys relocated between the steps on a store of 8 partitions
    (location transparency, Section 2.3).  As for ComplEx, a first AdaGrad step on a gradient component near zero
    magnifies the rounding differences the sides carry over, so a few values in ten thousand may leave the single-step
    tolerance; they must stay rare and small."""
    g, o = rescal_run(16, 4, 200, 300, 5, steps=4, single_step=False, G=0.0, workers=8, relocate=True)
    rows, owner, slot = g.export()
    assert (owner.numpy().view(np.uint32) == o.owner).all() and (slot.numpy().view(np.uint32) == o.slot).all()
    ok = close(rows.numpy(), o.rows)
    assert (~ok).mean() <= 1e-4, (~ok).sum()
    assert np.abs(rows.numpy().astype(np.float64) - o.rows).max() <= 1e-3
    assert close(loss_of(g), o.loss[0])


def test_rescal_bad_index_and_unsupported_shapes():
    d, ents, rels = 8, 20, 2
    K = ents + rels * d
    g, o = make_pair(K, 2 * d, rows=rescal_rows(ents, rels, d, 0, 0.1), max_batch_keys=4096)
    s, r, t = dev(np.array([1, 2, 3]), torch.int32), dev(np.array([0, 2, 1]), torch.int32), dev(np.array([4, 5, 6]), torch.int32)
    neg, side = dev(np.array([[7], [8], [9]]), torch.int32), dev(np.array([[0], [1], [0]]), torch.uint8)
    ps.ps_step_rescal(g.h, s, r, t, neg, side, 1, ents, d, 0.1, 1e-8, g.loss)       # relation 2 of 2: past the keys
    assert g.sync(check=False) == ps.PS_ERR_KEY_RANGE
    compare_state(g, o, exact_rows=True, what="bad rescal step")
    assert loss_of(g) == 0.0
    neg_bad = dev(np.array([[7], [ents], [9]]), torch.int32)                         # a negative in the relations' range
    r_ok = dev(np.array([0, 1, 1]), torch.int32)
    ps.ps_step_rescal(g.h, s, r_ok, t, neg_bad, side, 1, ents, d, 0.1, 1e-8, g.loss)
    assert g.sync(check=False) == ps.PS_ERR_KEY_RANGE
    compare_state(g, o, exact_rows=True, what="bad rescal negative")
    with pytest.raises(Exception):
        ps.ps_step_rescal(g.h, s, r_ok, t, neg, side, 1, ents, d + 1, 0.1, 1e-8, g.loss)    # row length does not fit
    ps.ps_step_rescal(g.h, s, r_ok, t, neg, side, 1, ents, d, 0.1, 1e-8, g.loss)    # and the handle still works
    o.step_rescal(s.cpu(), r_ok.cpu(), t.cpu(), neg.cpu(), side.cpu(), ents, d, 0.1, 1e-8)
    g.sync()
    compare_state(g, o, what="rescal step after the refused ones")


def test_rescal_pipelined_ordered_and_graph_replay_agree_bit_for_bit():
    """Eight steps with relocations in between: ordered calls, pipelined calls (the key kernel and the sort of step t+1
    beside step t's kernels) and pipelined calls captured into one CUDA graph leave identical stores and losses."""
    d, n_neg, batch, ents, rels, steps = 32, 6, 300, 400, 4, 8
    cfg = W.scaled(W.KGE_TINY, entities=ents, relations=rels, dim=4, n_neg=n_neg, batch=batch, n_triples=steps * batch)
    K = ents + rels * d
    rows = rescal_rows(ents, rels, d, 9, 0.0)
    data = [tuple(t.cuda() for t in W.kge_triples(cfg, *cfg.batch_range(b), "cpu")) for b in range(steps)]
    loc_keys = dev(np.random.default_rng(4).integers(0, K, size=300))

    def run(g, b):
        ps.ps_step_rescal(g.h, *data[b], n_neg, ents, d, 0.1, 1e-8, g.loss)
        if b % 3 == 1:
            g.localize(b % 4, loc_keys)

    stores = []
    for mode in ("ordered", "pipelined", "graph"):
        g, _ = make_pair(K, 2 * d, 4, K, rows=rows, max_batch_keys=(2 + n_neg + d) * batch)
        ps.ps_set_pipelining(g.h, mode != "ordered")
        if mode != "graph":
            for b in range(steps):
                run(g, b)
        else:
            run(g, 0)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                for b in range(1, steps - 1):
                    run(g, b)
            graph.replay()
            torch.cuda.synchronize()
            run(g, steps - 1)
        g.sync()
        stores.append((g.export(), loss_of(g)))
    for (e, l), what in zip(stores[1:], ("pipelined", "graph replay")):
        assert all((x == y).all() for x, y in zip(stores[0][0], e)), f"{what} differs from ordered calls"
        assert l == stores[0][1]
