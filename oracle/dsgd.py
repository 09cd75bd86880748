"""CPU oracle of the parameter-blocking schedule for matrix factorization.  Test infrastructure only.

Section 2.2 ("parameter blocking") and Appendix A of the paper: N workers; the rows of the matrix (and the row
factors) are split into N blocks, worker w works on row block w throughout; the columns are split into N blocks
too; an epoch has N subepochs; in subepoch s worker w works on column block (w + s) mod N, localizes the
parameters of that block when the subepoch starts, and all workers meet at a barrier when it ends.  Within a
subepoch no two workers touch a common parameter.

What the schedule computes, written out step by step on an OracleStore:
    for w in 0..N-1:      localize(w, row keys of block w)          (a worker's row factors live with it throughout)
    for s in 0..N-1:
        for w in 0..N-1:  localize(w, column keys of block (w + s) mod N)
        for w in 0..N-1:  SGD minibatches (ps step semantics) over the cells of (row block w, column block (w + s) mod N),
                          in their stored order, `batch` cells at a time
The cells of a stratum are all the cells (i, j) with row_block(i) = w and col_block(j) = (w + s) mod N, in the
order in which they appear in the input arrays.  Blocks are contiguous ranges of equal size (the last one ragged):
block(x) = x // ceil(count / N).
"""
from __future__ import annotations

import numpy as np


def block_of(x, count, n_blocks):
    size = -(-count // n_blocks)
    return np.asarray(x, dtype=np.int64) // size


def strata(i, j, rows, cols, n_workers):
    """For every (subepoch s, worker w): the indices of the cells of that stratum, in input order."""
    rb, cb = block_of(i, rows, n_workers), block_of(j, cols, n_workers)
    out = {}
    for s in range(n_workers):
        for w in range(n_workers):
            out[(s, w)] = np.nonzero((rb == w) & (cb == (w + s) % n_workers))[0]
    return out


def run_epoch(store, i, j, v, rows, cols, n_workers, batch, lr, lam):
    """One epoch of the schedule on an OracleStore with rows + cols keys and n_workers partitions."""
    i, j, v = np.asarray(i), np.asarray(j), np.asarray(v)
    size = -(-cols // n_workers)
    rsize = -(-rows // n_workers)
    st = strata(i, j, rows, cols, n_workers)
    for w in range(n_workers):
        store.localize(w, np.arange(w * rsize, min((w + 1) * rsize, rows), dtype=np.int64))
    for s in range(n_workers):
        for w in range(n_workers):
            blk = (w + s) % n_workers
            lo, hi = blk * size, min((blk + 1) * size, cols)
            store.localize(w, rows + np.arange(lo, hi, dtype=np.int64))
        for w in range(n_workers):
            idx = st[(s, w)]
            for b in range(0, len(idx), batch):
                part = idx[b:b + batch]
                store.step_mf(i[part], j[part], v[part], rows, lr, lam)
