"""Seeded synthetic inputs for the five workloads.

The recipes follow the experimental set-up of the paper (Section 4.1,
Table "datasets", Appendix A) at the sizes this repository is measured on:
matrix factorization on a planted low-rank matrix, ComplEx knowledge-graph
triples with sampled negatives, a skip-gram token stream with negatives, and a
pull/push/localize stress batch.  The paper's own datasets (synthetic MF
matrices, DBpedia-500k, the One Billion Word Benchmark) are not available
here; these generators stand in for them with the same shapes, value
distributions and skew.

Every array is a pure function of (seed, stream, index) -- see `rng.py` -- so a
batch can be produced without the batches before it.  Arrays are produced once
(on whichever device is asked for) and the same bytes are handed to the CUDA
library and to the CPU oracle.  No arithmetic of the training method lives
here.

Index arrays that the C interface takes as `uint32_t` are returned as
`torch.int32` (all values are below 2**31); `uint64_t` keys as `torch.int64`.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from functools import lru_cache

import torch

from . import rng

# stream ids (one per independent array)
_S_INIT = 1
_S_PLANT_P = 2
_S_PLANT_Q = 3
_S_MF_I = 4
_S_MF_J = 5
_S_MF_NOISE = 6
_S_KGE_S = 10
_S_KGE_R = 11
_S_KGE_O = 12
_S_KGE_NEG = 13
_S_KGE_SIDE = 14
_S_TOK = 20
_S_SGNS_NEG = 21
_S_STRESS_KEY = 30
_S_STRESS_UPD = 31


def _chunks(total: int, step: int):
    s = 0
    while s < total:
        yield s, min(step, total - s)
        s += step


@lru_cache(maxsize=8)
def _cdf_host(n: int, exponent: float):
    return torch.from_numpy(rng.power_law_cdf(n, exponent))


_cdf_dev_cache: dict = {}


def _cdf(n: int, exponent: float, device) -> torch.Tensor:
    key = (n, exponent, str(device))
    if key not in _cdf_dev_cache:
        _cdf_dev_cache[key] = _cdf_host(n, exponent).to(device)
    return _cdf_dev_cache[key]


def release_tables() -> None:
    """Drop cached CDF tables (they can be hundreds of MB on the device)."""
    _cdf_dev_cache.clear()
    _cdf_host.cache_clear()


# --------------------------------------------------------------------------
# Matrix factorization
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class MFConfig:
    name: str
    rows: int
    cols: int
    rank: int
    n_cells: int
    batch: int
    lr: float
    lam: float
    init_std: float
    noise_std: float
    col_zipf: float | None      # None = uniform columns
    seed: int = 0

    @property
    def num_keys(self) -> int:
        return self.rows + self.cols

    @property
    def row_len(self) -> int:
        return self.rank

    @property
    def col_key_base(self) -> int:
        return self.rows

    @property
    def n_batches(self) -> int:
        return (self.n_cells + self.batch - 1) // self.batch

    def batch_range(self, b: int) -> tuple[int, int]:
        s = b * self.batch
        return s, min(self.batch, self.n_cells - s)


MF_TINY = MFConfig("mf_tiny", 1_000, 1_000, 8, 100_000, 1_024, 0.01, 0.05, 0.1, 0.1, None)
MF_LARGE = MFConfig("mf_large", 10_000_000, 1_000_000, 100, 500_000_000, 65_536,
                    0.002, 0.05, 0.1, 0.5, 1.1)
# a fifth of the large matrix with the same minibatch: for profiler captures, which should hold little memory
MF_MEDIUM = MFConfig("mf_medium", 2_000_000, 200_000, 100, 100_000_000, 65_536,
                     0.002, 0.05, 0.1, 0.5, 1.1)


def mf_init_rows(cfg: MFConfig, key_start: int, count: int, device) -> torch.Tensor:
    """Initial factor rows for keys [key_start, key_start+count): N(0, init_std)."""
    L = cfg.rank
    idx = rng.counter(key_start * L, count * L, device)
    return rng.normal(cfg.seed, _S_INIT, idx, cfg.init_std).to(torch.float32).view(count, L)


def mf_planted(cfg: MFConfig, device, chunk_rows: int = 1 << 20):
    """Planted factors P (rows x rank), Q (cols x rank), entries N(0, rank**-1/4)."""
    std = cfg.rank ** -0.25
    out = []
    for n, stream in ((cfg.rows, _S_PLANT_P), (cfg.cols, _S_PLANT_Q)):
        m = torch.empty((n, cfg.rank), dtype=torch.float32, device=device)
        for s, c in _chunks(n, chunk_rows):
            idx = rng.counter(s * cfg.rank, c * cfg.rank, device)
            m[s:s + c] = rng.normal(cfg.seed, stream, idx, std).to(torch.float32).view(c, cfg.rank)
        out.append(m)
    return out[0], out[1]


def mf_cells(cfg: MFConfig, planted, start: int, count: int, device, chunk: int = 1 << 22):
    """Observed cells [start, start+count): (i int32, j int32, v float32)."""
    P, Q = planted
    i_out = torch.empty(count, dtype=torch.int32, device=device)
    j_out = torch.empty(count, dtype=torch.int32, device=device)
    v_out = torch.empty(count, dtype=torch.float32, device=device)
    for s, c in _chunks(count, chunk):
        idx = rng.counter(start + s, c, device)
        i = rng.uniform_int(cfg.seed, _S_MF_I, idx, cfg.rows)
        if cfg.col_zipf is None:
            j = rng.uniform_int(cfg.seed, _S_MF_J, idx, cfg.cols)
        else:
            j = rng.sample_cdf(_cdf(cfg.cols, cfg.col_zipf, device),
                               rng.uniform01(cfg.seed, _S_MF_J, idx))
        v = (P[i] * Q[j]).sum(dim=1, dtype=torch.float32)
        v = v + rng.normal(cfg.seed, _S_MF_NOISE, idx, cfg.noise_std).to(torch.float32)
        i_out[s:s + c] = i.to(torch.int32)
        j_out[s:s + c] = j.to(torch.int32)
        v_out[s:s + c] = v
    return i_out, j_out, v_out


def mf_stratify(i, j, v, rows: int, cols: int, n_workers: int):
    """Groups cells by stratum for the parameter-blocking schedule: stratum (s, w) holds the cells of row block w and
    column block (w + s) mod N (blocks are contiguous ranges of ceil(count / N)), strata in (s, w) order, the cells of
    a stratum in their input order.  Returns i, j, v regrouped and the N * N + 1 stratum boundaries (CPU int64)."""
    N = n_workers
    rb = i.to(torch.int64) // (-(-rows // N))
    cb = j.to(torch.int64) // (-(-cols // N))
    sub = (cb - rb) % N
    stratum = sub * N + rb
    order = torch.sort(stratum, stable=True).indices
    counts = torch.bincount(stratum, minlength=N * N)
    offsets = torch.zeros(N * N + 1, dtype=torch.int64)
    offsets[1:] = torch.cumsum(counts, 0).cpu()
    return i[order].contiguous(), j[order].contiguous(), v[order].contiguous(), offsets


# --------------------------------------------------------------------------
# ComplEx knowledge-graph embeddings
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class KGEConfig:
    name: str
    entities: int
    relations: int
    dim: int                    # complex dimensions; a row is [Re | Im | G_Re | G_Im]
    n_triples: int
    n_neg: int
    batch: int
    lr: float
    eps: float
    init_std: float
    ent_zipf: float
    seed: int = 0

    @property
    def num_keys(self) -> int:
        return self.entities + self.relations

    @property
    def row_len(self) -> int:
        return 4 * self.dim

    @property
    def rel_key_base(self) -> int:
        return self.entities

    @property
    def n_batches(self) -> int:
        return (self.n_triples + self.batch - 1) // self.batch

    def batch_range(self, b: int) -> tuple[int, int]:
        s = b * self.batch
        return s, min(self.batch, self.n_triples - s)


KGE = KGEConfig("kge", 500_000, 1_000, 100, 3_000_000, 10, 8_192, 0.1, 1e-8, 0.1, 1.0)
KGE_TINY = KGEConfig("kge_tiny", 2_000, 16, 12, 6_000, 10, 256, 0.1, 1e-8, 0.1, 1.0)
# The paper's ComplEx-Large (Section 4.1, Tables 4 and 5): 4000 complex dimensions, i.e. 8000 values plus 8000 AdaGrad
# accumulators per key (64 KB rows in fp32; a 32 GB store for the same 500k entities).  Minibatches of 2,048 triples:
# the update rows of a step are materialised for rows this wide, 1.7 GB at this size.
KGE_4000 = KGEConfig("kge_4000", 500_000, 1_000, 4000, 3_000_000, 10, 2_048, 0.1, 1e-8, 0.1, 1.0)
# the same rows on 20,000 entities: what the CPU oracle can hold when it is timed beside the full size
KGE_4000_TWIN = KGEConfig("kge_4000_twin", 20_000, 1_000, 4000, 3_000_000, 10, 2_048, 0.1, 1e-8, 0.1, 1.0)


def kge_init_rows(cfg: KGEConfig, key_start: int, count: int, device) -> torch.Tensor:
    """Embedding halves N(0, init_std); AdaGrad accumulator halves zero."""
    d2 = 2 * cfg.dim
    idx = rng.counter(key_start * d2, count * d2, device)
    emb = rng.normal(cfg.seed, _S_INIT, idx, cfg.init_std).to(torch.float32).view(count, d2)
    return torch.cat([emb, torch.zeros_like(emb)], dim=1).contiguous()


def kge_triples(cfg: KGEConfig, start: int, count: int, device):
    """Triples [start, start+count) and their negatives.

    Returns s, r, o (int32, [count]), neg_ent (int32, [count, n_neg]) and
    neg_side (uint8, [count, n_neg]; 0 = the negative replaces the subject,
    1 = it replaces the object).  Subjects and objects are Zipf over entities
    (rank 1 = entity 0), relations uniform, replacement entities uniform.
    """
    idx = rng.counter(start, count, device)
    cdf = _cdf(cfg.entities, cfg.ent_zipf, device)
    s = rng.sample_cdf(cdf, rng.uniform01(cfg.seed, _S_KGE_S, idx)).to(torch.int32)
    o = rng.sample_cdf(cdf, rng.uniform01(cfg.seed, _S_KGE_O, idx)).to(torch.int32)
    r = rng.uniform_int(cfg.seed, _S_KGE_R, idx, cfg.relations).to(torch.int32)
    nidx = rng.counter(start * cfg.n_neg, count * cfg.n_neg, device)
    neg = rng.uniform_int(cfg.seed, _S_KGE_NEG, nidx, cfg.entities).to(torch.int32)
    side = (rng.bits64(cfg.seed, _S_KGE_SIDE, nidx) & 1).to(torch.uint8)
    return s, r, o, neg.view(count, cfg.n_neg), side.view(count, cfg.n_neg)


# --------------------------------------------------------------------------
# RESCAL (the paper's other knowledge-graph model: entity dimension d, a d x d matrix per relation)
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class RescalConfig:
    """Triples come from kge_triples (same fields as KGEConfig).  All rows have one length, so a relation's matrix is
    `dim` keys, one per matrix row; a row is [dim values | dim AdaGrad accumulators]."""
    name: str
    entities: int
    relations: int
    dim: int
    n_triples: int
    n_neg: int
    batch: int
    lr: float
    eps: float
    init_std: float
    ent_zipf: float
    seed: int = 0

    @property
    def num_keys(self) -> int:
        return self.entities + self.relations * self.dim

    @property
    def row_len(self) -> int:
        return 2 * self.dim

    @property
    def rel_key_base(self) -> int:
        return self.entities

    @property
    def n_batches(self) -> int:
        return (self.n_triples + self.batch - 1) // self.batch

    def batch_range(self, b: int) -> tuple[int, int]:
        s = b * self.batch
        return s, min(self.batch, self.n_triples - s)


# Stand-in for the paper's RESCAL task on DBpedia-500k (Table 4: 490,598 entities and 573 relations, entity dimension
# 100, relation dimension 10,000, 10 negatives per triple): synthetic triples with Zipf entities, not the dataset.
RESCAL = RescalConfig("rescal", 500_000, 573, 100, 3_000_000, 10, 8_192, 0.1, 1e-8, 0.1, 1.0)
RESCAL_TINY = RescalConfig("rescal_tiny", 2_000, 7, 12, 3_000, 10, 128, 0.1, 1e-8, 0.1, 1.0)


def rescal_init_rows(cfg: RescalConfig, key_start: int, count: int, device) -> torch.Tensor:
    """Value halves N(0, init_std) (entities and matrix rows alike); AdaGrad accumulator halves zero."""
    d = cfg.dim
    idx = rng.counter(key_start * d, count * d, device)
    emb = rng.normal(cfg.seed, _S_INIT, idx, cfg.init_std).to(torch.float32).view(count, d)
    return torch.cat([emb, torch.zeros_like(emb)], dim=1).contiguous()


# --------------------------------------------------------------------------
# Skip-gram with negative sampling
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class SGNSConfig:
    name: str
    vocab: int
    n_tokens: int
    dim: int
    window: int
    n_neg: int
    batch: int                  # center words per step
    lr: float
    tok_zipf: float
    neg_power: float
    seed: int = 0

    @property
    def num_keys(self) -> int:
        return 2 * self.vocab

    @property
    def row_len(self) -> int:
        return self.dim

    @property
    def out_key_base(self) -> int:
        return self.vocab

    @property
    def n_batches(self) -> int:
        return (self.n_tokens + self.batch - 1) // self.batch

    def batch_range(self, b: int) -> tuple[int, int]:
        s = b * self.batch
        return s, min(self.batch, self.n_tokens - s)

    def n_ctx(self, p: int) -> int:
        """Number of context positions of center p (window clipped at the stream's ends)."""
        return min(p, self.window) + min(self.n_tokens - 1 - p, self.window)

    def pairs_before(self, p: int) -> int:
        """Number of (center, context) pairs of all centers q < p (closed form)."""
        W, T = self.window, self.n_tokens

        def left(n):            # sum_{q<n} min(q, W)
            m = min(n, W)
            return m * (m - 1) // 2 + (n - m) * W

        def right(n):           # sum_{q<n} min(T-1-q, W)
            full = max(0, min(n, T - W))            # q <= T-1-W  -> W each
            rest = n - full                         # q in [T-W, n): T-1-q each
            a = T - 1 - full                        # first term of the tail
            return full * W + rest * a - rest * (rest - 1) // 2

        return left(p) + right(p)


SGNS = SGNSConfig("sgns", 1_000_000, 100_000_000, 300, 5, 3, 32_768, 0.025, 1.0, 0.75)
SGNS_TINY = SGNSConfig("sgns_tiny", 3_000, 20_000, 20, 5, 3, 512, 0.025, 1.0, 0.75)


def sgns_init_rows(cfg: SGNSConfig, key_start: int, count: int, device) -> torch.Tensor:
    """Input vectors (keys < vocab) U(-0.5/dim, 0.5/dim); output vectors zero."""
    L = cfg.dim
    idx = rng.counter(key_start * L, count * L, device)
    u = (rng.uniform01(cfg.seed, _S_INIT, idx) - 0.5) / L
    rows = u.to(torch.float32).view(count, L)
    keys = torch.arange(key_start, key_start + count, device=device)
    rows[keys >= cfg.vocab] = 0.0
    return rows


def sgns_tokens(cfg: SGNSConfig, start: int, count: int, device, chunk: int = 1 << 24) -> torch.Tensor:
    """Tokens [start, start+count) of the stream: i.i.d. Zipf (rank 1 = word 0), int32."""
    out = torch.empty(count, dtype=torch.int32, device=device)
    cdf = _cdf(cfg.vocab, cfg.tok_zipf, device)
    for s, c in _chunks(count, chunk):
        idx = rng.counter(start + s, c, device)
        out[s:s + c] = rng.sample_cdf(cdf, rng.uniform01(cfg.seed, _S_TOK, idx)).to(torch.int32)
    return out


def sgns_negatives(cfg: SGNSConfig, first_pos: int, n_centers: int, device) -> torch.Tensor:
    """Negatives of every (center, context) pair of centers [first_pos, first_pos+n_centers).

    int32 [n_pairs * n_neg], pair-major, pairs in (center ascending, context
    position ascending) order.  Drawn from the unigram distribution raised to
    `neg_power`; unigram counts are the Zipf probabilities themselves, so the
    sampling law is a power law of exponent tok_zipf * neg_power.
    """
    p0 = cfg.pairs_before(first_pos)
    p1 = cfg.pairs_before(first_pos + n_centers)
    idx = rng.counter(p0 * cfg.n_neg, (p1 - p0) * cfg.n_neg, device)
    cdf = _cdf(cfg.vocab, cfg.tok_zipf * cfg.neg_power, device)
    return rng.sample_cdf(cdf, rng.uniform01(cfg.seed, _S_SGNS_NEG, idx)).to(torch.int32)


# --------------------------------------------------------------------------
# pull / push / localize stress
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class StressConfig:
    name: str
    num_keys: int
    row_len: int
    workers: int
    batch: int                  # keys per batch
    n_batches: int
    key_zipf: float
    localize_count: int         # the first `localize_count` keys of a batch are localized
    slack: float = 1.25         # slots_per_part = ceil(slack * ceil(K / N))
    seed: int = 0

    @property
    def part_size(self) -> int:
        return (self.num_keys + self.workers - 1) // self.workers

    @property
    def slots_per_part(self) -> int:
        return int(math.ceil(self.slack * self.part_size))

    def requester(self, b: int) -> int:
        return b % self.workers


STRESS = StressConfig("stress", 100_000_000, 128, 64, 1_000_000, 1_000, 0.9, 100_000)
STRESS_TINY = StressConfig("stress_tiny", 50_000, 128, 8, 6_000, 12, 0.9, 600)
# the stress batch (1M keys, 100k of them localized) on a store of 3 GB: for profiler captures.  Fewer workers and
# more spare slots than the full configuration, so that a partition can take 100k keys at a time.
STRESS_MEDIUM = StressConfig("stress_medium", 4_000_000, 128, 16, 1_000_000, 200, 0.9, 100_000, slack=1.5)


def stress_init_rows(cfg: StressConfig, key_start: int, count: int, device) -> torch.Tensor:
    L = cfg.row_len
    idx = rng.counter(key_start * L, count * L, device)
    return rng.normal(cfg.seed, _S_INIT, idx, 1.0).to(torch.float32).view(count, L)


def stress_keys(cfg: StressConfig, b: int, device) -> torch.Tensor:
    """Keys of batch b: int64 [batch], Zipf (rank 1 = key 0)."""
    idx = rng.counter(b * cfg.batch, cfg.batch, device)
    cdf = _cdf(cfg.num_keys, cfg.key_zipf, device)
    return rng.sample_cdf(cdf, rng.uniform01(cfg.seed, _S_STRESS_KEY, idx))


def stress_updates(cfg: StressConfig, b: int, device) -> torch.Tensor:
    """Additive updates of batch b: float32 [batch, row_len], N(0, 1)."""
    n = cfg.batch * cfg.row_len
    idx = rng.counter(b * n, n, device)
    return rng.normal(cfg.seed, _S_STRESS_UPD, idx, 1.0).to(torch.float32).view(cfg.batch, cfg.row_len)


def scaled(cfg, **kw):
    """A copy of a config with some fields replaced (scaled-down twins for tests)."""
    return replace(cfg, **kw)
