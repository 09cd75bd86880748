"""Benchmark of the parameter-store hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload mf_large] [--impl ours|reference]

A step is one pass of the whole hot path over one batch of seeded synthetic
input: for the training workloads one fused pull -> gradient -> push call
(ps_step_mf / ps_step_kge / ps_step_sgns), for the stress workload one ps_pull,
one ps_push and one ps_localize.  Default workload: matrix factorization,
10M x 1M, rank 100, minibatches of 65,536 cells.  The path does not shard
(one GPU holds the whole store), so with N > 1 every rank runs an independent
replica and the value is the sum over replicas.

Prints ONE JSON line: throughput with the batch resident in HBM (`value`),
the same through the host-buffer entry point (`e2e`), a per-kernel table with
each kernel's own bytes over its own time (`kernels`), the row of that table
with the largest share of a step as a fraction of the measured HBM copy
bandwidth (`roofline`), the same fraction for the bytes the method must move
per step over the whole timed step (`roofline_step`), and the CPU oracle timed
on a bounded sample of the same workload (`cpu_baseline`).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from synth import workloads as W

METRIC = "sgd_examples_per_sec"
FALLBACK_HBM_GBS = 6650.0


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


# ----------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons of one GPU through NVML while the timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, device_index: int):
        super().__init__(daemon=True)
        self.samples, self.reason_bits, self.max_mhz = [], 0, None
        self._halt = threading.Event()
        self.h = None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            try:
                uuid = torch.cuda.get_device_properties(device_index).uuid
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.h = None

    def run(self):
        if self.h is None:
            return
        nv = self.nv
        while not self._halt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            except Exception:
                break
            time.sleep(0.002)

    def stop(self):
        self._halt.set()
        self.join(timeout=2)
        if self.h is None or not self.samples:
            return smi_clocks()
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": [n for b, n in self.REASONS.items() if self.reason_bits & b], "samples": len(self.samples),
                "source": "nvml"}


def smi_clocks():
    try:
        out = subprocess.run(["nvidia-smi", "--query-gpu=clocks.sm,clocks.max.sm,clocks_event_reasons.active",
                              "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10).stdout
        sm, mx, reasons = [x.strip() for x in out.splitlines()[0].split(",")]
        return {"sm_mhz": float(sm), "sm_max_mhz": float(mx), "reasons": [reasons], "samples": 1,
                "source": "nvidia-smi after the timed region"}
    except Exception as e:                                     # noqa: BLE001
        return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "source": f"unavailable: {e}"}


# ----------------------------------------------------------------------------------------
# workloads
# ----------------------------------------------------------------------------------------
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/,
# keyed by (workload, kernel).  An entry is removed when its kernel changes after the capture.
TRAFFIC = {
    ("mf_large", "mf_sub_kernel<4,gather4>"): 46.1e6,                 # profiles/mf_step_kernels_ncu_full.md (same-batch twin)
    ("kge", "kge_reduce_kernel<2>"): 321.6e6,                   # profiles/kge_step_kernels_ncu_full.md
    ("rescal", "rescal_grad_kernel<4>"): 501.4e6,               # profiles/rescal_step_kernels_ncu_full.md
    ("sgns", "push_reduce_kernel<3,true>"): 1561.1e6,           # profiles/sgns_step_kernels_ncu_full.md
}


def n_unique(*tensors) -> int:
    return int(torch.unique(torch.cat([t.reshape(-1).to(torch.int64) for t in tensors])).numel())


def sort_bytes(occ, key_bits, extra=0):
    """The one-launch key sort: per pass keys and values in and out (the first pass reads no values)."""
    passes = (key_bits + 7) // 8
    return occ * (16 * passes - 4) + extra


def fixup_bytes(keys, tile, rb):
    """The launch that finishes segments (runs of one key in the sorted occurrences) crossing the borders of the
    reduction's tiles of `tile` positions: one parked fp64 partial row per tile such a segment touches, read once,
    plus the read-modify-write of the segment's row and its 16-byte list entry."""
    k = torch.sort(keys.reshape(-1).to(torch.int64)).values
    n = k.numel()
    if n == 0:
        return 0.0
    head = torch.ones(n, dtype=torch.bool, device=k.device)
    head[1:] = k[1:] != k[:-1]
    start = torch.nonzero(head).flatten()
    end = torch.cat([start[1:], torch.tensor([n], device=k.device)])
    parts = (end - 1) // tile - start // tile + 1
    cross = parts > 1
    return float(int(cross.sum()) * (2 * rb + 16) + int(parts[cross].sum()) * 2 * rb)


def kernel_bytes_of_step(batch_bytes, occ, u, rb, keys_prefix, step_prefix, key_bits, keys=None):
    """Bytes per LAUNCH that each kernel of a step call must move, by kernel-name prefix: what it reads of the
    batch, the table and the store, and what it has to write for the next kernel (keys, update rows)."""
    return {
        "push_fixup_kernel": fixup_bytes(keys, 32, rb) if keys is not None else None,
        keys_prefix: batch_bytes + occ * 4,                      # batch arrays in, one 32-bit key per occurrence out
        "sort_all_kernel": sort_bytes(occ, key_bits),
        step_prefix: batch_bytes + occ * (8 + rb) + occ * rb,    # table entry + row per occurrence in, update row out
        "push_reduce_kernel": occ * (8 + rb) + u * (8 + 2 * rb), # sorted pair + update row in; row read-modify-write
    }


class MFWorkload:
    """Matrix factorization (Section 4.1 task): cells/s through ps_step_mf."""

    def __init__(self, cfg):
        self.cfg, self.example = cfg, "cells"
        self.row_bytes = cfg.rank * 4

    def describe(self):
        c = self.cfg
        return {"workload": c.name, "rows": c.rows, "cols": c.cols, "rank": c.rank, "minibatch": c.batch,
                "store_gb": round(c.num_keys * c.rank * 4 / 1e9, 2),
                "l2": "inputs larger than L2 (random rows of the store; no flush between steps)"}

    def max_steps(self):
        return self.cfg.n_batches - 1                           # full batches only

    def gen_init(self, device, chunk=1 << 20):
        for s in range(0, self.cfg.num_keys, chunk):
            c = min(chunk, self.cfg.num_keys - s)
            yield s, W.mf_init_rows(self.cfg, s, c, device)

    def setup(self, ps, device, n_steps, keep_host_init):
        c = self.cfg
        self.ps = ps
        self.store = ps.Store(c.num_keys, c.rank, 1, max_batch_keys=2 * c.batch, device=device.index)
        self.host_init = torch.empty((c.num_keys, c.rank), dtype=torch.float32) if keep_host_init else None
        for s, rows in self.gen_init(device):
            self.store.set_rows(torch.arange(s, s + rows.shape[0], dtype=torch.int64, device=device), rows)
            if keep_host_init:
                self.host_init[s:s + rows.shape[0]] = rows.cpu()
        planted = W.mf_planted(c, device)
        self.i, self.j, self.v = W.mf_cells(c, planted, 0, n_steps * c.batch, device)
        del planted
        torch.cuda.synchronize(device)

    def units(self, k):
        return self.cfg.batch

    def side_stream_kernels(self):
        return ("sort_all_kernel",)

    def step(self, k):
        c, b = self.cfg, self.cfg.batch
        sl = slice(k * b, (k + 1) * b)
        self.ps.ps_step_mf(self.store.h, self.i[sl], self.j[sl], self.v[sl], c.col_key_base, c.lr, c.lam,
                           self.store.loss)

    def host_setup(self, steps):
        b = self.cfg.batch
        n = len(steps) * b
        lo = steps[0] * b
        self.hi_, self.hj_, self.hv_ = (t[lo:lo + n].cpu().pin_memory() for t in (self.i, self.j, self.v))
        self.h_lo = steps[0]
        self.h_loss = torch.zeros(len(steps), dtype=torch.float64).pin_memory()      # one word per step in flight
        # the batches as the caller would hold them: one view per array and step, made before the timed region
        self.h_batches = [(self.hi_[x * b:(x + 1) * b], self.hj_[x * b:(x + 1) * b], self.hv_[x * b:(x + 1) * b],
                           self.h_loss[x:x + 1]) for x in range(len(steps))]
        return b * 12, 8

    def step_host(self, k):
        c = self.cfg
        hi, hj, hv, h_loss = self.h_batches[k - self.h_lo]
        self.ps.ps_step_mf_host(self.store.h, hi, hj, hv, c.col_key_base, c.lr, c.lam, self.store.loss, h_loss)

    def alg_bytes(self, k):
        c, b = self.cfg, self.cfg.batch
        sl = slice(k * b, (k + 1) * b)
        u = n_unique(self.i[sl]) + n_unique(self.j[sl])
        return b * 12 + 2 * b * (8 + self.row_bytes) + u * 2 * self.row_bytes

    def kernel_bytes(self, k, moved=0.0):
        c, b = self.cfg, self.cfg.batch
        sl = slice(k * b, (k + 1) * b)
        u = n_unique(self.i[sl]) + n_unique(self.j[sl])
        occ, rb = 2 * b, self.row_bytes
        bits = int(c.num_keys).bit_length()
        if c.rank > 128:                                        # unfused path: update rows are materialised
            return kernel_bytes_of_step(b * 12, occ, u, rb, "mf_keys", "mf_step", bits,
                                        torch.cat([self.i[sl].to(torch.int64), c.col_key_base + self.j[sl].to(torch.int64)]))
        return {
            # batch arrays in (twice: keys, then records), two table entries per occurrence, keys and records out
            "sort_all_kernel": sort_bytes(occ, bits, extra=2 * b * 12 + occ * (16 + 4 + 16)),
            # the step's pull, gradient and push: the algorithmic bytes of the step (a table entry and a row per
            # occurrence, read + write of every distinct row); the fix-up launch only finishes segments that cross
            # tile borders and moves the few rows that had to be staged
            "mf_sub_kernel": b * 12 + occ * (8 + rb) + u * 2 * rb,
            # parked partials of the column factors whose occurrences cross tiles of 8 positions, their rows, and
            # the per-position list of staged rows (8 bytes each) it scans
            "push_fixup_kernel": fixup_bytes(c.col_key_base + self.j[sl].to(torch.int64), 8, rb) + occ * 8,
        }

    # --- oracle leg ---
    def oracle_setup(self, device):
        from oracle import OracleStore
        c = self.cfg
        o = OracleStore(c.num_keys, c.rank, 1)
        if getattr(self, "host_init", None) is not None:
            for s in range(0, c.num_keys, 1 << 20):
                e = min(s + (1 << 20), c.num_keys)
                o.set_rows(np.arange(s, e), self.host_init[s:e].numpy())
        else:
            for s, rows in self.gen_init(device):
                o.set_rows(np.arange(s, s + rows.shape[0]), rows.cpu().numpy())
        self.oracle = o
        return o

    def oracle_data(self, device, n_steps):
        if not hasattr(self, "i"):
            planted = W.mf_planted(self.cfg, device)
            self.i, self.j, self.v = W.mf_cells(self.cfg, planted, 0, n_steps * self.cfg.batch, device)
        n = n_steps * self.cfg.batch
        self.oi, self.oj, self.ov = (t[:n].cpu().numpy() for t in (self.i, self.j, self.v))

    def oracle_step(self, k, cells):
        c, b = self.cfg, self.cfg.batch
        sl = slice(k * b, k * b + cells)
        self.oracle.step_mf(self.oi[sl], self.oj[sl], self.ov[sl], c.col_key_base, c.lr, c.lam)
        return cells


class MFPushWorkload(MFWorkload):
    """ps_push alone on the key occurrences of MF-large batches (131,072 keys of 100 values per call): the shape on
    which the sorted push and the push by atomic adds (--atomic-push) are compared."""

    example = "keys"

    def __init__(self, cfg):
        super().__init__(cfg)
        self.example = "keys"

    def describe(self):
        return dict(super().describe(), workload="push_mf", call="ps_push of the batch's 2 x minibatch key occurrences")

    def setup(self, ps, device, n_steps, keep_host_init):
        super().setup(ps, device, n_steps, keep_host_init)
        c = self.cfg
        g = torch.Generator(device=device)
        g.manual_seed(0)
        self.upd = [torch.randn((2 * c.batch, c.rank), generator=g, device=device) * 1e-3 for _ in range(4)]
        b = c.batch
        self.keys = [torch.cat([self.i[k * b:(k + 1) * b].to(torch.int64),
                                c.col_key_base + self.j[k * b:(k + 1) * b].to(torch.int64)]) for k in range(n_steps)]

    def units(self, k):
        return 2 * self.cfg.batch

    def step(self, k):
        self.ps.ps_push(self.store.h, self.keys[k], self.upd[k % len(self.upd)])

    def host_setup(self, steps):
        return None

    def alg_bytes(self, k):
        n, rb = 2 * self.cfg.batch, self.row_bytes
        return n * (16 + rb) + n_unique(self.keys[k]) * 2 * rb

    def kernel_bytes(self, k, moved=0.0):
        n, rb = 2 * self.cfg.batch, self.row_bytes
        u = n_unique(self.keys[k])
        return {"push_reduce_kernel": n * (8 + rb) + u * (8 + 2 * rb), "push_fixup_kernel": fixup_bytes(self.keys[k], 32, rb),
                "sort_all_kernel": sort_bytes(n, int(self.cfg.num_keys).bit_length()) + 4 * n,
                "push_atomic_kernel": n * (16 + rb) + n * 2 * rb, "push_check_keys_kernel": n * 8}

    def oracle_setup(self, device):
        return None


class MFDsgdWorkload(MFWorkload):
    """Matrix factorization under parameter blocking (Section 2.2, Appendix A): ps_dsgd_epoch_mf with 8 workers.
    One timed repeat is ONE call over the cells of its steps (an epoch over that sample: the row blocks are
    localized once, the column blocks once per subepoch, then the minibatches of every stratum)."""

    WORKERS = 8
    graph_ok = False

    def describe(self):
        return dict(super().describe(), workload=self.cfg.name + "_dsgd", workers=self.WORKERS,
                    schedule="ps_dsgd_epoch_mf: 8 x 8 strata, one call per timed repeat over the repeat's cells")

    def setup(self, ps, device, n_steps, keep_host_init):
        c, N = self.cfg, self.WORKERS
        self.ps = ps
        slots = -(-c.num_keys // N) + -(-c.rows // N) + -(-c.cols // N)      # initial keys + a row block + a column block
        self.store = ps.Store(c.num_keys, c.rank, N, slots, max_batch_keys=max(2 * c.batch, 1 << 18),
                              device=device.index)
        for s, rows in self.gen_init(device):
            self.store.set_rows(torch.arange(s, s + rows.shape[0], dtype=torch.int64, device=device), rows)
        self.host_init = None
        planted = W.mf_planted(c, device)
        self.i, self.j, self.v = W.mf_cells(c, planted, 0, n_steps * c.batch, device)
        del planted
        self.grouped = {}
        torch.cuda.synchronize(device)

    def run_steps(self, ks):
        c, b = self.cfg, self.cfg.batch
        key = (ks[0], len(ks))
        if key not in self.grouped:                             # regrouping the cells by stratum is input preparation
            sl = slice(ks[0] * b, (ks[-1] + 1) * b)
            self.grouped[key] = W.mf_stratify(self.i[sl], self.j[sl], self.v[sl], c.rows, c.cols, self.WORKERS)
            torch.cuda.synchronize()
        gi, gj, gv, off = self.grouped[key]
        self.ps.ps_dsgd_epoch_mf(self.store.h, gi, gj, gv, off, c.rows, c.cols, b, c.lr, c.lam, self.store.loss)

    def prepare(self, chunks):
        for ch in chunks:
            c, b = self.cfg, self.cfg.batch
            sl = slice(ch[0] * b, (ch[-1] + 1) * b)
            self.grouped[(ch[0], len(ch))] = W.mf_stratify(self.i[sl], self.j[sl], self.v[sl], c.rows, c.cols, self.WORKERS)
        torch.cuda.synchronize()

    def host_setup(self, steps):
        return None

    def kernel_bytes(self, k, moved=0.0):
        kb = super().kernel_bytes(k, moved)
        c, rb = self.cfg, self.row_bytes
        # per step: the relocations' share (rows moved per step from the device counter; keys and table entries in)
        kb["loc_fused_kernel"] = None
        kb["key_range_kernel"] = None
        return kb

    def oracle_setup(self, device):
        return None


class KeyMapWorkload:
    """A store behind the sparse-map front end (Section 3.7): per step the batch's sparse 64-bit keys are
    translated (ps_keymap_insert: known keys are found, unseen ones added) and the rows pulled by dense key."""

    def __init__(self, cfg):
        self.cfg, self.example = cfg, "keys"
        self.row_bytes = cfg.row_len * 4

    def describe(self):
        c = self.cfg
        return {"workload": "keymap_" + c.name, "keys": c.num_keys, "row_len": c.row_len, "batch_keys": c.batch,
                "store_gb": round(c.num_keys * c.row_len * 4 / 1e9, 2),
                "l2": "inputs larger than L2 (random rows of the store; no flush between steps)"}

    def max_steps(self):
        return min(self.cfg.n_batches, 400)

    def side_stream_kernels(self):
        return ()

    def setup(self, ps, device, n_steps, keep_host_init):
        c = self.cfg
        self.ps = ps
        self.store = ps.Store(c.num_keys, c.row_len, 1, max_batch_keys=c.batch, device=device.index)
        self.map = ps.KeyMap(c.num_keys, max_batch_keys=c.batch, device=device.index)
        # a sparse name per dense key of the generator: an odd multiplier makes a bijection on 64 bits
        self.keys = [(W.stress_keys(c, k, device) * 0x9E3779B97F4A7C15 + 12345) for k in range(n_steps)]
        self.dense = torch.empty(c.batch, dtype=torch.int64, device=device)
        self.out = torch.empty((c.batch, c.row_len), dtype=torch.float32, device=device)
        torch.cuda.synchronize(device)

    def units(self, k):
        return self.cfg.batch

    def step(self, k):
        self.ps.ps_keymap_insert(self.map.h, self.keys[k], self.dense)
        self.ps.ps_pull(self.store.h, self.dense, self.out)

    def host_setup(self, steps):
        return None

    def alg_bytes(self, k):
        n, rb = self.cfg.batch, self.row_bytes
        return n * (8 + 16 + 8) + n * (16 + 2 * rb)             # key in, slot (key word + value word) read, dense key out; then the pull

    def kernel_bytes(self, k, moved=0.0):
        n, rb = self.cfg.batch, self.row_bytes
        return {"map_insert_kernel": n * (8 + 16 + 8 + 8), "pull_bulk_kernel": n * (16 + 2 * rb)}

    def extra_profile(self):
        """The map's kernels are not launched through the store handle: time them here, alone, with CUDA events."""
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        us = []
        for k in range(5):
            torch.cuda.synchronize()
            a.record()
            self.ps.ps_keymap_insert(self.map.h, self.keys[k], self.dense)
            b.record()
            torch.cuda.synchronize()
            us.append(a.elapsed_time(b) * 1e3)
        n = getattr(self, "_prof_steps", 1)
        return {"map_insert_kernel": (n, float(np.median(us)) * n)}

    def oracle_setup(self, device):
        return None


class KGEWorkload:
    """ComplEx + AdaGrad (Section 4.1 / Appendix A task): triples/s through ps_step_kge."""

    def __init__(self, cfg, twin=None):
        self.cfg, self.example = cfg, "triples"
        self.row_bytes = cfg.row_len * 4
        self.twin = twin                        # a store with fewer keys for the oracle leg, where the full one does not fit the host

    def describe(self):
        c = self.cfg
        return {"workload": c.name, "entities": c.entities, "relations": c.relations, "dim_complex": c.dim,
                "negatives": c.n_neg, "minibatch": c.batch, "store_gb": round(c.num_keys * c.row_len * 4 / 1e9, 2),
                "l2": "inputs larger than L2 (random rows of the store; no flush between steps)"}

    def max_steps(self):
        return self.cfg.n_batches - 1

    def setup(self, ps, device, n_steps, keep_host_init):
        c = self.cfg
        self.ps = ps
        self.store = ps.Store(c.num_keys, c.row_len, 1, max_batch_keys=(3 + c.n_neg) * c.batch, device=device.index)
        keep = keep_host_init and self.twin is None
        self.host_init = torch.empty((c.num_keys, c.row_len), dtype=torch.float32) if keep else None
        chunk = max(1, (1 << 28) // (c.row_len * 4))             # rows per 256 MB
        for s in range(0, c.num_keys, chunk):
            n = min(chunk, c.num_keys - s)
            rows = W.kge_init_rows(c, s, n, device)
            self.store.set_rows(torch.arange(s, s + n, dtype=torch.int64, device=device), rows)
            if keep:
                self.host_init[s:s + n] = rows.cpu()
        self.s, self.r, self.o, self.neg, self.side = W.kge_triples(c, 0, n_steps * c.batch, device)
        torch.cuda.synchronize(device)

    def units(self, k):
        return self.cfg.batch

    def side_stream_kernels(self):
        return ("sort_all_kernel", "kge_keys")

    def _sl(self, k):
        b = self.cfg.batch
        return slice(k * b, (k + 1) * b)

    def step(self, k):
        c, sl = self.cfg, self._sl(k)
        self.ps.ps_step_kge(self.store.h, self.s[sl], self.r[sl], self.o[sl], self.neg[sl], self.side[sl], c.n_neg,
                            c.rel_key_base, c.dim, c.lr, c.eps, self.store.loss)

    def host_setup(self, steps):
        b = self.cfg.batch
        lo, n = steps[0] * b, len(steps) * b
        self.h = [t[lo:lo + n].cpu().contiguous().pin_memory() for t in (self.s, self.r, self.o, self.neg, self.side)]
        self.h_lo = steps[0]
        self.h_loss = torch.zeros(len(steps), dtype=torch.float64).pin_memory()
        self.h_batches = [tuple(t[x * b:(x + 1) * b] for t in self.h) + (self.h_loss[x:x + 1],) for x in range(len(steps))]
        return b * (12 + self.cfg.n_neg * 5), 8

    def step_host(self, k):
        c = self.cfg
        s, r, o, neg, side, h_loss = self.h_batches[k - self.h_lo]
        self.ps.ps_step_kge_host(self.store.h, s, r, o, neg, side, c.n_neg, c.rel_key_base, c.dim, c.lr, c.eps,
                                 self.store.loss, h_loss)

    def alg_bytes(self, k):
        c, sl, b = self.cfg, self._sl(k), self.cfg.batch
        occ = (3 + c.n_neg) * b
        u = n_unique(self.s[sl], self.o[sl], self.neg[sl]) + n_unique(self.r[sl])
        return b * (12 + c.n_neg * 5) + occ * (8 + self.row_bytes) + u * 2 * self.row_bytes

    def kernel_bytes(self, k, moved=0.0):
        c, sl, b = self.cfg, self._sl(k), self.cfg.batch
        u = n_unique(self.s[sl], self.o[sl], self.neg[sl]) + n_unique(self.r[sl])
        keys = torch.cat([t.reshape(-1).to(torch.int64) for t in (self.s[sl], self.o[sl], self.neg[sl])] +
                         [c.rel_key_base + self.r[sl].to(torch.int64)])
        kb = kernel_bytes_of_step(b * (12 + c.n_neg * 5), (3 + c.n_neg) * b, u, self.row_bytes, "kge_keys", "kge_step",
                                  int(c.num_keys).bit_length(), keys)
        occ, rb = (3 + c.n_neg) * b, self.row_bytes
        # the step kernel reads the embedding half of every row and writes a gradient row of the same size; the
        # reduction reads those and read-modify-writes every distinct row
        if c.dim % 2 == 0 and c.dim <= 128:
            kb["kge_step"] = b * (12 + c.n_neg * 5) + occ * (8 + rb // 2) + occ * (rb // 2)
            kb["kge_reduce_kernel"] = occ * (8 + rb // 2) + u * (8 + 2 * rb)
        # (wider rows: the step kernel reads whole rows and writes finished update rows, reduced like a push's)
        return kb

    def oracle_setup(self, device):
        from oracle import OracleStore
        c = self.twin or self.cfg
        if self.twin is not None:
            self.oracle_name = (f"{c.name} ({c.entities} entities, the same rows and minibatch: a K-scaled twin of "
                                f"{self.cfg.name}, whose store the oracle would have to hold in host memory)")
        o = OracleStore(c.num_keys, c.row_len, 1)
        if getattr(self, "host_init", None) is not None:
            o.set_rows(np.arange(c.num_keys), self.host_init.numpy())
        else:
            chunk = max(1, (1 << 28) // (c.row_len * 4))
            for s in range(0, c.num_keys, chunk):
                n = min(chunk, c.num_keys - s)
                o.set_rows(np.arange(s, s + n), W.kge_init_rows(c, s, n, device).cpu().numpy())
        self.oracle = o
        return o

    def oracle_data(self, device, n_steps):
        c = self.twin or self.cfg
        if self.twin is not None or not hasattr(self, "s"):
            n_steps = min(n_steps, 16)
            d = W.kge_triples(c, 0, n_steps * c.batch, device)
        else:
            d = (self.s, self.r, self.o, self.neg, self.side)
        n = n_steps * c.batch
        self.od = [t[:n].cpu().numpy() for t in d]
        self.o_steps = n_steps

    def oracle_step(self, k, n):
        c, b = self.twin or self.cfg, self.cfg.batch
        k = k % self.o_steps
        sl = slice(k * b, k * b + n)
        s, r, o, neg, side = (t[sl] for t in self.od)
        self.oracle.step_kge(s, r, o, neg, side, c.rel_key_base, c.dim, c.lr, c.eps)
        return n


class RescalWorkload(KGEWorkload):
    """RESCAL + AdaGrad (the paper's second knowledge-graph model, Section 4.1 / Table 4): triples/s through
    ps_step_rescal.  A relation's d x d matrix is d keys of the store, so a data point has 2 + n_neg + d occurrences."""

    def __init__(self, cfg):
        super().__init__(cfg)

    def describe(self):
        c = self.cfg
        return {"workload": c.name, "entities": c.entities, "relations": c.relations, "dim": c.dim,
                "relation_matrix": f"{c.dim} x {c.dim} as {c.dim} keys", "negatives": c.n_neg, "minibatch": c.batch,
                "store_gb": round(c.num_keys * c.row_len * 4 / 1e9, 2),
                "l2": "inputs larger than L2 (random rows of the store; no flush between steps)"}

    def _occ(self):
        c = self.cfg
        return (2 + c.n_neg + c.dim) * c.batch

    def setup(self, ps, device, n_steps, keep_host_init):
        c = self.cfg
        self.ps = ps
        self.store = ps.Store(c.num_keys, c.row_len, 1, max_batch_keys=self._occ(), device=device.index)
        self.host_init = torch.empty((c.num_keys, c.row_len), dtype=torch.float32) if keep_host_init else None
        chunk = max(1, (1 << 28) // (c.row_len * 4))
        for s in range(0, c.num_keys, chunk):
            n = min(chunk, c.num_keys - s)
            rows = W.rescal_init_rows(c, s, n, device)
            self.store.set_rows(torch.arange(s, s + n, dtype=torch.int64, device=device), rows)
            if keep_host_init:
                self.host_init[s:s + n] = rows.cpu()
        self.s, self.r, self.o, self.neg, self.side = W.kge_triples(c, 0, n_steps * c.batch, device)
        torch.cuda.synchronize(device)

    def side_stream_kernels(self):
        return ("sort_all_kernel", "rescal_keys")

    def step(self, k):
        c, sl = self.cfg, self._sl(k)
        self.ps.ps_step_rescal(self.store.h, self.s[sl], self.r[sl], self.o[sl], self.neg[sl], self.side[sl], c.n_neg,
                               c.rel_key_base, c.dim, c.lr, c.eps, self.store.loss)

    def host_setup(self, steps):
        return None                                 # (no host-batch entry point for this step)

    def _distinct(self, sl):
        return n_unique(self.s[sl], self.o[sl], self.neg[sl]) + n_unique(self.r[sl]) * self.cfg.dim

    def alg_bytes(self, k):
        c, sl, b = self.cfg, self._sl(k), self.cfg.batch
        return b * (12 + c.n_neg * 5) + self._occ() * (8 + self.row_bytes) + self._distinct(sl) * 2 * self.row_bytes

    def kernel_bytes(self, k, moved=0.0):
        c, sl, b = self.cfg, self._sl(k), self.cfg.batch
        u, occ, rb = self._distinct(sl), self._occ(), self.row_bytes
        rows_of = (c.rel_key_base + self.r[sl].to(torch.int64)[:, None] * c.dim +
                   torch.arange(c.dim, device=self.r.device, dtype=torch.int64)[None, :])
        keys = torch.cat([t.reshape(-1).to(torch.int64) for t in (self.s[sl], self.o[sl], self.neg[sl])] + [rows_of.reshape(-1)])
        kb = kernel_bytes_of_step(b * (12 + c.n_neg * 5), occ, u, rb, "rescal_keys", "rescal_grad",
                                  int(c.num_keys).bit_length(), keys)
        # the gradient kernel reads the value half of every row (the matrix once per data point) and writes a gradient
        # row of the same size per occurrence; the reduction reads those and read-modify-writes every distinct row
        kb["rescal_grad"] = b * (12 + c.n_neg * 5) + occ * (8 + rb // 2) + occ * (rb // 2)
        kb["kge_reduce_kernel"] = occ * (8 + rb // 2) + u * (8 + 2 * rb)
        return kb

    def oracle_setup(self, device):
        from oracle import OracleStore
        c = self.cfg
        o = OracleStore(c.num_keys, c.row_len, 1)
        if getattr(self, "host_init", None) is not None:
            o.set_rows(np.arange(c.num_keys), self.host_init.numpy())
        else:
            chunk = max(1, (1 << 28) // (c.row_len * 4))
            for s in range(0, c.num_keys, chunk):
                n = min(chunk, c.num_keys - s)
                o.set_rows(np.arange(s, s + n), W.rescal_init_rows(c, s, n, device).cpu().numpy())
        self.oracle = o
        return o

    def oracle_step(self, k, n):
        c, b = self.cfg, self.cfg.batch
        k = k % self.o_steps
        sl = slice(k * b, k * b + n)
        s, r, o, neg, side = (t[sl] for t in self.od)
        self.oracle.step_rescal(s, r, o, neg, side, c.rel_key_base, c.dim, c.lr, c.eps)
        return n


class SGNSWorkload:
    """Skip-gram with negative sampling (Section 4.1 / Appendix A task): center words/s through ps_step_sgns."""

    def __init__(self, cfg):
        self.cfg, self.example = cfg, "centers"
        self.row_bytes = cfg.dim * 4

    def describe(self):
        c = self.cfg
        return {"workload": c.name, "vocab": c.vocab, "dim": c.dim, "window": c.window, "negatives": c.n_neg,
                "minibatch_centers": c.batch, "store_gb": round(c.num_keys * c.dim * 4 / 1e9, 2),
                "l2": "inputs larger than L2 (random rows of the store; no flush between steps)"}

    def max_steps(self):
        return min(self.cfg.n_batches - 2, 400)

    def setup(self, ps, device, n_steps, keep_host_init):
        c = self.cfg
        self.ps = ps
        occ = c.batch * (1 + 2 * c.window * (1 + c.n_neg))
        self.store = ps.Store(c.num_keys, c.dim, 1, max_batch_keys=occ, device=device.index)
        rows = W.sgns_init_rows(c, 0, c.num_keys, device)
        self.store.set_all_rows(rows)
        self.host_init = rows.cpu() if keep_host_init else None
        del rows
        self.prefix = n_steps * c.batch + c.window + 1
        self.tokens = W.sgns_tokens(c, 0, self.prefix, device)
        self.negs = [W.sgns_negatives(c, k * c.batch, c.batch, device) for k in range(n_steps)]
        torch.cuda.synchronize(device)

    def units(self, k):
        return self.cfg.batch

    def side_stream_kernels(self):
        return ("sort_all_kernel", "sgns_keys")

    def step(self, k):
        c = self.cfg
        self.ps.ps_step_sgns(self.store.h, self.tokens, k * c.batch, c.batch, c.window, self.negs[k], c.n_neg,
                             c.out_key_base, c.lr, self.store.loss)

    def host_setup(self, steps):
        c = self.cfg
        self.h_tokens = self.tokens.cpu().pin_memory()
        self.h_negs = {k: self.negs[k].cpu().pin_memory() for k in steps}
        self.h_lo = steps[0]
        self.h_loss = torch.zeros(len(steps), dtype=torch.float64).pin_memory()
        return (c.batch + 2 * c.window) * 4 + int(np.mean([v.numel() for v in self.h_negs.values()])) * 4, 8

    def step_host(self, k):
        c = self.cfg
        first = k * c.batch
        lo, hi = max(0, first - c.window), min(self.prefix, first + c.batch + c.window)
        self.ps.ps_step_sgns_host(self.store.h, self.h_tokens[lo:hi], lo, first, c.batch, self.prefix, c.window,
                                  self.h_negs[k], c.n_neg, c.out_key_base, c.lr, self.store.loss,
                                  self.h_loss[k - self.h_lo:k - self.h_lo + 1])

    def alg_bytes(self, k):
        c = self.cfg
        first = k * c.batch
        pairs = c.pairs_before(first + c.batch) - c.pairs_before(first)
        centers = self.tokens[first:first + c.batch]
        lo = max(0, first - c.window)
        ctx = self.tokens[lo:first + c.batch + c.window]
        u = n_unique(centers) + n_unique(ctx, self.negs[k])    # contexts: every token of the window span, to rounding
        occ = c.batch + pairs * (1 + c.n_neg)
        return c.batch * 4 + pairs * (1 + c.n_neg) * 4 + occ * (8 + self.row_bytes) + u * 2 * self.row_bytes

    def _occ_u(self, k):
        c = self.cfg
        first = k * c.batch
        pairs = c.pairs_before(first + c.batch) - c.pairs_before(first)
        lo = max(0, first - c.window)
        u = n_unique(self.tokens[first:first + c.batch]) + \
            n_unique(self.tokens[lo:first + c.batch + c.window], self.negs[k])
        return pairs, c.batch + pairs * (1 + c.n_neg), u

    def kernel_bytes(self, k, moved=0.0):
        c = self.cfg
        pairs, occ, u = self._occ_u(k)
        first = k * c.batch
        span = self.tokens[max(0, first - c.window):first + c.batch + c.window].to(torch.int64)
        # occurrence keys: the centers, every token of the span about 2 x window times as a context, the negatives
        keys = torch.cat([self.tokens[first:first + c.batch].to(torch.int64),
                          (c.out_key_base + span).repeat(2 * c.window), c.out_key_base + self.negs[k].to(torch.int64)])
        kb = kernel_bytes_of_step(c.batch * 4 + pairs * (1 + c.n_neg) * 4, occ, u, self.row_bytes,
                                  "sgns_keys", "sgns_step", int(c.num_keys).bit_length(), keys)
        # the step kernel writes two source rows per center and one factor per occurrence, not a row per occurrence
        kb["sgns_step"] += c.batch * 2 * self.row_bytes + occ * 4 - occ * self.row_bytes
        # ... and the reduction reads a factor per occurrence and those 2 x centers source rows (from L2 after the first touch)
        kb["push_reduce_kernel"] += occ * 4 + c.batch * 2 * self.row_bytes - occ * self.row_bytes
        return kb

    def oracle_setup(self, device):
        from oracle import OracleStore
        c = self.cfg
        o = OracleStore(c.num_keys, c.dim, 1)
        if getattr(self, "host_init", None) is not None:
            rows = self.host_init
        else:
            rows = W.sgns_init_rows(c, 0, c.num_keys, device).cpu()
        o.set_rows(np.arange(c.num_keys), rows.numpy())
        self.oracle = o
        return o

    def oracle_data(self, device, n_steps):
        c = self.cfg
        if not hasattr(self, "tokens"):
            self.prefix = n_steps * c.batch + c.window + 1
            self.tokens = W.sgns_tokens(c, 0, self.prefix, device)
            self.negs = [W.sgns_negatives(c, k * c.batch, c.batch, device) for k in range(n_steps)]
        self.o_tokens = self.tokens.cpu().numpy()
        self.o_negs = [t.cpu().numpy() for t in self.negs[:n_steps]]

    def oracle_step(self, k, n):
        c = self.cfg
        first = k * c.batch
        pairs = c.pairs_before(first + n) - c.pairs_before(first)
        self.oracle.step_sgns(self.o_tokens, first, n, c.window, self.o_negs[k][:pairs * c.n_neg], c.n_neg,
                              c.out_key_base, c.lr)
        return n


class StressWorkload:
    """pull + push + localize of one key batch: keys/s through ps_pull, ps_push, ps_localize."""

    POOL = 8        # distinct pre-generated batches; step k uses batch k % POOL's updates and batch k's keys

    def __init__(self, cfg):
        self.cfg, self.example = cfg, "keys"
        self.row_bytes = cfg.row_len * 4

    def describe(self):
        c = self.cfg
        return {"workload": c.name, "keys": c.num_keys, "row_len": c.row_len, "workers": c.workers,
                "batch_keys": c.batch, "localize_keys": c.localize_count,
                "store_gb": round(c.workers * c.slots_per_part * c.row_len * 4 / 1e9, 2),
                "l2": "inputs larger than L2 (random rows of the store; no flush between steps)"}

    def max_steps(self):
        return min(self.cfg.n_batches, 400)

    def setup(self, ps, device, n_steps, keep_host_init):
        c = self.cfg
        self.ps = ps
        self.store = ps.Store(c.num_keys, c.row_len, c.workers, c.slots_per_part, max_batch_keys=c.batch,
                              device=device.index)
        chunk = 1 << 21
        for s in range(0, c.num_keys, chunk):
            n = min(chunk, c.num_keys - s)
            self.store.set_rows(torch.arange(s, s + n, dtype=torch.int64, device=device),
                                W.stress_init_rows(c, s, n, device))
        self.keys = [W.stress_keys(c, k, device) for k in range(n_steps)]
        self.upd = [W.stress_updates(c, k, device) for k in range(min(self.POOL, n_steps))]
        self.out = torch.empty((c.batch, c.row_len), dtype=torch.float32, device=device)
        self.moved_before = 0
        torch.cuda.synchronize(device)

    def units(self, k):
        return self.cfg.batch

    prelocalize = None      # None: localize the batch's own keys after its push; "same": the NEXT batch's keys on the
                            # same stream; "beside": the next batch's keys on a second stream, beside the push

    def step(self, k):
        c, h = self.cfg, self.store.h
        self.ps.ps_pull(h, self.keys[k], self.out)
        self.ps.ps_push(h, self.keys[k], self.upd[k % len(self.upd)])
        if self.prelocalize is None:
            self.ps.ps_localize(h, c.requester(k), self.keys[k][:c.localize_count])
            return
        nxt = self.keys[min(k + 1, len(self.keys) - 1)][:c.localize_count]
        if self.prelocalize == "same":
            self.ps.ps_localize(h, c.requester(k + 1), nxt)
        else:
            self.ps.ps_localize_beside(h, c.requester(k + 1), nxt, self.loc_stream)

    def host_setup(self, steps):
        return None

    def alg_bytes(self, k):
        c, n, rb = self.cfg, self.cfg.batch, self.row_bytes
        u = n_unique(self.keys[k])
        pull = n * (16 + 2 * rb)
        push = n * (16 + rb) + u * 2 * rb
        loc = c.localize_count * 16                              # rows moved are added from the device counter
        return pull + push + loc

    def side_stream_kernels(self):
        return ("sort_all_kernel",)

    def kernel_bytes(self, k, moved=0.0):
        c, n, rb = self.cfg, self.cfg.batch, self.row_bytes
        u = n_unique(self.keys[k])
        bits = int(c.num_keys).bit_length()
        nl = c.localize_count
        return {"pull_bulk_kernel": n * (16 + 2 * rb), "pull_kernel": n * (16 + 2 * rb),
                "push_reduce_kernel": n * (8 + rb) + u * (8 + 2 * rb),
                "push_fixup_kernel": fixup_bytes(self.keys[k], 32, rb),
                "push_atomic_kernel": n * (16 + rb) + n * 2 * rb, "push_check_keys_kernel": n * 8,
                # two sorts per step (push: 1M keys, localize: 100k keys), 64-bit caller keys in
                "sort_all_kernel": (sort_bytes(n, bits) + 4 * n + sort_bytes(nl, bits) + 4 * nl) / 2,
                # the relocation after its key sort: sorted keys and table entries in (twice: count, then assign),
                # per moved row: free slot in, table entry and vacated slot out, the row read and written
                "loc_fused_kernel": nl * 2 * (4 + 8) + moved * (2 * rb + 8 + 4 + 4),
                "loc_plan_kernel": nl * 2 * (4 + 8) + moved * (8 + 4 + 20), "loc_apply_kernel": moved * (2 * rb + 24)}

    # --- oracle leg: a K-scaled twin (the oracle would need the 51 GB store in host memory) ---
    TWIN = W.STRESS_MEDIUM

    def oracle_setup(self, device):
        from oracle import OracleStore
        c = self.TWIN
        self.oracle_name = (f"{c.name} (the stress batch on a store of {c.num_keys} keys and {c.workers} workers: a "
                            f"K-scaled twin of {self.cfg.name}, whose 51 GB store the oracle would have to hold in host memory)")
        o = OracleStore(c.num_keys, c.row_len, c.workers, c.slots_per_part)
        chunk = 1 << 20
        for s in range(0, c.num_keys, chunk):
            n = min(chunk, c.num_keys - s)
            o.set_rows(np.arange(s, s + n), W.stress_init_rows(c, s, n, device).cpu().numpy())
        self.oracle = o
        return o

    def oracle_data(self, device, n_steps):
        c = self.TWIN
        n_steps = min(n_steps, 8)
        self.o_keys = [W.stress_keys(c, k, device).cpu().numpy() for k in range(n_steps)]
        self.o_upd = W.stress_updates(c, 0, device).cpu().numpy()
        self.o_steps = n_steps

    def oracle_step(self, k, n):
        c = self.TWIN
        keys = self.o_keys[k % self.o_steps][:n]
        self.oracle.pull(keys)
        self.oracle.push(keys, self.o_upd[:n])
        nl = min(n, c.localize_count)
        self.oracle.localize(c.requester(k), keys[:nl])
        return n


def make_workload(name):
    table = {"mf_dsgd": lambda: MFDsgdWorkload(W.MF_LARGE), "mf_medium_dsgd": lambda: MFDsgdWorkload(W.MF_MEDIUM),
             "keymap": lambda: KeyMapWorkload(W.STRESS_MEDIUM),
             "push_mf": lambda: MFPushWorkload(W.MF_LARGE), "mf_large": lambda: MFWorkload(W.MF_LARGE), "mf_tiny": lambda: MFWorkload(W.MF_TINY),
             "mf_medium": lambda: MFWorkload(W.MF_MEDIUM),
             "kge": lambda: KGEWorkload(W.KGE), "kge_tiny": lambda: KGEWorkload(W.KGE_TINY),
             "kge_4000": lambda: KGEWorkload(W.KGE_4000, twin=W.KGE_4000_TWIN),
             "rescal": lambda: RescalWorkload(W.RESCAL), "rescal_tiny": lambda: RescalWorkload(W.RESCAL_TINY),
             "sgns": lambda: SGNSWorkload(W.SGNS), "sgns_tiny": lambda: SGNSWorkload(W.SGNS_TINY),
             "stress": lambda: StressWorkload(W.STRESS), "stress_tiny": lambda: StressWorkload(W.STRESS_TINY),
             "stress_medium": lambda: StressWorkload(W.STRESS_MEDIUM)}
    return table[name]()


# ----------------------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------------------
def dist_setup(n_gpus):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group(backend="nccl" if torch.cuda.is_available() else "gloo")
    return rank, world, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x, world, device):
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def timed_loop(fn, steps, device, world):
    """CUDA-event time (ms) of fn(k) for k in steps, bracketed by barrier + synchronize."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    torch.cuda.synchronize(device)
    a.record()
    t0 = time.perf_counter()
    for k in steps:
        fn(k)
    timed_loop.host_enqueue_ms = (time.perf_counter() - t0) * 1e3      # host time to enqueue, before any wait
    b.record()
    torch.cuda.synchronize(device)
    barrier(world)
    return max_over_ranks(a.elapsed_time(b), world, device)


def cpu_baseline(wl, device, max_steps, budget_s=15.0):
    """The oracle, as it stands, on this machine's host cores (one thread), on a bounded sample of the workload."""
    if wl.oracle_setup(device) is None:
        return None
    wl.oracle_data(device, max_steps)
    full = wl.units(0)
    t0 = time.perf_counter()
    done, k = 0, 0
    probe = max(1, full // 16)
    done += wl.oracle_step(0, probe)                            # a short probe sizes the rest
    rate = done / max(time.perf_counter() - t0, 1e-9)
    k = 1
    while k < max_steps and (time.perf_counter() - t0) + full / rate < budget_s:
        done += wl.oracle_step(k, full)
        k += 1
    dt = time.perf_counter() - t0
    return {"value": done / dt, "unit": f"{wl.example}/s", "cores": 1, "kind": "oracle", "host_cores": os.cpu_count(),
            "sample": f"{done} {wl.example} ({k} batches: one of {probe}, then full ones) of "
                      f"{getattr(wl, 'oracle_name', wl.cfg.name)}, "
                      f"{dt:.1f} s of CPU time, sequential C oracle, fp64 accumulation"}


def plan_repeats(args, wl):
    """K steps per timed repeat and R repeats, every repeat on batches of its own.  R grows for short runs so that
    the median is taken over a region of some length: at least 5, at most 30."""
    avail = wl.max_steps() - args.warmup
    r = args.repeats if args.repeats > 0 else max(5, min(30, 2000 // max(args.steps, 1)))
    k = min(args.steps, max(1, avail // (r + 1)))
    return k, r


def run_ours(args):
    import paper_2002_00655_b200 as ps
    rank, world, local = dist_setup(args.gpus)
    assert torch.cuda.is_available(), "bench.py needs a CUDA device: the library has no CPU path"
    device = torch.device("cuda", local if world > 1 else 0)
    torch.cuda.set_device(device)
    wl = make_workload(args.workload)
    steps, repeats = plan_repeats(args, wl)
    e2e_steps = min(steps, 200)
    prof_steps = min(steps, 50)
    total = args.warmup + steps * (repeats + 1)                 # warm-up, one untimed repeat, the timed repeats
    want_cpu = world == 1 and not args.no_cpu_baseline
    wl.setup(ps, device, total, keep_host_init=want_cpu)
    h = wl.store.h
    code = wl.store.sync(check=False)
    assert code == 0, f"device error during setup: {code}"
    # every batch array exists and is complete before the first step: the precondition of pipelined mode
    ps.ps_set_pipelining(h, not args.no_pipelining)
    if args.atomic_push:
        ps.ps_set_push_mode(h, ps.PS_PUSH_ATOMIC)
    if args.mf_by_column:
        ps.ps_set_mf_path(h, ps.PS_MF_BY_COLUMN)
    if args.prelocalize:
        assert hasattr(wl, "prelocalize"), "--prelocalize is for the stress workloads"
        wl.prelocalize = args.prelocalize
        wl.loc_stream = torch.cuda.Stream(device)
        if args.prelocalize == "beside":
            wl.graph_ok = False                                 # two caller streams: the calls are issued eagerly

    if hasattr(wl, "run_steps"):
        wl.run_steps(list(range(args.warmup)))
    else:
        for k in range(args.warmup):
            wl.step(k)
    torch.cuda.synchronize(device)
    # repeat r works on steps chunks[r]; chunk 0 is run once untimed (first launch of the graphs, caches, clocks)
    chunks = [list(range(args.warmup + r * steps, args.warmup + (r + 1) * steps)) for r in range(repeats + 1)]
    if hasattr(wl, "prepare"):
        wl.prepare(chunks)
    wl._prof_steps = prof_steps
    # The launch-bound loop of steps is captured into CUDA graphs (one per repeat, every step with its own batch
    # pointers) and each is replayed with one launch; --no-graph issues the calls one by one instead.
    # Short repeats are issued eagerly: replaying a graph of K multi-stream steps costs a launch of its own (about
    # 60 us here) that K = 20 steps do not amortise (52 us per MF-large step from a graph, 50 from eager calls; from
    # about 64 steps on the graph is the faster form, and it keeps host jitter out of the timed region).
    graphs = None
    if not args.no_graph and steps >= 64 and getattr(wl, "graph_ok", True):
        try:
            graphs = []
            for ch in chunks:
                torch.cuda.synchronize(device)
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    for k in ch:
                        wl.step(k)
                graphs.append(g)
        except Exception as e:                                 # noqa: BLE001
            sys.stderr.write(f"graph capture failed ({e}); timing eager launches\n")
            graphs = None

    def run_chunk(r):
        if graphs is not None:
            return timed_loop(lambda _k: graphs[r].replay(), [0], device, world)
        if hasattr(wl, "run_steps"):                            # a call that takes a whole run of steps (an epoch schedule)
            return timed_loop(lambda _k: wl.run_steps(chunks[r]), [0], device, world)
        return timed_loop(wl.step, chunks[r], device, world)

    run_chunk(0)                                                # untimed
    moved0 = ps.ps_rows_moved(h)
    sampler = ClockSampler(device.index)
    sampler.start()
    ms_all, host_ms = [], 0.0
    for r in range(1, repeats + 1):
        ms_all.append(run_chunk(r))
        host_ms += timed_loop.host_enqueue_ms
    clocks = sampler.stop()
    timed = [k for ch in chunks[1:] for k in ch]
    moved = ps.ps_rows_moved(h) - moved0
    code = wl.store.sync(check=False)
    assert code == 0, f"device error in the timed region: {ps.ps_status_string(code)}"
    loss = float(wl.store.loss.cpu()[0])
    # Summed pushes give a hot key an effective step of lr x (its multiplicity in the batch); a workload
    # whose hottest keys occur thousands of times per batch can leave the finite range.  That changes no
    # byte moved or instruction issued, so the throughput stands; the line says so instead of hiding it.
    finite = bool(np.isfinite(loss))

    ms = float(np.median(ms_all))                               # one repeat of `steps` steps
    units = sum(wl.units(k) for k in chunks[1])
    value = units * world / (ms / 1e3)
    sample_ks = timed[:: max(1, len(timed) // 16)]
    moved_per_step = moved / len(timed)
    alg = float(np.mean([wl.alg_bytes(k) for k in sample_ks]))
    if moved:
        alg += moved_per_step * (2 * wl.row_bytes + 8)
    peak, peak_src = measured_hbm_peak()
    achieved = alg / (ms / 1e3 / steps) / 1e9

    # end to end: batch in pinned host memory, copies and the loss read-back inside the timed region
    e2e = None
    e2e_ks = chunks[1][:e2e_steps]
    hb = wl.host_setup(e2e_ks)
    if hb is not None:
        h2d, d2h = hb
        # batches travel on the library's copy stream beside the steps before them; the calls do not wait, every
        # step's loss lands in its own pinned word, and the timed region ends with a wait for all of it
        ps.ps_set_host_overlap(h, True)
        for k in e2e_ks[:3]:
            wl.step_host(k)
        ms_e_all = [timed_loop(wl.step_host, e2e_ks, device, world) for _ in range(3)]
        ms_e = float(np.median(ms_e_all))
        ps.ps_set_host_overlap(h, False)
        e2e = {"value": sum(wl.units(k) for k in e2e_ks) * world / (ms_e / 1e3), "unit": f"{wl.example}/s",
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": len(e2e_ks), "repeats": 3,
               "ms_per_step": ms_e / len(e2e_ks), "ms_per_step_min": min(ms_e_all) / len(e2e_ks),
               "mode": "ps_step_*_host with ps_set_host_overlap: pinned host batch copied per step, loss read back per step, "
                       "one wait at the end of the timed region; median of 3 passes over the same host batches"}

    # per-kernel times from event pairs around every launch (a separate, untimed pass)
    launches_a = ps.ps_launch_count(h)
    if hasattr(wl, "run_steps"):
        prof_steps = steps
    ps.ps_profile_start(h, 64 * prof_steps + 4096)
    if hasattr(wl, "run_steps"):
        wl.run_steps(chunks[1])
    else:
        for k in chunks[1][:prof_steps]:
            wl.step(k)
    prof = ps.ps_profile_stop(h)
    prof.update(wl.extra_profile() if hasattr(wl, "extra_profile") else {})
    launches_per_step = (ps.ps_launch_count(h) - launches_a) / prof_steps
    tot_us = sum(us for _, us in prof.values()) or 1.0
    kb = {}
    for k in sample_ks:
        for pre, v in wl.kernel_bytes(k, moved_per_step).items():
            if v is not None:
                kb[pre] = kb.get(pre, 0.0) + v / len(sample_ks)
    side = wl.side_stream_kernels() if not args.no_pipelining else ()
    kernels = []
    for name, (n, us) in prof.items():
        row = {"name": name, "launches_per_step": n / prof_steps, "us_per_launch": us / n, "us_per_step": us / prof_steps,
               "share": us / tot_us, "stream": "internal" if name.startswith(tuple(side)) else "caller",
               "alg_bytes_per_launch": None, "gbs": None, "frac": None, "frac_of_nominal_8TBs": None}
        pre = next((p for p in sorted(kb, key=len, reverse=True) if name.startswith(p)), None)
        if pre is not None:
            row["alg_bytes_per_launch"] = kb[pre]
            row["gbs"] = kb[pre] / (us / n * 1e-6) / 1e9
            row["frac"] = row["gbs"] / peak
            row["frac_of_nominal_8TBs"] = row["gbs"] / 8000.0
        kernels.append(row)
    # the dominant kernel: the largest share of a step among the kernels on the caller's stream (the key sort and
    # key extraction run on the library's internal streams beside them in pipelined mode and are listed apart)
    rated = [r for r in kernels if r["frac"] is not None and r["stream"] == "caller"]
    dom = max(rated, key=lambda r: r["us_per_step"]) if rated else None

    out = {
        "metric": METRIC, "value": value, "unit": f"{wl.example}/s", "n_gpus": world, "steps": steps,
        "warmup": args.warmup, "repeats": repeats, "ms_per_step": ms / steps,
        "ms_per_step_min": min(ms_all) / steps, "ms_per_step_max": max(ms_all) / steps,
        "timing": f"median of {repeats} timed repeats of {steps} steps, each repeat on batches of its own, after "
                  f"{args.warmup} warm-up steps and one untimed repeat",
        "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "impl": "ours",
        "config": dict(wl.describe(), parallelism="replicas only" if world > 1 else "single GPU",
                       accumulation="per-key sums of update terms in f64 (a key that occurs once in the batch: one f32 "
                                    "add, the same single rounding); terms formed in f32; state f32",
                       pipelining="off" if args.no_pipelining else "key sort of step t+1 beside step t (ps_set_pipelining)",
                       push="atomic adds (no sort, not reproducible)" if args.atomic_push else "sorted segmented reduction",
                       **({"mf_path": "one launch over the column side"} if args.mf_by_column else {}),
                       **({"prelocalize": f"keys of the next batch, {args.prelocalize}",
                           "localize_stats": ps.ps_localize_stats(h)} if args.prelocalize else {})),
        "gpu_launches": int(round(launches_per_step * steps * repeats)), "launches_per_step": launches_per_step,
        "host_enqueue_ms_per_step": host_ms / len(timed),
        "launch_mode": "one CUDA graph per repeat" if graphs is not None else "eager calls (graphs from 64 steps per repeat on)",
        # `roofline`: the kernel on the caller's stream that takes the largest share of a step, its own bytes over its
        # own time (launched alone, events on its stream, in the per-kernel pass after the timed region).
        # `roofline_step`: the bytes the METHOD must move per step (no update rows, no sort traffic) over the
        # whole timed step.
        "roofline": None if dom is None else {
            "bound": "hbm", "kernel": dom["name"], "achieved": dom["gbs"], "peak": peak, "unit": "GB/s",
            "frac": dom["frac"], "traffic": TRAFFIC.get((wl.cfg.name, dom["name"])), "peak_source": peak_src,
            "algorithmic_bytes_per_launch": dom["alg_bytes_per_launch"], "us_per_launch": dom["us_per_launch"],
            "frac_of_nominal_8TBs": dom["gbs"] / 8000.0},
        "roofline_step": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                          "algorithmic_bytes_per_step": alg, "frac_of_nominal_8TBs": achieved / 8000.0,
                          "target": "0.60 of nominal 8 TB/s = 4800 GB/s = %.2f of the measured peak" % (4800.0 / peak),
                          "scope": "one step = all kernels of one C-ABI call sequence; algorithmic bytes = batch "
                                   "arrays + occurrences x (8 B table entry + row read) + distinct keys x (row read "
                                   "+ row write)"},
        "kernels": kernels, "e2e": e2e, "clocks": clocks, "loss_sum": loss if finite else None,
        "loss_finite": finite,
    }
    if want_cpu:
        try:
            out["cpu_baseline"] = cpu_baseline(wl, device, min(256, total))
        except MemoryError as e:
            out["cpu_baseline"] = {"unavailable": f"host memory: {e}"}
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# ----------------------------------------------------------------------------------------
# reference arm: the CPU oracle on the same workload
# ----------------------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    device = torch.device("cuda", 0) if torch.cuda.is_available() else torch.device("cpu")
    wl = make_workload(args.workload)
    if wl.oracle_setup(device) is None:
        print(json.dumps({"impl": "reference", "unavailable": "no oracle leg for this workload at full size"}))
        return
    total = args.warmup + args.steps
    n_batches = min(total, 64)
    wl.oracle_data(device, n_batches)
    full = wl.units(0)
    # size one step so that the whole run stays within about two minutes
    t0 = time.perf_counter()
    probe = max(1, full // 16)
    wl.oracle_step(0, probe)
    rate = probe / max(time.perf_counter() - t0, 1e-9)
    per_step = int(max(1, min(full, rate * 120.0 / max(total, 1))))
    for k in range(args.warmup):
        wl.oracle_step(k % n_batches, per_step)
    t0 = time.perf_counter()
    done = 0
    for k in range(args.steps):
        done += wl.oracle_step((args.warmup + k) % n_batches, per_step)
    dt = time.perf_counter() - t0
    value = done / dt
    sample = (f"each step = the first {per_step} {wl.example} of a batch of {full} ({wl.cfg.name}); sequential C oracle, "
              f"1 thread of {os.cpu_count()} host cores")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": f"{wl.example}/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / max(args.steps, 1) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": wl.describe(),
        "cpu_baseline": {"value": value, "unit": f"{wl.example}/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": f"{wl.example}/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="mf_large",
                    choices=["mf_dsgd", "mf_medium_dsgd", "keymap", "push_mf", "mf_large", "mf_medium", "mf_tiny", "kge", "kge_tiny", "kge_4000", "rescal", "rescal_tiny", "sgns", "sgns_tiny", "stress", "stress_tiny",
                             "stress_medium"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--repeats", type=int, default=0,
                    help="timed repeats of --steps steps, each on batches of its own (0: 5 to 30, more for short runs)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--atomic-push", action="store_true",
                    help="ps_push by vector atomic adds instead of the sorted segmented reduction (measured alternative)")
    ap.add_argument("--mf-by-column", action="store_true", help="ps_step_mf as one launch over the column side")
    ap.add_argument("--prelocalize", choices=["same", "beside"], default=None,
                    help="stress workload: localize the NEXT batch's keys after each push, on the same stream or on a "
                         "second stream beside the push (ps_localize_beside; eager launches)")
    ap.add_argument("--no-graph", action="store_true", help="issue every step's launches from the host")
    ap.add_argument("--no-pipelining", action="store_true",
                    help="order each step's key sort after all earlier work instead of beside the previous step")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started by hand for N GPUs: become N replica ranks (one process per GPU) through torchrun
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    if args.impl == "ours" and args.warmup < 3:
        sys.stderr.write(f"--warmup {args.warmup} raised to 3 (the timing rules ask for at least three warm-up steps)\n")
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
