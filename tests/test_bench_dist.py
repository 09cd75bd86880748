"""The N > 1 plumbing of bench.py on CPU: two gloo ranks, barrier and max-over-ranks timing; the
reference arm prints on rank 0 only.  (The path itself does not shard: N ranks are N replicas.)"""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch
import bench
rank, world, local = bench.dist_setup(2)
assert world == 2 and rank == int(os.environ["RANK"])
bench.barrier(world)
mine = 10.0 + 5.0 * rank                      # rank 1 is the slow one
got = bench.max_over_ranks(mine, world, torch.device("cpu"))
units = 1000
print(json.dumps({{"rank": rank, "max_ms": got, "value": units * world / (got / 1e3)}}))
import torch.distributed as dist
dist.destroy_process_group()
"""


def _env(rank, port):
    e = dict(os.environ)
    e.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
             CUDA_VISIBLE_DEVICES="")
    return e


def test_two_gloo_ranks_agree_on_the_slowest_rank_time():
    port = 29000 + os.getpid() % 2000
    code = WORKER.format(root=ROOT)
    procs = [subprocess.Popen([sys.executable, "-c", code], env=_env(r, port), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e
    res = [json.loads(o.strip().splitlines()[-1]) for o, _ in outs]
    assert all(r["max_ms"] == 15.0 for r in res)               # every rank sees the max
    assert all(abs(r["value"] - 2 * 1000 / 0.015) < 1e-6 for r in res)   # whole-job units over the slowest time


def test_reference_arm_runs_on_rank_zero_only():
    base = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "mf_tiny",
            "--steps", "5", "--warmup", "1", "--gpus", "2"]
    e1 = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", CUDA_VISIBLE_DEVICES="")
    out1 = subprocess.run(base, env=e1, capture_output=True, text=True, timeout=300)
    assert out1.returncode == 0 and out1.stdout.strip() == ""
    e0 = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0", CUDA_VISIBLE_DEVICES="")
    out0 = subprocess.run(base, env=e0, capture_output=True, text=True, timeout=300)
    assert out0.returncode == 0, out0.stderr
    line = json.loads(out0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["unit"] == "cells/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_gpus_flag_without_a_launcher_starts_the_ranks_itself():
    """`python bench.py --gpus 2` run by hand (no RANK / WORLD_SIZE in the environment) becomes two ranks through
    torchrun; with the reference arm that needs no GPU: rank 0 prints the one line, the other rank prints nothing."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["CUDA_VISIBLE_DEVICES"] = ""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "mf_tiny",
                          "--steps", "3", "--warmup", "1", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
