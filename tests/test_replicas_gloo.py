"""Multi-process launch logic on CPU (gloo, world size 2).

The path has no exchange between GPUs: `bench.py --gpus N` runs one replica per rank, and the only
collectives are the barrier and the max over ranks of the elapsed time.  This test runs that logic
with two gloo ranks: both ranks time the same bounded CPU-oracle sample, rank 0 reports
N x units / max time, and the reference arm of bench.py prints its line on rank 0 only."""
from __future__ import annotations

import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, time, json
sys.path.insert(0, %(root)r)
import numpy as np
import torch
import torch.distributed as dist
import oracle
from paper_2607_12324_b200 import workloads as W

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
g = W.make_graph("cfg1-train", 0.1)
B = 64
lv = W.policies_for(g, B=B).numpy()
dist.barrier()
t0 = time.perf_counter()
r = oracle.batch(g, lv, B=B, want_slack=True)
dt = torch.tensor([time.perf_counter() - t0], dtype=torch.float64)
dist.all_reduce(dt, op=dist.ReduceOp.MAX)
chk = torch.tensor([int(r["makespan"].sum())], dtype=torch.int64)
gathered = [torch.zeros_like(chk) for _ in range(world)]
dist.all_gather(gathered, chk)
dist.barrier()
if rank == 0:
    print(json.dumps({"world": world, "value": world * B * g.m * 2 / float(dt.item()),
                      "same": all(int(x.item()) == int(chk.item()) for x in gathered)}))
dist.destroy_process_group()
"""


def _torchrun(args, timeout=600):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29517"] + args
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_replicas_barrier_and_max_time(tmp_path, oracle_mod):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % {"root": ROOT})
    p = _torchrun([str(script)])
    assert p.returncode == 0, p.stderr[-2000:]
    line = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(line) == 1, p.stdout
    out = json.loads(line[0])
    assert out["world"] == 2 and out["same"] and out["value"] > 0


def test_reference_arm_prints_once_under_torchrun(oracle_mod):
    p = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                   "--workload", "cfg1-train"])
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, p.stdout
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["cpu_baseline"]["kind"] == "oracle"
    assert out["e2e"]["h2d_bytes_per_step"] == 0 and out["value"] > 0
