"""Two gloo ranks on CPU: the host logic of the multi-GPU benchmark path.

The path has no exchange step (states are independent), so ranks run replicas:
same graph and weights, their own states, and the job's throughput is all
ranks' states over the slowest rank's time. The reference arm runs on rank 0
only."""
from __future__ import annotations

import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = bench.make_workload("tiny", rank)
    # graph and weights identical on every rank, states differ
    sig = torch.tensor([float(cfg["src"].sum()), float(cfg["weights"]["f_down"]["W1"].sum()),
                        float(cfg["dev"].sum()) + float(cfg["cur"].sum())], dtype=torch.float64)
    gathered = [torch.zeros_like(sig) for _ in range(world)]
    dist.all_gather(gathered, sig)
    local_ms = 10.0 * (rank + 1)                       # rank 1 is the slow one
    value, slowest = bench.job_throughput(local_ms, cfg["B"], 5, dist, "cpu")
    if rank == 0:
        json.dump({"sigs": [g.tolist() for g in gathered], "value": value, "slowest": slowest,
                   "B": cfg["B"]}, open(os.path.join(out_dir, "r0.json"), "w"))
    dist.destroy_process_group()


def test_two_ranks_shard_states_and_reduce_time(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    out = json.load(open(tmp_path / "r0.json"))
    (s0, s1) = out["sigs"]
    assert s0[0] == s1[0] and s0[1] == s1[1]          # same graph, same weights
    assert s0[2] != s1[2]                             # each rank has its own states
    assert out["slowest"] == 20.0
    assert np.isclose(out["value"], 2 * out["B"] * 5 / 0.020)


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", LOCAL_RANK="1", RANK="1")
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
           "--steps", "2", "--warmup", "1", "--gpus", "2"]
    r1 = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    env.update(RANK="0", LOCAL_RANK="0")
    r0 = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
    assert line["unit"] == "evaluations/s" and line["config"]["workload"] == "tiny"
