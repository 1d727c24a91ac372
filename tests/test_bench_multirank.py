"""The benchmark's N > 1 path on CPU: two gloo ranks stand in for two GPUs.

Every chain is independent per row, so ranks are replicas with no collective on the data path;
what has to be right across ranks is the bookkeeping: each rank draws its own batch, the job
time is the slowest rank's, the value is the aggregate over ranks, and the reference arm runs on
rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
import kf_inputs as ki  # noqa: E402


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = [7.0, 11.5][rank]                                  # rank 1 is the slow one
    got = bench.max_over_ranks(ms, world)
    d = ki.gemm_inputs("c2", seed=bench.rank_seed(rank), M=8, N=8, K=16)
    digest = float(ki.widen(d["X"]).sum())
    dist.barrier()
    with open(os.path.join(out_dir, "r%d.json" % rank), "w") as f:
        json.dump({"max_ms": got, "digest": digest}, f)
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0 = json.load(open(tmp_path / "r0.json"))
    r1 = json.load(open(tmp_path / "r1.json"))
    assert r0["max_ms"] == 11.5 and r1["max_ms"] == 11.5
    assert r0["digest"] != r1["digest"]                     # each rank has its own batch


def test_whole_job_value_is_the_aggregate():
    one = bench.whole_job_tflops(bench.FLOPS_C2, 1, 0.2)
    assert abs(one - 274.877906944e9 / 0.2e-3 / 1e12) < 1e-9
    assert abs(bench.whole_job_tflops(bench.FLOPS_C2, 8, 0.2) - 8 * one) < 1e-9
    assert bench.max_over_ranks(3.0, 1) == 3.0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--gpus", "2", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
