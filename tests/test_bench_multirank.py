"""Host logic of the multi-GPU bench path (independent replicas, no data-path collective), run as two gloo ranks
on CPU: distinct data per rank, max-over-ranks timing, whole-job value, and the reference arm printing on rank 0 only."""
import json
import os
import socket
import subprocess
import sys
from pathlib import Path

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parents[1]
sys.path.insert(0, str(ROOT))


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2510_24824_b200.inputs import make_problem
    spec = bench.replica_spec(0, rank)
    p = make_problem(spec)
    my_ms = 10.0 + 5.0 * rank  # rank 1 is the slow one
    slowest = bench.max_over_ranks(my_ms, world)
    value = bench.job_steps_per_s(world, slowest)
    dist.barrier()
    Path(out_dir, f"r{rank}.json").write_text(json.dumps(
        {"seed": spec["seed"], "q0": float(p.q.ravel()[0]), "slowest": slowest, "value": value}))
    dist.destroy_process_group()


def test_two_gloo_ranks_replicas_and_max_timing(tmp_path):
    port = free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0, r1 = (json.loads((tmp_path / f"r{i}.json").read_text()) for i in range(2))
    assert r0["seed"] != r1["seed"] and r0["q0"] != r1["q0"]          # every replica streams its own data
    assert r0["slowest"] == r1["slowest"] == 15.0                      # max over ranks
    assert r0["value"] == pytest.approx(2 * 1e3 / 15.0)                # whole-job steps/s of two replicas


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", OMP_NUM_THREADS="2")
    cmd = [sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "2", "--warmup", "1",
           "--workload", "0"]
    out1 = subprocess.run(cmd, env=dict(env, RANK="1", LOCAL_RANK="1"), capture_output=True, text=True, timeout=300)
    assert out1.returncode == 0 and out1.stdout.strip() == ""
    out0 = subprocess.run(cmd, env=dict(env, RANK="0", LOCAL_RANK="0"), capture_output=True, text=True, timeout=300)
    assert out0.returncode == 0, out0.stderr
    line = json.loads(out0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0 and line["n_gpus"] == 2
