"""The multi-rank side of bench.py on CPU: N replicas, no exchange in the data path; the only collective is
the max over the ranks' times.  Run as two gloo ranks; the reference arm must run on rank 0 alone."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def rank_main(rank, world, port, out):
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow replica
    rate = bench.whole_job_rate(300, world, ms * 1e-3)
    with open(f"{out}.{rank}", "w") as f:
        json.dump({"ms": ms, "rate": rate}, f)
    dist.destroy_process_group()


def test_time_is_the_max_over_ranks_and_the_rate_counts_every_replica(tmp_path):
    world, port, out = 2, free_port(), str(tmp_path / "r")
    mp.spawn(rank_main, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        got = json.load(open(f"{out}.{rank}"))
        assert got["ms"] == 15.0                          # every rank sees the slowest one's time
        assert abs(got["rate"] - 2 * 300 / 0.015) < 1e-6  # whole job: both replicas' steps over that time


def test_single_process_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5) == 3.5 and bench.whole_job_rate(10, 1, 2.0) == 5.0


def test_reference_arm_runs_on_rank_zero_only():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "toy", "--steps", "1",
           "--warmup", "0", "--gpus", "2"]
    env = dict(os.environ, WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(free_port()))
    r1 = subprocess.run(cmd, env=dict(env, RANK="1", LOCAL_RANK="1"), capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""            # the other ranks leave without work
    r0 = subprocess.run(cmd, env=dict(env, RANK="0", LOCAL_RANK="0"), capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0, r0.stderr[-500:]
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
