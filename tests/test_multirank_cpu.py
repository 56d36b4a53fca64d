"""The benchmark's multi-rank bookkeeping on CPU: two gloo ranks on 127.0.0.1.

The path has no exchange step (replicas only), so the only cross-rank logic is the
max-over-ranks of device times and the whole-job rate; the reference arm must run on rank 0 only.
"""

import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r measured (r + 1) ms for the step loop and (10 - r) ms for attention
    got = bench.max_over_ranks([rank + 1.0, 10.0 - rank])
    dist.barrier()
    rate = bench.whole_job_rate(world, 100, got[0])
    with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
        f.write(f"{got[0]} {got[1]} {rate}")
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_rate_with_two_gloo_ranks(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        a, b, rate = (float(x) for x in open(tmp_path / f"r{r}.txt").read().split())
        assert a == 2.0 and b == 10.0                    # slowest rank on each entry
        assert rate == pytest.approx(2 * 100 / 2e-3)     # 200 steps in 2 ms


def test_without_process_group_values_pass_through():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.5]) == [3.0, 4.5]
    assert bench.whole_job_rate(1, 50, 25.0) == pytest.approx(2000.0)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
