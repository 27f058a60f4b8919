"""The N > 1 path of the benchmark (independent replicas, slowest rank sets the time) on two gloo ranks on the CPU."""
import os
import subprocess
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, str(ROOT))
    from paper_2602_01744_b200.replicas import max_over_ranks, whole_job_throughput
    local_ms = 10.0 if rank == 0 else 25.0                      # rank 1 is the slow one
    value, ms = whole_job_throughput(1000, 5, local_ms, dist)
    out[rank] = (max_over_ranks(float(rank), dist), value, ms)
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_ranks_time_and_the_whole_jobs_units():
    world, port = 2, 29731
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        mx, value, ms = res[rank]
        assert mx == 1.0
        assert ms == 25.0
        assert abs(value - 2 * 1000 * 5 / 25e-3) < 1e-6


def test_single_process_needs_no_group():
    from paper_2602_01744_b200.replicas import whole_job_throughput
    value, ms = whole_job_throughput(100, 2, 4.0)
    assert ms == 4.0 and value == 100 * 2 / 4e-3


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
