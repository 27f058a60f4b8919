"""Multi-GPU bookkeeping of the benchmark.  The path has no exchange step, so N GPUs run N independent replicas of the
workload; the only thing that crosses ranks is timing: the job's step time is the slowest rank's, and the whole-job
throughput is the units all ranks processed divided by that time.  Works on any torch.distributed backend (NCCL on
GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import torch


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The maximum of `value` over all ranks (the value itself without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank_per_step: int, steps: int, local_ms: float, dist=None, device="cpu"):
    """(units per second over all ranks, job milliseconds) from each rank's own elapsed time for `steps` steps."""
    world = 1 if dist is None or not dist.is_initialized() else dist.get_world_size()
    ms = max_over_ranks(local_ms, dist, device)
    return world * units_per_rank_per_step * steps / (ms * 1e-3), ms
