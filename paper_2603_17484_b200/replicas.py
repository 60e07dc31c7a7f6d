"""Multi-GPU policy of the benchmark: replicas only.

The hot path has no exchange step (the target is one GPU; (batch, KV-head) units are independent), so N GPUs
run N independent replicas of the workload with no data-path collective.  The only communication is the timing
reduction: the step time of the job is the slowest rank's, and the job's throughput is the work of all ranks
over that time.  Works with any torch.distributed backend (nccl on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import torch


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """Maximum of a per-rank scalar over all ranks (identity when not distributed)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(world: int, work_per_replica: float, ms_slowest: float) -> float:
    """Whole-job rate: every replica does `work_per_replica`; the job takes as long as its slowest rank."""
    return world * work_per_replica / (ms_slowest * 1e-3)


def rank_seed_offset(rank: int) -> int:
    """Each replica draws its own inputs (same shapes and distributions)."""
    return 7919 * rank
