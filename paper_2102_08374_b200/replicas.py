"""Host-side helpers for running independent replicas of the step, one process per GPU.

The IntSGD step has no exchange between GPUs in this library (the workers are buffers on one
device), so N GPUs run N replicas.  The only inter-process traffic is for timing: a barrier and the
maximum of the per-rank durations.  These helpers take any ``torch.distributed`` backend (``nccl``
on GPUs, ``gloo`` in CPU tests).
"""
from __future__ import annotations


def max_over_ranks(dist, value: float, device=None) -> float:
    """Maximum of ``value`` over all ranks (or ``value`` itself without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(dist, units_per_rank: int, local_seconds: float, device=None) -> float:
    """Units all ranks processed divided by the slowest rank's time (weak scaling: every rank
    processes ``units_per_rank``)."""
    world = 1 if (dist is None or not dist.is_initialized()) else dist.get_world_size()
    slowest = max_over_ranks(dist, local_seconds, device)
    return world * units_per_rank / slowest


def rank_seed_base(rank: int, base: int = 500, stride: int = 1000) -> int:
    """Distinct input seeds per replica."""
    return base + stride * rank
