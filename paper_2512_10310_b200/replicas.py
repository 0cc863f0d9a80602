"""Timing reduction for replica runs: the path has no exchange step, so N GPUs run N
independent replicas and only the measured time crosses ranks (max over ranks)."""
from __future__ import annotations


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Largest `value` over all ranks of the default process group (identity without one)."""
    if dist is None or not dist.is_initialized():
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_steps_per_s(us_per_step: float, world: int) -> float:
    """Whole-job rate of `world` replicas that each need `us_per_step` (slowest rank) per step."""
    return world / (us_per_step * 1e-6)
