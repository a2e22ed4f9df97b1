"""Multi-GPU runs are independent replicas: the path has no exchange step, so ranks share only a
barrier and a max-reduction of their timings. Works with any ``torch.distributed`` backend (NCCL
on GPUs, gloo on CPU)."""
from __future__ import annotations

from typing import Optional


def max_over_ranks(value: float, device=None, group=None) -> float:
    """Maximum of a per-rank scalar over all ranks (identity when not initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def aggregate_rate(units_per_rank: float, local_seconds: float, world_size: int, device=None,
                   group=None) -> float:
    """Whole-job rate of ``world_size`` replicas that each processed ``units_per_rank`` units:
    all units divided by the slowest rank's time."""
    slowest = max_over_ranks(local_seconds, device=device, group=group)
    return world_size * units_per_rank / slowest


def rank_info(env: Optional[dict] = None):
    """(rank, local_rank, world_size) from the launcher's environment."""
    import os
    e = os.environ if env is None else env
    return int(e.get("RANK", "0")), int(e.get("LOCAL_RANK", "0")), int(e.get("WORLD_SIZE", "1"))
