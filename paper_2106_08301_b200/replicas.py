"""Replica bookkeeping for multi-process runs: the path does not shard, so N processes run N
independent replicas; the only cross-rank step is agreeing on the slowest rank's time."""
from __future__ import annotations

import torch


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """Largest `value` over all ranks (the value itself when there is one process)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms: float) -> float:
    """Units per second of the whole job: every replica did `units_per_rank` in `ms`."""
    return world * units_per_rank / (ms * 1e-3)
