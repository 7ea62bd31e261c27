"""Multi-GPU runs of the block are independent replicas (the block has no exchange step): this module holds the
only cross-rank logic there is, the aggregation of per-rank timings into whole-job numbers."""
from __future__ import annotations

import torch


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The slowest rank's value (a job of replicas is as slow as its slowest member)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, ms_per_step: float, world: int) -> float:
    """Units per second of `world` replicas that each process units_per_rank per step of ms_per_step."""
    return world * units_per_rank / (ms_per_step * 1e-3)
