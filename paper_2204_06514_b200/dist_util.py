"""Rank plumbing of the multi-replica benchmark: one process per GPU, no data-path
collective.  The only communication is the timing reduction (max over ranks)."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(value: float, device: torch.device | str = "cpu") -> float:
    """Largest `value` over all ranks (identity when torch.distributed is not initialised)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms_max: float) -> float:
    """Whole-job throughput of `world` replicas that each processed units_per_rank
    units in at most ms_max milliseconds."""
    return world * units_per_rank / (ms_max * 1e-3)
