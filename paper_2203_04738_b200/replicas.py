"""Replicas-only multi-GPU accounting: the path does not shard, so N ranks run N independent copies of the
step and the job's throughput is (units of all ranks) / (slowest rank's time).  No data-path collective."""
from __future__ import annotations

import torch
import torch.distributed as dist


def max_over_ranks(ms: float, device=None) -> float:
    """Time of the slowest rank (identity without an initialised process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, ms_per_step: float, world: int) -> float:
    """Whole-job units per second for `world` replicas that each process units_per_rank per step."""
    return world * units_per_rank / (ms_per_step * 1e-3)
