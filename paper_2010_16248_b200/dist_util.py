"""Multi-process plumbing of the benchmark: independent replicas, one process per GPU.

The path has no exchange step between GPUs (the workers are simulated on each GPU and averaged there),
so ranks only meet at barriers and to take the maximum of their timings.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def replica_seed_offset(rank: int) -> int:
    """Offset added to the iteration index of the gradient stream so that every rank draws its own batches."""
    return 1000 * int(rank)


def max_over_ranks(value: float, device=None) -> float:
    """Maximum of a per-rank scalar over all ranks (identity without an initialised process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank_per_step: float, ms_per_step_max: float, world: int) -> float:
    """Units all ranks processed per second, from the slowest rank's step time."""
    return units_per_rank_per_step * world / (ms_per_step_max * 1e-3)
