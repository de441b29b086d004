"""Multi-process plumbing, one process per GPU.

The benchmark runs independent replicas: the workers are simulated on each GPU and averaged there, so its
ranks only meet at barriers and to take the maximum of their timings.  ``Exchange`` serves the real-worker
path (``pipeline.DistributedStep``), where the compressed factors do cross GPUs.
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


class Exchange:
    """The two collectives of the real-worker path (Section 5.1: all-reduce for the PowerSGD factors and the
    uncompressed tensors, all-gather for TopK's values and indices), over ``torch.distributed`` -- NCCL between
    GPUs, gloo in the CPU tests.  Without an initialised process group it is the one-rank identity."""

    def __init__(self, group=None):
        self.group = group
        self.on = dist.is_available() and dist.is_initialized()
        self.world = dist.get_world_size(group) if self.on else 1
        self.rank = dist.get_rank(group) if self.on else 0

    def sum_(self, t: torch.Tensor) -> torch.Tensor:
        """In-place sum over ranks."""
        if self.on and self.world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.SUM, group=self.group)
        return t

    def gather_into(self, out: torch.Tensor, t: torch.Tensor) -> torch.Tensor:
        """``out`` (world x the size of ``t``, rank-major) <- every rank's ``t``."""
        if self.on and self.world > 1:
            dist.all_gather_into_tensor(out, t, group=self.group)
        else:
            out.copy_(t.reshape(out.shape))
        return out
