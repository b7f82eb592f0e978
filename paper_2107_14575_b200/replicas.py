"""Timing of independent replicas.

The path has no exchange step on one node: with N GPUs, N processes each run the whole
path on their own M buffers.  The only cross-rank arithmetic is the reporting rule:
a timed region lasts as long as its slowest rank, and the job's rate is the units all
ranks processed divided by that time.  The helpers work on any initialised
``torch.distributed`` backend (NCCL on GPUs, gloo on CPU).
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_rank() -> Tuple[int, int, int]:
    """(rank, world size, local rank) as torchrun exports them; (0, 1, 0) outside it."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(ms: float, device=None) -> float:
    """Largest of the ranks' values (the duration of a region all ranks ran side by side)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms: float) -> float:
    """Units per second of the whole job: every rank did ``units_per_rank`` in ``ms`` (max over ranks)."""
    return world * units_per_rank / (ms * 1e-3)
