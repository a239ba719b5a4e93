"""Whole-job aggregation for replica runs (one process per GPU, every rank verifies its own batch).

The verify step has no cross-GPU exchange; the only collectives are the ones the timing needs:
the slowest rank's time (MAX) and the bytes all ranks processed (SUM)."""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def replica_seed(base_seed: int, rank: int) -> int:
    """Distinct, reproducible input seed per replica."""
    return base_seed + 1000 * rank


def aggregate(local_units: float, local_seconds: float, device: torch.device) -> Tuple[float, float]:
    """Returns (units processed by all ranks, slowest rank's seconds). Works without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(local_units), float(local_seconds)
    t = torch.tensor([local_seconds], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(u.item()), float(t.item())


def throughput(local_units: float, local_seconds: float, device: torch.device) -> float:
    units, sec = aggregate(local_units, local_seconds, device)
    return units / sec
