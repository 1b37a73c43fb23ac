"""Multi-GPU use of the batch-1 path: replicas only.

The per-layer step has no exchange between GPUs (one token's neurons are few and every stage ends in a tiny
reduction that lives inside one GPU), so N GPUs run N independent copies of the stack, each on its own token stream.
This module holds the only cross-rank logic there is: which stream a rank decodes and how per-rank timings become the
whole-job figure (units of all ranks divided by the slowest rank's time).
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def stream_of_rank(rank: int) -> int:
    """Token stream a replica decodes (stream ids seed the synthetic token generator)."""
    return int(rank)


def barrier() -> None:
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def aggregate(local_ms: float, local_units: int, device: torch.device) -> Tuple[float, int]:
    """(slowest rank's milliseconds, units processed by all ranks)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(local_ms), int(local_units)
    ms = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    units = torch.tensor([int(local_units)], dtype=torch.int64, device=device)
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    dist.all_reduce(units, op=dist.ReduceOp.SUM)
    return float(ms.item()), int(units.item())


def throughput(local_ms: float, local_units: int, device: torch.device) -> float:
    """Whole-job units per second."""
    ms, units = aggregate(local_ms, local_units, device)
    return units / (ms * 1e-3) if ms > 0 else 0.0
