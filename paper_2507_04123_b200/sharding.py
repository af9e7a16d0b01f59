"""Frame sharding for runs on several GPUs (host logic only).

Frames are independent units of the bridge, so N processes each take their own frames and never
exchange data; the only collectives are the timing barrier and the max-over-ranks of the timed
interval, from which whole-job throughput is derived.
"""
from __future__ import annotations

from typing import List, Optional

import torch
import torch.distributed as dist


def frames_for_rank(rank: int, world: int, frames_per_rank: int) -> List[int]:
    """Global frame ids owned by ``rank``: a contiguous, disjoint block per rank."""
    if not (0 <= rank < world) or frames_per_rank < 0:
        raise ValueError("rank outside the world or negative frame count")
    return list(range(rank * frames_per_rank, (rank + 1) * frames_per_rank))


def max_over_ranks(value: float, device: Optional[torch.device] = None) -> float:
    """Largest ``value`` over all ranks (the value itself without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, seconds_this_rank: float, device: Optional[torch.device] = None) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    return world * units_per_rank / max_over_ranks(seconds_this_rank, device)
