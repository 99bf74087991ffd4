"""Host-side helpers for running the SALAD path on several GPUs of one node.

The attention path shards by (batch, head): every head's K and V are private to that head, so
ranks never exchange tensors.  The only collective is the timing reduction of the benchmark
(maximum over ranks).  These helpers hold no CUDA code and work with any torch.distributed
backend (the tests run them under gloo on CPU).
"""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def shard_heads(B: int, H: int, world: int, rank: int) -> List[Tuple[int, int]]:
    """(batch, head) pairs owned by `rank` when B*H pairs are dealt round-robin to `world` ranks.
    Every pair is owned by exactly one rank; counts differ by at most one."""
    if world <= 0 or not (0 <= rank < world):
        raise ValueError("bad world/rank")
    return [(bh // H, bh % H) for bh in range(B * H) if bh % world == rank]


def max_over_ranks(value: float, device: torch.device | str = "cpu") -> float:
    """Maximum of a per-rank scalar over all ranks (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, local_ms: float, device: torch.device | str = "cpu") -> Tuple[float, float]:
    """Whole-job throughput for weak scaling: every rank processed `units_per_rank` units in
    `local_ms`; the job took the slowest rank's time.  Returns (units per second, ms)."""
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    ms = max_over_ranks(local_ms, device)
    return units_per_rank * world / (ms * 1e-3), ms
