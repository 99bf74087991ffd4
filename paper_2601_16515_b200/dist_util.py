"""Host-side helpers for running the SALAD path on several GPUs of one node.

The attention path shards by (batch, head): every head's K and V are private to that head, so
ranks never exchange tensors.  The only collective is the timing reduction of the benchmark
(maximum over ranks).  These helpers hold no CUDA code and work with any torch.distributed
backend (the tests run them under gloo on CPU).
"""
from __future__ import annotations

from typing import List, Tuple

import numpy as np
import torch
import torch.distributed as dist


def shard_heads(B: int, H: int, world: int, rank: int) -> List[Tuple[int, int]]:
    """(batch, head) pairs owned by `rank` when B*H pairs are dealt round-robin to `world` ranks.
    Every pair is owned by exactly one rank; counts differ by at most one."""
    if world <= 0 or not (0 <= rank < world):
        raise ValueError("bad world/rank")
    return [(bh // H, bh % H) for bh in range(B * H) if bh % world == rank]


def head_range(H: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous head range [h0, h1) of `rank` when the H heads of ONE layer are split over `world`
    ranks (strong scaling): the ranges are disjoint, cover [0, H) in rank order and differ in length by
    at most one.  A rank's call then runs on the [B, h1 - h0, N, d] slices of Q, K, V."""
    if world <= 0 or not (0 <= rank < world) or H < 0:
        raise ValueError("bad world/rank")
    return H * rank // world, H * (rank + 1) // world


def slice_head_lists(row_ptr, col_idx, nQb: int, h0: int, h1: int):
    """Per-head block lists (Hm = H: row r = h*nQb + i) restricted to the heads [h0, h1): the rows of those
    heads with offsets that start at 0 again, and their block ids.  int32 numpy arrays in, the same out."""
    row_ptr = np.asarray(row_ptr); col_idx = np.asarray(col_idx)
    lo, hi = int(row_ptr[h0 * nQb]), int(row_ptr[h1 * nQb])
    rp = (row_ptr[h0 * nQb:h1 * nQb + 1].astype(np.int64) - lo).astype(np.int32)
    return rp, col_idx[lo:hi].astype(np.int32)


def sum_over_ranks(value: float, device: torch.device | str = "cpu") -> float:
    """Sum of a per-rank scalar over all ranks (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


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
