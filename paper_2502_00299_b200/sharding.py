"""Host-side helpers for running the path on several GPUs.

Every (sequence, layer, KV head) is an independent unit of ChunkKV compression, so ranks never
exchange data: each rank compresses its own units. The only communication is the timing
reduction (max over ranks) and a barrier, which work on any torch.distributed backend.
"""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def partition(n_units: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous, balanced [begin, end) slice of n_units owned by `rank` (sizes differ by <= 1)."""
    if world < 1 or not 0 <= rank < world or n_units < 0:
        raise ValueError("need world >= 1, 0 <= rank < world, n_units >= 0")
    return n_units * rank // world, n_units * (rank + 1) // world


def max_over_ranks(value: float, device: torch.device | str = "cpu") -> float:
    """The largest `value` any rank holds (the job is as slow as its slowest rank)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: torch.device | str = "cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_local: float, ms_local: float, device: torch.device | str = "cpu") -> Tuple[float, float]:
    """Whole-job units per second = (sum of units over ranks) / (max time over ranks).
    Returns (units_per_second, max_ms)."""
    ms = max_over_ranks(ms_local, device)
    units = sum_over_ranks(units_local, device)
    return (units / (ms * 1e-3) if ms > 0 else 0.0), ms


def gather_index_shards(idx_local: torch.Tensor, world: int) -> List[torch.Tensor]:
    """All-gather per-rank kept-index tensors of equal shape (head-sharded layers), for callers
    that want every rank to hold the indices of all KV heads. Not used on the hot path."""
    if world == 1 or not (dist.is_available() and dist.is_initialized()):
        return [idx_local]
    out = [torch.empty_like(idx_local) for _ in range(world)]
    dist.all_gather(out, idx_local)
    return out
