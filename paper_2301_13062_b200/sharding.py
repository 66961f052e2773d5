"""Multi-GPU plumbing: one process per GPU, environments split by contiguous global-id ranges.

The path has no exchange step: every random draw is a function of the global environment id, so
a rank's results do not depend on the partition. The only cross-rank operation is the sum of the
two 64-bit totals, done with one all-reduce (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from .inputs import shard_range


def rank_env_range(n_total: int, rank: int | None = None, world: int | None = None) -> tuple[int, int]:
    """[lo, hi) of this rank for a job of n_total environments (strong scaling split)."""
    if rank is None:
        rank = dist.get_rank() if dist.is_initialized() else 0
    if world is None:
        world = dist.get_world_size() if dist.is_initialized() else 1
    return shard_range(n_total, rank, world)


def weak_env_offset(n_per_rank: int, rank: int | None = None) -> int:
    """Offset of this rank when every rank runs a full batch of n_per_rank environments."""
    if rank is None:
        rank = dist.get_rank() if dist.is_initialized() else 0
    return rank * n_per_rank


def reduce_totals(totals: torch.Tensor) -> torch.Tensor:
    """Sum the per-rank {sum of returns, episode count} pair (int64[2]) over all ranks, in place."""
    if totals.dtype != torch.int64 or totals.numel() != 2:
        raise ValueError("totals must be an int64 tensor of two elements")
    if dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(totals, op=dist.ReduceOp.SUM)
    return totals


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """Largest value over ranks (used for timings)."""
    if not (dist.is_initialized() and dist.get_world_size() > 1):
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])
