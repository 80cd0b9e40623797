"""Sequence sharding for more than one GPU.

Every step of the path works on one sequence at a time, so a batch splits across ranks by
contiguous blocks of sequences with no collective on the data path.  The helpers below are the
whole multi-GPU layer: which block a rank owns, gathering the small per-sequence outputs, and the
max-over-ranks of a timing.  They work on any torch.distributed backend (nccl on GPUs, gloo in
the CPU tests).
"""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def shard_range(B: int, rank: int, world: int) -> Tuple[int, int]:
    """Sequences [b0, b1) owned by `rank`: blocks differ in size by at most one."""
    if not (0 <= rank < world):
        raise ValueError("rank outside [0, world)")
    base, extra = divmod(B, world)
    b0 = rank * base + min(rank, extra)
    return b0, b0 + base + (1 if rank < extra else 0)


def gather_sequences(local: torch.Tensor, B: int) -> torch.Tensor:
    """All-gather per-sequence outputs ([b_local, ...] on each rank) into [B, ...] on every rank."""
    world = dist.get_world_size()
    sizes = [shard_range(B, r, world) for r in range(world)]
    widest = max(b1 - b0 for b0, b1 in sizes)
    pad = torch.zeros((widest,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    pad[: local.shape[0]] = local
    parts: List[torch.Tensor] = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(parts, pad)
    return torch.cat([p[: b1 - b0] for p, (b0, b1) in zip(parts, sizes)], dim=0)


def max_over_ranks(seconds: float, device=None) -> float:
    """Slowest rank's time: the only number a multi-GPU measurement may report."""
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
