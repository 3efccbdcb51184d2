"""Data-parallel sharding of verification batches over GPUs: host logic only.

Sequences are independent (each tree is verified from its own logits), so a job over several GPUs
gives every rank its own sequences and needs no exchange on the data path.  The only communication
is for measurement: a barrier around a timed region and the maximum of the per-rank durations.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_seeds(rank: int, world: int, copies: int) -> list[int]:
    """Seeds of the ``copies`` input batches of one rank; no seed is shared between ranks."""
    if not 0 <= rank < world or copies <= 0:
        raise ValueError("need 0 <= rank < world and copies > 0")
    return [rank * copies + i for i in range(copies)]


def shard_sequences(B_total: int, rank: int, world: int) -> range:
    """Contiguous block of a global batch owned by ``rank`` (sizes differ by at most one)."""
    if not 0 <= rank < world or B_total < 0:
        raise ValueError("need 0 <= rank < world and B_total >= 0")
    base, extra = divmod(B_total, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def barrier(world: int) -> None:
    if world > 1:
        dist.barrier()


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Largest ``value`` held by any rank (a job is as slow as its slowest rank)."""
    if world <= 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gather_results(local: torch.Tensor, world: int) -> torch.Tensor:
    """Concatenate per-rank result tensors (equal shapes) along dim 0, in rank order, on every rank."""
    if world <= 1:
        return local
    parts = [torch.empty_like(local) for _ in range(world)]
    dist.all_gather(parts, local.contiguous())
    return torch.cat(parts, 0)
