"""Data-parallel plumbing of the EMA codebook update (host side only).

Encode and decode need no exchange: head vectors are independent given the
codebooks, so ranks simply take disjoint ranges of vectors.  The EMA statistics
are sums over vectors; ranks add theirs with one all-reduce before every rank
applies the same update.  Works on CPU tensors with gloo and on CUDA tensors
with NCCL.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_range(n: int, rank: int, world: int) -> tuple[int, int]:
    """Half-open range of head vectors owned by `rank`: contiguous, sizes differ by at most one."""
    base, extra = divmod(n, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def stats_buffer(depth: int, codebook_size: int, group_dim: int, device=None):
    """One flat float32 buffer holding the batch counts [R][K] and then the batch sums [R][K][gd], with
    views of both: the statistics of a step then travel in a single all-reduce."""
    bins = depth * codebook_size
    flat = torch.empty(bins * (group_dim + 1), dtype=torch.float32, device=device)
    return flat, flat[:bins].view(depth, codebook_size), flat[bins:].view(depth, codebook_size, group_dim)


def allreduce_stats(batch_count: torch.Tensor, batch_sum: torch.Tensor | None = None, group=None) -> None:
    """Sum the per-rank EMA statistics in place: one collective for a flat buffer from
    `stats_buffer` (pass it alone), two for separate tensors."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return
    dist.all_reduce(batch_count, group=group)
    if batch_sum is not None:
        dist.all_reduce(batch_sum, group=group)
