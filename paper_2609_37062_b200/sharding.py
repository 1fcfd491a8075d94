"""How the path spreads over several GPUs (one process per GPU).

The path shards by sequence: every rank keeps the pages of its own sequences
and runs plan / run / combine on them; nothing is exchanged.  A single long
sequence can instead be sharded by KV range (context parallel): every rank
attends its token range and the partial results - (unnormalised output,
running max, sum) per head, a few KB - are all-gathered once and merged in
rank order by the same log-sum-exp merge the combine kernel uses.

This module holds the host-side logic only (index arithmetic and the
max-over-ranks timing reduction); it contains none of the attention
arithmetic.  It works with any torch.distributed backend (nccl on GPUs, gloo
in the CPU tests).
"""
from __future__ import annotations

from typing import List, Tuple


def shard_range(n_items: int, world_size: int, rank: int) -> Tuple[int, int]:
    """Contiguous [begin, end) of `n_items` for `rank`; sizes differ by at most one."""
    assert 0 <= rank < world_size
    base, rem = divmod(n_items, world_size)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)


def shard_sequences(batch: int, world_size: int, rank: int) -> List[int]:
    """Indices of the sequences `rank` owns."""
    b, e = shard_range(batch, world_size, rank)
    return list(range(b, e))


def shard_kv_range(seq_len: int, page_size: int, world_size: int, rank: int) -> Tuple[int, int]:
    """Token range [begin, end) of one sequence for `rank`, cut at page boundaries."""
    pages = (seq_len + page_size - 1) // page_size
    pb, pe = shard_range(pages, world_size, rank)
    return min(pb * page_size, seq_len), min(pe * page_size, seq_len)


def max_over_ranks(value: float, device=None) -> float:
    """The slowest rank's time: what a multi-GPU step costs."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
