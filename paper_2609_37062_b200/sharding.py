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


def shard_kv_tables(block_table, seq_lens, page_size: int, world_size: int, rank: int):
    """What `rank` attends when every sequence is cut by KV range at page
    boundaries: (local block table [B, max local pages], local lengths [B]),
    CPU int32 tensors.  A sequence with fewer pages than ranks leaves some
    ranks an empty range (length 0)."""
    import torch
    bt = block_table.detach().cpu()
    lens = [int(x) for x in seq_lens.detach().cpu().tolist()]
    spans = []
    for L in lens:
        pages = (L + page_size - 1) // page_size
        pb, pe = shard_range(pages, world_size, rank)
        spans.append((pb, pe, max(0, min(pe * page_size, L) - pb * page_size)))
    width = max(1, max(pe - pb for pb, pe, _ in spans))
    local_bt = torch.zeros((len(lens), width), dtype=torch.int32)
    for b, (pb, pe, _) in enumerate(spans):
        local_bt[b, : pe - pb] = bt[b, pb:pe]
    return local_bt, torch.tensor([n for _, _, n in spans], dtype=torch.int32)


def gather_shards(out_local, lse_local, group=None):
    """The one exchange step of KV-range sharding: all-gathers every rank's
    normalised output [B, Hq, D] and log-sum-exp [B, Hq] (any backend).
    Returns ([R, B, Hq, D], [R, B, Hq]) in rank order = ascending token order."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    outs = [torch.empty_like(out_local) for _ in range(world)]
    lses = [torch.empty_like(lse_local) for _ in range(world)]
    dist.all_gather(outs, out_local.contiguous(), group=group)
    dist.all_gather(lses, lse_local.contiguous(), group=group)
    return torch.stack(outs), torch.stack(lses)


def merge_over_ranks(shape, out_local, lse_local, out, lse=None, group=None, stream=None):
    """gather_shards, then the library's shard merge on this rank's GPU.
    out_local fp32 [B, Hq, D] and lse_local fp32 [B, Hq] are CUDA tensors."""
    from . import binding
    import torch.distributed as dist
    outs, lses = gather_shards(out_local, lse_local, group)
    binding.decode_attn_merge_shards(shape, dist.get_world_size(group), outs, lses, out, lse, stream=stream)
    return out, lse


def max_over_ranks(value: float, device=None) -> float:
    """The slowest rank's time: what a multi-GPU step costs."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
