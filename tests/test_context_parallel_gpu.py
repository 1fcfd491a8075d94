"""Sharding the KV range of long sequences over ranks (context parallelism):
every shard runs the ordinary plan / run / combine on its token range and the
shards' (output, log-sum-exp) pairs are merged by decode_attn_merge_shards in
rank order.  The ranks are emulated one after the other on one GPU - they do
not wait on one another, the exchange is a plain gather - and the result is
held against the oracle's attention over the whole sequence."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2609_37062_b200 import sharding
from paper_2609_37062_b200 import workloads as wl
from gpu_util import assert_parity, da, oracle_of, to_device

pytestmark = pytest.mark.gpu


def shards_of(w, world, policy):
    outs, lses = [], []
    for rank in range(world):
        bt, lens = sharding.shard_kv_tables(w.block_table, w.seq_lens, w.page_size, world, rank)
        local = dataclasses.replace(to_device(w), block_table=bt.cuda(), seq_lens=lens.cuda(),
                                    max_pages_per_seq=bt.shape[1])
        o, l = da.run_workload(local, policy)
        outs.append(o)
        lses.append(l)
    return torch.stack(outs), torch.stack(lses)


@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_kv_range_shards_merge_to_the_whole(world):
    w = wl.make_workload("cp", [5000, 777, 16, 1, 2049], 32, 8, 128, seed=31)     # short ones leave ranks empty
    ref_out, ref_lse = oracle_of(w)
    outs, lses = shards_of(w, world, da.make_policy())
    if world > 2:
        assert torch.isneginf(lses[-1, 3]).all()                                   # one token: the last rank has none
    shape = da.shape_of_workload(to_device(w))
    out = torch.full((5, 32, 128), float("nan"), device="cuda")
    lse = torch.full((5, 32), float("nan"), device="cuda")
    da.decode_attn_merge_shards(shape, world, outs, lses, out, lse)
    assert_parity(out, lse, ref_out, ref_lse)
    # the merge is a fixed-order sum: the same inputs give the same bits
    out2 = torch.empty_like(out)
    da.decode_attn_merge_shards(shape, world, outs, lses, out2, None)
    assert torch.equal(out, out2)


def test_merge_of_empty_rows_and_bf16_output():
    w = wl.make_workload("cp", [300, 0, 64], 8, 2, 64, seed=32)
    ref_out, ref_lse = oracle_of(w)
    outs, lses = shards_of(w, 4, da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=64))
    shape = da.shape_of_workload(to_device(w), out_dtype=da.DA_DTYPE_BF16)
    out = torch.full((3, 8, 64), float("nan"), device="cuda", dtype=torch.bfloat16)
    lse = torch.full((3, 8), float("nan"), device="cuda")
    da.decode_attn_merge_shards(shape, 4, outs, lses, out, lse)
    assert not out[1].any() and torch.isneginf(lse[1]).all()                       # a row with no tokens anywhere
    want = torch.from_numpy(ref_out).to(torch.bfloat16).float()
    assert float((out.float().cpu() - want).abs().max()) <= 2.0 ** -7 * float(want.abs().max())   # one bf16 step


def test_merge_refuses_bad_arguments():
    w = to_device(wl.config_tiny())
    shape = da.shape_of_workload(w)
    outs = torch.zeros((2, 4, 8, 64), device="cuda")
    lses = torch.zeros((2, 4, 8), device="cuda")
    out = torch.zeros((4, 8, 64), device="cuda")
    assert da.decode_attn_merge_shards(shape, 0, outs, lses, out, None, check=False) == da.DA_ERR_INVALID_ARG
    assert da.decode_attn_merge_shards(shape, 2, None, lses, out, None, check=False) == da.DA_ERR_INVALID_ARG
    assert da.decode_attn_merge_shards(shape, 2, outs.data_ptr() + 4, lses, out, None, check=False) == da.DA_ERR_INVALID_ARG
