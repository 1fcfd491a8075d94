"""Parity at the benchmark's sizes, in the launch configuration bench.py
times (AUTO split, tensor-core kernel, combine kernel): the whole batch
against the oracle where the oracle finishes in seconds, sampled sequences
where it does not, and bitwise determinism of a sequence across batch sizes
at full contexts."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2609_37062_b200 import workloads as wl
from gpu_util import assert_parity, da, oracle_of, to_device

pytestmark = pytest.mark.gpu


def extract_sequences(w, idxs):
    """Host copy of the sequences `idxs` of a device workload: their pages are
    gathered (bit for bit) into a small pool with an identity block table."""
    P = w.page_size
    lens = [int(w.seq_lens[i]) for i in idxs]
    pages = [(l + P - 1) // P for l in lens]
    total = max(sum(pages), 1)
    k = torch.empty((total,) + tuple(w.k_pool.shape[1:]), dtype=torch.int16)
    v = torch.empty_like(k)
    bt = torch.full((len(idxs), max(max(pages), 1)), -1, dtype=torch.int32)
    cur = 0
    for r, (i, n) in enumerate(zip(idxs, pages)):
        ids = w.block_table[i, :n].long()
        k[cur:cur + n] = w.k_pool[ids].cpu()
        v[cur:cur + n] = w.v_pool[ids].cpu()
        bt[r, :n] = torch.arange(cur, cur + n, dtype=torch.int32)
        cur += n
    return dataclasses.replace(w, batch=len(idxs), num_pages=total, max_pages_per_seq=bt.shape[1],
                               seq_lens=torch.tensor(lens, dtype=torch.int32), block_table=bt,
                               q_bits=w.q_bits[idxs].cpu(), k_pool=k, v_pool=v)


def bench_policy(**kw):
    return da.make_policy(**kw)        # AUTO split, AUTO kernel (tensor cores at G = 4), combine kernel


def test_long_sequence_full_size():
    w = wl.config_long(device="cuda")
    out, lse = da.run_workload(w, bench_policy())
    ref_out, ref_lse = oracle_of(to_device(w, "cpu"))
    assert_parity(out, lse, ref_out, ref_lse, "long_32k")
    fused, fused_lse = da.run_workload(w, bench_policy(fuse_combine=1))
    assert torch.equal(out, fused) and torch.equal(lse, fused_lse)


def test_short_chat_full_size():
    w = wl.config_short_chat(device="cuda")
    out, lse = da.run_workload(w, bench_policy())
    ref_out, ref_lse = oracle_of(to_device(w, "cpu"))
    assert_parity(out, lse, ref_out, ref_lse, "short_chat")


def test_shared_prefix_full_size():
    w = wl.config_shared_prefix(device="cuda")
    out, lse = da.run_workload(w, bench_policy())
    ref_out, ref_lse = oracle_of(to_device(w, "cpu"))
    assert_parity(out, lse, ref_out, ref_lse, "shared_prefix")


@pytest.mark.parametrize("context,batch", [(512, 256), (2048, 64), (8192, 64), (32768, 8), (131072, 2), (16384, 64)])
def test_sweep_cells_on_sampled_sequences(context, batch):
    """First, last and two seeded picks of the cell, one by one against the oracle.  (16,384 x 64 is
    a cell whose 512 whole-sequence units do not divide over the resident blocks: the planner cuts
    every sequence in four.)"""
    w = wl.config_sweep_cell(context, batch, device="cuda")
    if (context, batch) == (16384, 64):
        plan = da.decode_attn_plan(da.shape_of_workload(w), bench_policy(), w.seq_lens)
        assert plan.info().n_units == 2048 and plan.info().chunk_tokens == 4096
        plan.destroy()
    out, lse = da.run_workload(w, bench_policy())
    g = torch.Generator().manual_seed(context + batch)
    picks = sorted({0, batch - 1, *torch.randint(0, batch, (2,), generator=g).tolist()})
    sub = extract_sequences(w, picks)
    ref_out, ref_lse = oracle_of(sub)
    assert_parity(out[picks], lse[picks], ref_out, ref_lse, f"{context}x{batch}")
    assert torch.isfinite(out).all()


@pytest.mark.parametrize("context,batches", [(512, (256, 64, 8, 1)), (2048, (256, 64, 8, 1)), (8192, (256, 64, 8, 1)),
                                             (32768, (64, 8, 1)), (131072, (8, 2, 1))])
def test_deterministic_mode_every_sequence_across_batch_sizes(context, batches):
    """Sequence i has the same content in every batch size of a sweep cell (and other page
    placement): in deterministic mode every sequence of every smaller batch must come out with the
    bits it has in the largest one."""
    pol = da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC)
    big = None
    for b in batches:
        w = wl.config_sweep_cell(context, b, device="cuda", table_seed=b)
        out, lse = da.run_workload(w, pol)
        if big is None:
            big = (out, lse)
            picks = sorted({0, b - 1, b // 3})
            ref_out, ref_lse = oracle_of(extract_sequences(w, picks))
            assert_parity(out[picks], lse[picks], ref_out, ref_lse)
        else:
            assert torch.equal(out, big[0][:b]) and torch.equal(lse, big[1][:b]), (context, b)
        del w
