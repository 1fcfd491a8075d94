"""Shared-prefix planning: batches whose sequences start with the same cached
prefix (the few-shot workload, served from the prefix cache in the paper's
engine, Appendix J) attend the prefix once per block of sequences.  Same
oracle, same tolerance; the records of prefix and own-suffix units meet in
the combine kernel."""
import numpy as np
import pytest
import torch

from paper_2609_37062_b200 import workloads as wl
from gpu_util import assert_parity, da, oracle_of, to_device

pytestmark = pytest.mark.gpu


def policy(prefix, **kw):
    return da.make_policy(shared_prefix_tokens=prefix, kernel=da.DA_KERNEL_MMA_TMA, **kw)


def check(w, pol, run_mask=None):
    ref_out, ref_lse = oracle_of(w, run_mask=run_mask)
    mask = None if run_mask is None else torch.tensor(run_mask, dtype=torch.uint8, device="cuda")
    out, lse = da.run_workload(to_device(w), pol, run_mask=mask)
    return assert_parity(out, lse, ref_out, ref_lse), out, lse


@pytest.mark.parametrize("batch,prefix", [(12, 512), (5, 128), (1, 256), (33, 1536)])
def test_reduced_few_shot_batches(batch, prefix):
    w = wl.config_shared_prefix(batch=batch, prefix=prefix)
    check(w, policy(prefix))
    check(w, policy(prefix, split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=128))


def test_full_few_shot_configuration():
    w = wl.config_shared_prefix()
    assert da.decode_attn_validate_shared_prefix(da.shape_of_workload(w), 1536, w.seq_lens, w.block_table) == da.DA_OK
    check(w, policy(1536))


@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 64), (16, 8, 128), (8, 8, 128), (24, 8, 64)])
def test_other_groups_and_head_dims(hq, hkv, d):
    lens = [256 + x for x in (0, 1, 16, 17, 100, 255, 300, 31, 64)]      # one sequence is the bare prefix
    w = wl.make_workload("p", lens, hq, hkv, d, seed=23, shared_prefix_tokens=256)
    check(w, policy(256))


def test_masked_rows_inside_a_block_emit_zero():
    w = wl.config_shared_prefix(batch=10, prefix=256)
    mask = [1, 0, 1, 1, 0, 0, 0, 0, 1, 0]
    _, out, lse = check(w, policy(256), run_mask=mask)
    for b, keep in enumerate(mask):
        if not keep:
            assert not out[b].any() and torch.isneginf(lse[b]).all()


def test_prefix_and_plain_plans_agree():
    w = to_device(wl.config_shared_prefix(batch=16, prefix=512))
    a, la = da.run_workload(w, policy(512))
    b, lb = da.run_workload(w, da.make_policy())
    assert float((a - b).abs().max()) < 1e-3 and float((la - lb).abs().max()) < 1e-3


def test_stale_lengths_are_reported():
    w = to_device(wl.config_shared_prefix(batch=6, prefix=256))
    pol = policy(256)
    plan = da.decode_attn_plan(da.shape_of_workload(w), pol, w.seq_lens)
    out = torch.zeros((6, 32, 128), dtype=torch.float32, device="cuda")
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device="cuda")
    lens = w.seq_lens.clone()
    lens[4] += 1
    da.decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, w.block_table, lens, out, None, ws, plan.workspace_bytes)
    da.decode_attn_combine(plan, ws, out)
    assert da.decode_attn_last_device_status(plan) == da.DA_ERR_STALE_PLAN
