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


PREFIX_KERNELS = [da.DA_KERNEL_MMA_TMA, da.DA_KERNEL_UMMA_PREFIX]
PREFIX_KERNEL_IDS = ["mma_sync", "tcgen05"]


def policy(prefix, kernel=da.DA_KERNEL_MMA_TMA, **kw):
    return da.make_policy(shared_prefix_tokens=prefix, kernel=kernel, **kw)


def check(w, pol, run_mask=None):
    ref_out, ref_lse = oracle_of(w, run_mask=run_mask)
    mask = None if run_mask is None else torch.tensor(run_mask, dtype=torch.uint8, device="cuda")
    out, lse = da.run_workload(to_device(w), pol, run_mask=mask)
    return assert_parity(out, lse, ref_out, ref_lse), out, lse


@pytest.mark.parametrize("kernel", PREFIX_KERNELS, ids=PREFIX_KERNEL_IDS)
@pytest.mark.parametrize("batch,prefix", [(12, 512), (5, 128), (1, 256), (33, 1536), (70, 400 * 16)])
def test_reduced_few_shot_batches(batch, prefix, kernel):
    w = wl.config_shared_prefix(batch=batch, prefix=prefix)
    check(w, policy(prefix, kernel))
    check(w, policy(prefix, kernel, split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=128))
    check(w, policy(prefix, kernel, split_mode=da.DA_SPLIT_DETERMINISTIC))


@pytest.mark.parametrize("kernel", PREFIX_KERNELS, ids=PREFIX_KERNEL_IDS)
def test_full_few_shot_configuration(kernel):
    w = wl.config_shared_prefix()
    assert da.decode_attn_validate_shared_prefix(da.shape_of_workload(w), 1536, w.seq_lens, w.block_table) == da.DA_OK
    check(w, policy(1536, kernel))


@pytest.mark.parametrize("hq,hkv", [(8, 8), (16, 8), (32, 8), (16, 2), (24, 8), (10, 2), (12, 2), (28, 4), (18, 2), (48, 4),
                                    (13, 1), (128, 8)])
def test_tcgen05_prefix_groups(hq, hkv):
    """Groups of 1 to 16 heads (128 rows hold floor(128 / G) sequences; where G does not divide 128
    the last rows of a unit stay empty; what follows the prefix runs on the mma.sync kernel, with two
    tiles of heads above 8); a prefix that is not a whole number of 128-token tiles
    (zero-filled tail pages) and more sequences than one 128-row block holds."""
    prefix = 13 * 16
    lens = [prefix + x for x in ([0, 1, 16, 17, 100, 255, 300, 31, 64] * (3 if hq // hkv >= 5 else 1))]
    if hq // hkv == 1:
        lens = lens * 15                     # 135 sequences: two blocks of rows at one head per sequence
    w = wl.make_workload("p", lens, hq, hkv, 128, seed=29, shared_prefix_tokens=prefix)
    check(w, policy(prefix, da.DA_KERNEL_UMMA_PREFIX))


def test_tcgen05_prefix_long_units_and_few_blocks():
    """A planner told of 8 SMs leaves the whole 6,400-token prefix to one unit (50 tiles: the stage
    ring and the tensor-memory buffers wrap many times) and runs the 16 units of the two sequence
    blocks on 8 persistent thread blocks (two units each, barriers set up again in between)."""
    w = wl.config_shared_prefix(batch=40, prefix=6400)
    pol = policy(6400, da.DA_KERNEL_UMMA_PREFIX, sm_count=8)
    plan = da.decode_attn_plan(da.shape_of_workload(w), pol, w.seq_lens)
    front = [u for u in da.decode_attn_plan_get_units(plan) if u.kv_head >> 16]
    assert len(front) == 16 and all(u.tok_end - u.tok_begin == 6400 for u in front)
    plan.destroy()
    check(w, pol)


def test_tcgen05_prefix_refuses_what_it_cannot_run():
    w = wl.make_workload("p", [300, 400], 8, 2, 64, seed=1, shared_prefix_tokens=256)      # head_dim 64
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_plan(da.shape_of_workload(w), policy(256, da.DA_KERNEL_UMMA_PREFIX), w.seq_lens)
    assert e.value.status == da.DA_ERR_UNSUPPORTED
    w = wl.make_workload("p", [300, 400], 32, 8, 128, seed=1)                              # no shared prefix
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_plan(da.shape_of_workload(w), da.make_policy(kernel=da.DA_KERNEL_UMMA_PREFIX), w.seq_lens)
    assert e.value.status == da.DA_ERR_UNSUPPORTED


@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 64), (16, 8, 128), (8, 8, 128), (24, 8, 64)])
def test_other_groups_and_head_dims(hq, hkv, d):
    lens = [256 + x for x in (0, 1, 16, 17, 100, 255, 300, 31, 64)]      # one sequence is the bare prefix
    w = wl.make_workload("p", lens, hq, hkv, d, seed=23, shared_prefix_tokens=256)
    check(w, policy(256))


@pytest.mark.parametrize("kernel", PREFIX_KERNELS, ids=PREFIX_KERNEL_IDS)
def test_masked_rows_inside_a_block_emit_zero(kernel):
    w = wl.config_shared_prefix(batch=10, prefix=256)
    mask = [1, 0, 1, 1, 0, 0, 0, 0, 1, 0]
    _, out, lse = check(w, policy(256, kernel), run_mask=mask)
    for b, keep in enumerate(mask):
        if not keep:
            assert not out[b].any() and torch.isneginf(lse[b]).all()


@pytest.mark.parametrize("kernel", PREFIX_KERNELS, ids=PREFIX_KERNEL_IDS)
def test_prefix_and_plain_plans_agree(kernel):
    w = to_device(wl.config_shared_prefix(batch=16, prefix=512))
    a, la = da.run_workload(w, policy(512, kernel))
    b, lb = da.run_workload(w, da.make_policy())
    assert float((a - b).abs().max()) < 1e-3 and float((la - lb).abs().max()) < 1e-3


@pytest.mark.parametrize("kernel", PREFIX_KERNELS, ids=PREFIX_KERNEL_IDS)
def test_stale_lengths_are_reported(kernel):
    w = to_device(wl.config_shared_prefix(batch=6, prefix=256))
    pol = policy(256, kernel)
    plan = da.decode_attn_plan(da.shape_of_workload(w), pol, w.seq_lens)
    out = torch.zeros((6, 32, 128), dtype=torch.float32, device="cuda")
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device="cuda")
    lens = w.seq_lens.clone()
    lens[4] += 1
    da.decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, w.block_table, lens, out, None, ws, plan.workspace_bytes)
    da.decode_attn_combine(plan, ws, out)
    assert da.decode_attn_last_device_status(plan) == da.DA_ERR_STALE_PLAN
