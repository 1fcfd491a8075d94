"""Failure detection without faulting the GPU: bad arguments are refused on
the host with a status code and no launch; stale lengths and page ids outside
the pool are caught by the kernels, recorded in the status word and skipped."""
import pytest
import torch

from paper_2609_37062_b200 import workloads as wl
from gpu_util import KERNELS, KERNEL_IDS, da, to_device

pytestmark = pytest.mark.gpu


def setup(kernel=da.DA_KERNEL_AUTO, **pol):
    w = to_device(wl.config_tiny())
    policy = da.make_policy(kernel=kernel, **pol)
    plan = da.decode_attn_plan(da.shape_of_workload(w), policy, w.seq_lens)
    out = torch.zeros((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device="cuda")
    return w, plan, out, ws


def test_null_and_misaligned_pointers_are_refused():
    w, plan, out, ws = setup(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=2)
    args = [w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, out]
    for i in range(6):
        a = list(args)
        a[i] = None
        rc = da.decode_attn_run(plan, *a, None, ws, plan.workspace_bytes, check=False)
        assert rc == da.DA_ERR_INVALID_ARG
    rc = da.decode_attn_run(plan, w.q_bits.data_ptr() + 2, *args[1:], None, ws, plan.workspace_bytes, check=False)
    assert rc == da.DA_ERR_INVALID_ARG
    rc = da.decode_attn_run(plan, *args, None, ws.data_ptr() + 16, plan.workspace_bytes, check=False)
    assert rc == da.DA_ERR_INVALID_ARG
    rc = da.decode_attn_run(plan, *args, None, None, 0, check=False)
    assert rc == da.DA_ERR_INVALID_ARG
    rc = da.decode_attn_run(plan, *args, None, ws, plan.workspace_bytes - 1, check=False)
    assert rc == da.DA_ERR_WORKSPACE_TOO_SMALL
    assert da.decode_attn_combine(plan, None, out, check=False) == da.DA_ERR_INVALID_ARG
    assert da.decode_attn_combine(plan, ws, None, check=False) == da.DA_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert not out.any()                                   # nothing was launched
    assert da.decode_attn_last_device_status(plan) == da.DA_OK


def test_plan_rejects_lengths_longer_than_the_block_table():
    w = to_device(wl.config_tiny())
    lens = w.seq_lens.clone()
    lens[0] = 16 * w.max_pages_per_seq + 1
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_plan(da.shape_of_workload(w), da.make_policy(), lens)
    assert e.value.status == da.DA_ERR_INVALID_ARG


def test_plan_check_reports_stale_lengths_on_the_host():
    w, plan, out, ws = setup()
    assert da.decode_attn_plan_check(plan, w.seq_lens) == da.DA_OK
    lens = w.seq_lens.clone()
    lens[1] += 1
    assert da.decode_attn_plan_check(plan, lens) == da.DA_ERR_STALE_PLAN
    assert da.decode_attn_plan_check(plan, lens[:3]) == da.DA_ERR_STALE_PLAN


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("fused", [0, 1])
def test_stale_device_lengths_are_detected_by_the_kernel(kernel, fused):
    """Invariant 2: a plan made for one set of lengths must not silently run
    on another.  The kernel compares the device lengths with the planned ones,
    records the condition and skips the row's reads."""
    w, plan, out, ws = setup(kernel, fuse_combine=fused, split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=2)
    lens = w.seq_lens.clone()
    lens[2] += 1
    da.decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, w.block_table, lens, out, None, ws, plan.workspace_bytes)
    if not fused:
        da.decode_attn_combine(plan, ws, out)
    assert da.decode_attn_last_device_status(plan) == da.DA_ERR_STALE_PLAN
    assert da.decode_attn_last_device_status(plan) == da.DA_OK          # cleared by the read
    # the same plan still works with the right lengths afterwards
    da.decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, out, None, ws,
                       plan.workspace_bytes)
    if not fused:
        da.decode_attn_combine(plan, ws, out)
    assert da.decode_attn_last_device_status(plan) == da.DA_OK
    assert torch.isfinite(out).all() and out.abs().sum() > 0


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_page_ids_outside_the_pool_are_flagged_not_dereferenced(kernel):
    w, plan, out, ws = setup(kernel)
    for bad in (-1, w.num_pages, 1 << 30):
        bt = w.block_table.clone()
        bt[3, 5] = bad
        da.decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, bt, w.seq_lens, out, None, ws, plan.workspace_bytes)
        da.decode_attn_combine(plan, ws, out)
        assert da.decode_attn_last_device_status(plan) == da.DA_ERR_BAD_PAGE
    bt = w.block_table.clone()
    bt[0, 2] = 1 << 30                                      # beyond the row's pages: never read
    da.decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, bt, w.seq_lens, out, None, ws, plan.workspace_bytes)
    da.decode_attn_combine(plan, ws, out)
    assert da.decode_attn_last_device_status(plan) == da.DA_OK


def test_empty_batch_is_a_no_op():
    w = to_device(wl.config_tiny())
    s = da.shape_of_workload(w)
    s.batch = 0
    plan = da.decode_attn_plan(s, da.make_policy(), [])
    assert plan.workspace_bytes == 0 and plan.info().n_units == 0
    out = torch.zeros(4, device="cuda")
    assert da.decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, out) == da.DA_OK
    assert da.decode_attn_combine(plan, None, out) == da.DA_OK
