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


@pytest.mark.parametrize("fused", [0, 1])
@pytest.mark.parametrize("lens", [[300, 5000, 64, 1200], [40000]])
def test_a_bounded_wait_that_runs_out_is_reported_and_the_plan_recovers(fused, lens):
    """The waits of the tensor-core kernel (consumers on a stage's arrival, the producer on its
    release, the merge blocks on a group's records) all carry a limit.  The test hook withholds
    the producer's loads and cuts the limit to about a millisecond: nothing is at fault, the waits
    simply run out.  The launch must come back by itself, report DA_ERR_TIMEOUT, and leave the plan
    and the context good for the next ordinary launch."""
    import time
    from gpu_util import assert_parity, oracle_of
    w = to_device(wl.make_workload("expire", lens, 32, 8, 128, seed=53))
    plan = da.decode_attn_plan(da.shape_of_workload(w), da.make_policy(kernel=da.DA_KERNEL_MMA_TMA, fuse_combine=fused),
                               w.seq_lens)
    out = torch.zeros((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32, device="cuda")
    lse = torch.zeros((w.batch, w.num_q_heads), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device="cuda")
    args = (w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, out, lse, ws, plan.workspace_bytes)
    t0 = time.perf_counter()
    assert da.decode_attn_debug_expire_wait(plan, *args, limit_cycles=2_000_000) == da.DA_OK
    assert da.decode_attn_last_device_status(plan) == da.DA_ERR_TIMEOUT      # synchronises: the launch returned
    assert time.perf_counter() - t0 < 5.0                                    # long before the ordinary one-second limits add up
    assert da.decode_attn_last_device_status(plan) == da.DA_OK               # cleared by the read
    # the very same plan, an ordinary launch: clean status, correct result
    da.decode_attn_run(plan, *args)
    if not fused:
        da.decode_attn_combine(plan, ws, out, lse)
    assert da.decode_attn_last_device_status(plan) == da.DA_OK
    ref_out, ref_lse = oracle_of(to_device(w, "cpu"))
    assert_parity(out, lse, ref_out, ref_lse)
    # the hook refuses what it does not cover, and a non-positive limit
    assert da.decode_attn_debug_expire_wait(plan, *args, limit_cycles=0) == da.DA_ERR_INVALID_ARG
    simt = da.decode_attn_plan(da.shape_of_workload(w), da.make_policy(kernel=da.DA_KERNEL_SIMT), w.seq_lens)
    assert da.decode_attn_debug_expire_wait(simt, *args[:8], simt.workspace_bytes) in (da.DA_ERR_UNSUPPORTED,
                                                                                       da.DA_ERR_WORKSPACE_TOO_SMALL)


def test_a_plan_may_be_destroyed_while_its_kernels_are_still_queued():
    """A step is plan / run / combine / destroy with no synchronisation in between.  The next
    plan takes the destroyed plan's device buffer from the library's cache and uploads its own
    work list there: that upload has to wait, on the device, for the first plan's kernels."""
    from gpu_util import oracle_of
    a = wl.config_sweep_cell(2048, 64, device="cuda")                  # ~80 us of kernel time queued behind one another
    b = to_device(wl.make_workload("other", [700, 33, 5000, 16, 1800], 32, 8, 128, seed=77))
    want_a, want_a_lse = da.run_workload(a, da.make_policy())
    want_b, want_b_lse = da.run_workload(b, da.make_policy())
    torch.cuda.synchronize()
    for _ in range(20):
        outs = []
        for w in (a, b, a, b):
            plan = da.decode_attn_plan(da.shape_of_workload(w), da.make_policy(), w.seq_lens)
            out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
            lse = torch.full((w.batch, w.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
            ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device="cuda")
            da.decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, out, lse, ws,
                               plan.workspace_bytes)
            da.decode_attn_combine(plan, ws, out, lse)
            plan.destroy()                                              # kernels still queued or running
            outs.append((out, lse, ws))
        torch.cuda.synchronize()
        assert torch.equal(outs[0][0], want_a) and torch.equal(outs[2][0], want_a)
        assert torch.equal(outs[1][0], want_b) and torch.equal(outs[3][0], want_b)
        assert torch.equal(outs[0][1], want_a_lse) and torch.equal(outs[3][1], want_b_lse)
