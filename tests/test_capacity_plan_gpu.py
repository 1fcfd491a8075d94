"""Capacity plans: a fixed grid whose surplus blocks exit at once (Alg. 1
step 6, "grid exit") and a work list that is refreshed in place, so one
captured CUDA graph serves every live batch up to the capacity - and the
metadata is rebuilt from the current rows every step (Invariant 2)."""
import pytest
import torch

from paper_2609_37062_b200 import workloads as wl
from gpu_util import KERNELS, KERNEL_IDS, assert_parity, da, oracle_of, to_device

pytestmark = pytest.mark.gpu

CAP_B, CAP_TOK = 8, 24000


def build(lens, seed=40):
    """A workload padded to the capacity's shapes: block table [CAP_B, wide], q/out [CAP_B, ...]."""
    w = wl.make_workload("cap", lens, 32, 8, 128, seed=seed, pool_pages=2000, max_pages_per_seq=640)
    return w


def padded(t, rows):
    out = torch.zeros((rows,) + tuple(t.shape[1:]), dtype=t.dtype, device="cuda")
    out[: t.shape[0]] = t.cuda()
    return out


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("fused", [0, 1])
@pytest.mark.parametrize("mode", [da.DA_SPLIT_AUTO, da.DA_SPLIT_DETERMINISTIC])
def test_update_in_place_and_graph_replay(kernel, fused, mode):
    steps = [[3000, 17, 900, 5000], [64], [1000] * 8, [0, 8000, 1], [2500, 2600, 2700, 2800, 2900, 3000]]
    w0 = build(steps[0])
    shape = da.shape_of_workload(w0)
    pol = da.make_policy(split_mode=mode, chunk_tokens=512, kernel=kernel, fuse_combine=fused, capacity_batch=CAP_B,
                         capacity_tokens=CAP_TOK)
    plan = da.decode_attn_plan(shape, pol, w0.seq_lens)
    info = plan.info()
    assert info.grid > 0                                    # a fixed launch shape, whatever the live batch
    # device buffers with fixed addresses, sized for the capacity
    k_pool, v_pool = w0.k_pool.cuda(), w0.v_pool.cuda()
    q = padded(w0.q_bits, CAP_B)
    bt = padded(w0.block_table, CAP_B)
    sl = padded(w0.seq_lens, CAP_B)
    out = torch.zeros((CAP_B, 32, 128), dtype=torch.float32, device="cuda")
    lse = torch.zeros((CAP_B, 32), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device="cuda")

    def launch():
        da.decode_attn_run(plan, q, k_pool, v_pool, bt, sl, out, lse, ws, plan.workspace_bytes)
        if not fused:
            da.decode_attn_combine(plan, ws, out, lse)

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        launch()                                            # warm-up outside capture
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            launch()
        grid0 = plan.info().grid
        for i, lens in enumerate(steps):
            w = build(lens, seed=40 + i)
            k_pool.copy_(w.k_pool)
            v_pool.copy_(w.v_pool)
            q.zero_(); bt.zero_(); sl.zero_()
            q[: len(lens)] = w.q_bits.cuda()
            bt[: len(lens)] = w.block_table.cuda()
            sl[: len(lens)] = w.seq_lens.cuda()
            out.fill_(float("nan"))
            da.decode_attn_plan_update(plan, w.seq_lens, stream)   # Invariant 2: rebuilt from the current rows
            graph.replay()
            stream.synchronize()
            assert da.decode_attn_last_device_status(plan, stream) == da.DA_OK
            assert plan.info().grid == grid0                        # the launch shape never changes
            ref_out, ref_lse = oracle_of(w)
            assert_parity(out[: len(lens)], lse[: len(lens)], ref_out, ref_lse, f"step {i}")
            assert torch.isnan(out[len(lens):]).all()               # rows past the live batch are untouched
    # a graph replayed without refreshing the plan is caught, not silently wrong
    sl[0] += 1
    with torch.cuda.stream(stream):
        graph.replay()
        stream.synchronize()
    assert da.decode_attn_last_device_status(plan, stream) == da.DA_ERR_STALE_PLAN


def test_updates_beyond_the_capacity_are_refused():
    w0 = build([100, 200])
    pol = da.make_policy(capacity_batch=4, capacity_tokens=1000)
    plan = da.decode_attn_plan(da.shape_of_workload(w0), pol, w0.seq_lens)
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_plan_update(plan, [10] * 5)
    assert e.value.status == da.DA_ERR_INVALID_ARG
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_plan_update(plan, [600, 600])
    assert e.value.status == da.DA_ERR_INVALID_ARG
    plain = da.decode_attn_plan(da.shape_of_workload(w0), da.make_policy(), w0.seq_lens)
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_plan_update(plain, [100, 200])
    assert e.value.status == da.DA_ERR_UNSUPPORTED


@pytest.mark.parametrize("fused", [0, 1])
def test_run_mask_in_a_captured_capacity_graph(fused):
    """The paper's deployment: one captured launch for the capacity, a RUN mask that changes every
    step.  With many rows masked the kernel deals the (refreshed) work list out again among all
    blocks of the fixed grid, surplus ones included; rows past the live batch stay untouched."""
    cap_b, cap_tok = 96, 90000
    steps = [([700] * 60, 0.6), ([300, 5, 1200, 64] * 12, 0.5), ([900] * 96, 0.0), ([100] * 7, 0.9), ([500] * 90, 1.0)]
    first = wl.make_workload("capm", steps[0][0], 32, 8, 128, seed=60, pool_pages=6000, max_pages_per_seq=80)
    shape = da.shape_of_workload(first)
    pol = da.make_policy(kernel=da.DA_KERNEL_MMA_TMA, chunk_tokens=128, fuse_combine=fused, capacity_batch=cap_b,
                         capacity_tokens=cap_tok)
    plan = da.decode_attn_plan(shape, pol, first.seq_lens)
    k_pool, v_pool = first.k_pool.cuda(), first.v_pool.cuda()
    q = padded(first.q_bits, cap_b)
    bt = padded(first.block_table, cap_b)
    sl = padded(first.seq_lens, cap_b)
    mask = torch.ones((cap_b,), dtype=torch.uint8, device="cuda")
    out = torch.zeros((cap_b, 32, 128), dtype=torch.float32, device="cuda")
    lse = torch.zeros((cap_b, 32), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device="cuda")

    def launch():
        da.decode_attn_run(plan, q, k_pool, v_pool, bt, sl, out, lse, ws, plan.workspace_bytes, run_mask=mask)
        if not fused:
            da.decode_attn_combine(plan, ws, out, lse)

    stream = torch.cuda.Stream()
    rng = torch.Generator().manual_seed(5)
    with torch.cuda.stream(stream):
        launch()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            launch()
        for i, (lens, frac) in enumerate(steps):
            w = wl.make_workload("capm", lens, 32, 8, 128, seed=61 + i, pool_pages=6000, max_pages_per_seq=80)
            host_mask = (torch.rand(len(lens), generator=rng) >= frac).to(torch.uint8)
            k_pool.copy_(w.k_pool)
            v_pool.copy_(w.v_pool)
            q.zero_(); bt.zero_(); sl.zero_(); mask.fill_(1)
            q[: len(lens)] = w.q_bits.cuda()
            bt[: len(lens)] = w.block_table.cuda()
            sl[: len(lens)] = w.seq_lens.cuda()
            mask[: len(lens)] = host_mask.cuda()
            out.fill_(float("nan"))
            da.decode_attn_plan_update(plan, w.seq_lens, stream)
            graph.replay()
            stream.synchronize()
            assert da.decode_attn_last_device_status(plan, stream) == da.DA_OK
            ref_out, ref_lse = oracle_of(w, run_mask=host_mask.numpy())
            assert_parity(out[: len(lens)], lse[: len(lens)], ref_out, ref_lse, f"step {i}")
            assert torch.isnan(out[len(lens):]).all()
    plan.destroy()
