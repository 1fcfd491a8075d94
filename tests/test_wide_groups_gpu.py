"""Groups of 9 to 16 query heads per KV head (large models shard down to such
ratios): the tensor-core kernel attends them as two 8-column tiles of heads
per K/V tile.  Same oracle, same tolerance: every split mode, fused and
separate merge, both head dimensions and input types, ragged lengths with
poisoned padding, a run mask, and bit-equal results across batch compositions
in the deterministic mode."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_37062_b200 import workloads as wl
from gpu_util import assert_parity, check_workload, da, oracle_of, to_device

pytestmark = pytest.mark.gpu

MMA = da.DA_KERNEL_MMA_TMA
POLICIES = [("auto", dict()), ("auto_fused", dict(fuse_combine=1)),
            ("fixed1", dict(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=1)),
            ("fixed5", dict(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=5)),
            ("det16", dict(split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=16)),
            ("det_default_fused", dict(split_mode=da.DA_SPLIT_DETERMINISTIC, fuse_combine=1))]


@pytest.mark.parametrize("name,pol", POLICIES, ids=[p[0] for p in POLICIES])
@pytest.mark.parametrize("hq,hkv,d", [(18, 2, 128), (20, 2, 64), (24, 2, 128), (26, 2, 64), (32, 2, 128),
                                      (32, 2, 64), (128, 8, 128), (11, 1, 128)])
def test_wide_group_parity(name, pol, hq, hkv, d):
    w = wl.make_workload("wide", [200, 31, 1000, 0, 16, 4133], hq, hkv, d, seed=31)
    check_workload(w, da.make_policy(kernel=MMA, **pol), what=f"{name} G={hq // hkv} D={d}")
    check_workload(w, da.make_policy(**pol), what=f"{name} auto kernel G={hq // hkv} D={d}")


@pytest.mark.parametrize("g", [9, 12, 16])
def test_wide_group_fp16_and_head_major(g):
    lens = [1, 16, 33, 700, 2049, 0, 255]
    for layout in ("token_major", "head_major"):
        for dtype in ("bf16", "fp16"):
            w = wl.make_workload("wide16", lens, 2 * g, 2, 128, seed=7, layout=layout, dtype=dtype)
            check_workload(w, da.make_policy(), what=f"G={g} {layout} {dtype}")


@pytest.mark.parametrize("g", [10, 16])
def test_wide_group_edge_lengths_with_poisoned_padding(g):
    lens = [0, 1, 15, 16, 17, 31, 32, 33, 63, 64, 65, 255, 256, 257, 1023, 1024, 1025]
    w = wl.make_workload("wide_edges", lens, 2 * g, 2, 128, seed=5, pool_pages=400)
    ref_out, ref_lse = oracle_of(w)
    for pol in (dict(), dict(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=3, fuse_combine=1),
                dict(split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=16)):
        out, lse = da.run_workload(to_device(w), da.make_policy(**pol))
        assert_parity(out, lse, ref_out, ref_lse, str(pol))
        assert not out[0].any() and torch.isneginf(lse[0]).all()


def test_wide_group_sharp_rows_keep_their_precision():
    """One dominant token per row: the low part of the weights must reach both tiles of heads."""
    w = wl.make_workload("wide_sharp", [1500, 900], 32, 2, 128, seed=3)
    ref_out, _ = oracle_of(w, scale=1.0)
    out, _ = da.run_workload(to_device(w), da.make_policy(), sm_scale=1.0)
    diff = np.abs(out.double().cpu().numpy() - ref_out)
    assert diff.max() < 2e-4, diff.max()


@pytest.mark.parametrize("g", [12, 16])
def test_wide_group_run_mask(g):
    """Masked rows emit zeros and lse = -inf whatever their pages hold; enough rows are masked for the
    kernel to deal the work list out again."""
    lens = wl.lengths_short_chat(40, 4)
    w = wl.make_workload("wide_mask", lens, 4 * g, 4, 128, seed=2)
    for every in (2, 5):
        mask = [i % every != 0 for i in range(len(lens))]
        ref_out, ref_lse = oracle_of(w, run_mask=mask)
        for pol in (dict(), dict(fuse_combine=1), dict(split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=128)):
            out, lse = da.run_workload(to_device(w), da.make_policy(**pol),
                                       run_mask=torch.tensor(mask, dtype=torch.uint8, device="cuda"))
            assert_parity(out, lse, ref_out, ref_lse, f"every {every} {pol}")
            assert not out[0].any() and torch.isneginf(lse[0]).all()


def test_wide_group_deterministic_mode_is_bit_equal_across_batches():
    lens = [3000, 517, 64, 1, 2222, 900, 31, 4096]
    pol = da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=256)

    def run(rows, table_seed):
        w = wl.make_workload("wide_det", [lens[r] for r in rows], 48, 4, 128, seed=11, seq_uids=rows,
                             table_seed=table_seed, device="cuda")
        return da.run_workload(w, pol)

    full, full_lse = run(list(range(len(lens))), 1)
    for k, rows in enumerate(([0], [4, 1], [7, 6, 5, 3], [2, 0, 4])):
        out, lse = run(rows, 2 + k)
        for i, r in enumerate(rows):
            assert torch.equal(out[i], full[r]) and torch.equal(lse[i], full_lse[r]), (rows, r)


def test_wide_group_static_step_host_step_and_captured_capacity_plan():
    w = wl.make_workload("wide_s", [900, 40, 333, 0, 2100], 64, 4, 128, seed=49)
    ref_out, ref_lse = oracle_of(w)
    wd = to_device(w)
    s = da.shape_of_workload(wd)
    out = torch.empty((w.batch, 64, 128), dtype=torch.float32, device="cuda")
    lse = torch.empty((w.batch, 64), dtype=torch.float32, device="cuda")
    da.decode_attn_step_static(s, w.seq_lens, wd.q_bits, wd.k_pool, wd.v_pool, wd.block_table, wd.seq_lens, out, lse)
    torch.cuda.synchronize()
    assert_parity(out, lse, ref_out, ref_lse, "static step")
    hout = torch.empty((w.batch, 64, 128), dtype=torch.float32).pin_memory()
    da.decode_attn_host_step(s, da.make_policy(), w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, hout)
    da.decode_attn_host_release()
    assert_parity(hout, None, ref_out, ref_lse, "host step")
    # a capacity plan captured once and replayed (buffers sized for the capacity, fixed addresses)
    cap = 8

    def padded(t):
        full = torch.zeros((cap,) + tuple(t.shape[1:]), dtype=t.dtype, device="cuda")
        full[: t.shape[0]] = t.cuda()
        return full

    pol = da.make_policy(capacity_batch=cap, capacity_tokens=16384, fuse_combine=1)
    plan = da.decode_attn_plan(s, pol, w.seq_lens)
    q, bt, sl = padded(w.q_bits), padded(w.block_table), padded(w.seq_lens)
    cout = torch.zeros((cap, 64, 128), dtype=torch.float32, device="cuda")
    clse = torch.zeros((cap, 64), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        da.decode_attn_run(plan, q, wd.k_pool, wd.v_pool, bt, sl, cout, clse, ws, plan.workspace_bytes)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            da.decode_attn_run(plan, q, wd.k_pool, wd.v_pool, bt, sl, cout, clse, ws, plan.workspace_bytes)
        cout.zero_()
        graph.replay()
        stream.synchronize()
    assert da.decode_attn_last_device_status(plan) == da.DA_OK
    assert_parity(cout[: w.batch], clse[: w.batch], ref_out, ref_lse, "captured capacity plan")
    plan.destroy()


def test_wide_groups_are_refused_where_unsupported():
    w = wl.make_workload("wide_no", [100, 300], 24, 2, 128, seed=1)
    with pytest.raises(da.DecodeAttnError) as e:
        da.run_workload(to_device(w), da.make_policy(kernel=da.DA_KERNEL_SIMT))
    assert e.value.status == da.DA_ERR_UNSUPPORTED
    w = wl.make_workload("wide_no", [100, 300], 34, 2, 128, seed=1)        # a group of 17
    with pytest.raises(da.DecodeAttnError) as e:
        da.run_workload(to_device(w), da.make_policy())
    assert e.value.status == da.DA_ERR_UNSUPPORTED
