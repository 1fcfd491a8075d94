"""Own-layer KV write on the GPU (Invariant 1; Alg. 1 step 2, first half):
bit-exact against the oracle's byte copy, and seen by the attention launch
that follows it on the same stream - for masked rows too."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_37062_b200 import workloads as wl
from gpu_util import assert_parity, da, to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("layout", ["token_major", "head_major"])
@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 64), (32, 8, 128), (24, 2, 128)])
def test_append_then_attend(layout, hq, hkv, d):
    lens = [1, 16, 17, 300, 0, 1024, 1025, 77]
    w = wl.make_workload("append", lens, hq, hkv, d, seed=17, layout=layout, pool_pages=300)
    B = len(lens)
    new_k = wl.normal_bf16_bits(wl.stream_key(17, wl.TENSOR_NEW_K, 0), 0, B * hkv * d).view(B, hkv, d)
    new_v = wl.normal_bf16_bits(wl.stream_key(17, wl.TENSOR_NEW_V, 0), 0, B * hkv * d).view(B, hkv, d)
    inp = oracle.PagedInputs.from_workload(w)
    k_ref, v_ref = oracle.append_kv(inp, new_k, new_v)
    wd = to_device(w)
    shape = da.shape_of_workload(wd)
    mask = torch.tensor([1, 0, 1, 0, 1, 1, 0, 1], dtype=torch.uint8, device="cuda")
    plan = da.decode_attn_plan(shape, da.make_policy(chunk_tokens=256), w.seq_lens)
    out = torch.empty((B, hq, d), dtype=torch.float32, device="cuda")
    lse = torch.empty((B, hq), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device="cuda")
    # write, then attend, back to back on one stream
    da.decode_attn_append_kv(shape, new_k.cuda(), new_v.cuda(), wd.block_table, wd.seq_lens, wd.k_pool, wd.v_pool)
    da.decode_attn_run(plan, wd.q_bits, wd.k_pool, wd.v_pool, wd.block_table, wd.seq_lens, out, lse, ws,
                       plan.workspace_bytes, run_mask=mask)
    da.decode_attn_combine(plan, ws, out, lse)
    assert da.decode_attn_last_device_status(plan) == da.DA_OK
    # the pools: bit for bit, masked rows included (every layer writes its own KV)
    assert np.array_equal(wd.k_pool.cpu().numpy().view(np.uint16).ravel(), k_ref.ravel())
    assert np.array_equal(wd.v_pool.cpu().numpy().view(np.uint16).ravel(), v_ref.ravel())
    # attention over the appended cache
    w.k_pool = torch.from_numpy(k_ref.view(np.int16).reshape(tuple(w.k_pool.shape)))
    w.v_pool = torch.from_numpy(v_ref.view(np.int16).reshape(tuple(w.v_pool.shape)))
    ref_out, ref_lse = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w), run_mask=mask.cpu().numpy())
    assert_parity(out, lse, ref_out, ref_lse)


def test_append_rejects_bad_arguments_and_skips_bad_pages():
    w = to_device(wl.config_tiny())
    shape = da.shape_of_workload(w)
    nk = torch.zeros((4, 2, 64), dtype=torch.int16, device="cuda")
    assert da.decode_attn_append_kv(shape, None, nk, w.block_table, w.seq_lens, w.k_pool, w.v_pool,
                                    check=False) == da.DA_ERR_INVALID_ARG
    assert da.decode_attn_append_kv(shape, nk.data_ptr() + 2, nk, w.block_table, w.seq_lens, w.k_pool, w.v_pool,
                                    check=False) == da.DA_ERR_INVALID_ARG
    before = w.k_pool.clone()
    bt = w.block_table.clone()
    bt[:, :] = 1 << 30                                   # every mapping points outside the pool
    da.decode_attn_append_kv(shape, nk, nk, bt, w.seq_lens, w.k_pool, w.v_pool)
    torch.cuda.synchronize()
    assert torch.equal(before, w.k_pool)                 # nothing was written, nothing faulted


def test_checked_append_reports_rows_it_could_not_write():
    """Invariant 1 is only kept if a dropped write is known: with a plan given, a row whose page
    id lies outside the pool is skipped (nothing faults) and reported through the plan's status."""
    w = to_device(wl.config_tiny())
    plan = da.decode_attn_plan(da.shape_of_workload(w), da.make_policy(), w.seq_lens)
    nk = wl.normal_bf16_bits(wl.stream_key(3, wl.TENSOR_NEW_K, 0), 0, 4 * 2 * 64).view(4, 2, 64).cuda()
    before = w.k_pool.clone()
    da.decode_attn_append_kv_checked(plan, nk, nk, w.block_table, w.seq_lens, w.k_pool, w.v_pool)
    assert da.decode_attn_last_device_status(plan) == da.DA_OK
    assert not torch.equal(before, w.k_pool)
    bt = w.block_table.clone()
    last = (int(w.seq_lens[2]) - 1) // w.page_size
    bt[2, last] = w.num_pages                                # one row's last page: outside the pool
    mid = w.k_pool.clone()
    da.decode_attn_append_kv_checked(plan, nk, nk, bt, w.seq_lens, w.k_pool, w.v_pool)
    assert da.decode_attn_last_device_status(plan) == da.DA_ERR_BAD_PAGE
    assert torch.equal(mid, w.k_pool)                        # the other rows rewrote the same bytes, row 2 wrote nothing
    assert da.decode_attn_last_device_status(plan) == da.DA_OK


@pytest.mark.parametrize("page_size", [16, 64])
@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 64), (32, 8, 128), (64, 8, 128), (96, 8, 128)])
@pytest.mark.parametrize("mode", ["auto", "deterministic", "fixed3"])
def test_fused_write_and_attend_equals_write_then_attend(page_size, hq, hkv, d, mode):
    """Algorithm 1 step 2 in one launch: the attention kernel stores every row's new K/V at
    position seq_len - 1 (masked rows too) and attends over it in the same pass.  Pools and
    outputs must equal, bit for bit, what decode_attn_append_kv followed by an ordinary launch
    gives - and the oracle over the appended cache."""
    lens = [1, 16, 17, 300, 0, 1024, 1025, 77, 4096, 31, 32, 33]
    w = wl.make_workload("fused_append", lens, hq, hkv, d, seed=19, page_size=page_size, pool_pages=900 * 16 // page_size)
    B = len(lens)
    new_k = wl.normal_bf16_bits(wl.stream_key(19, wl.TENSOR_NEW_K, 0), 0, B * hkv * d).view(B, hkv, d).cuda()
    new_v = wl.normal_bf16_bits(wl.stream_key(19, wl.TENSOR_NEW_V, 0), 0, B * hkv * d).view(B, hkv, d).cuda()
    mask = torch.tensor([1, 0, 1, 0, 1, 1, 0, 1, 1, 1, 0, 1], dtype=torch.uint8, device="cuda")
    pol = {"auto": da.make_policy(chunk_tokens=256),
           "deterministic": da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC),
           "fixed3": da.make_policy(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=3)}[mode]
    results = []
    for fused in (False, True):
        for run_mask in (None, mask):
            wd = to_device(w)
            shape = da.shape_of_workload(wd)
            plan = da.decode_attn_plan(shape, pol, w.seq_lens)
            out = torch.full((B, hq, d), float("nan"), dtype=torch.float32, device="cuda")
            lse = torch.full((B, hq), float("nan"), dtype=torch.float32, device="cuda")
            ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device="cuda")
            if fused:
                da.decode_attn_run(plan, wd.q_bits, wd.k_pool, wd.v_pool, wd.block_table, wd.seq_lens, out, lse, ws,
                                   plan.workspace_bytes, run_mask=run_mask, new_k=new_k, new_v=new_v)
            else:
                da.decode_attn_append_kv(shape, new_k, new_v, wd.block_table, wd.seq_lens, wd.k_pool, wd.v_pool)
                da.decode_attn_run(plan, wd.q_bits, wd.k_pool, wd.v_pool, wd.block_table, wd.seq_lens, out, lse, ws,
                                   plan.workspace_bytes, run_mask=run_mask)
            da.decode_attn_combine(plan, ws, out, lse)
            assert da.decode_attn_last_device_status(plan) == da.DA_OK
            results.append((out, lse, wd.k_pool.clone(), wd.v_pool.clone()))
    for i in (0, 1):                                       # without / with the mask
        a, b = results[i], results[2 + i]
        assert torch.equal(a[2], b[2]) and torch.equal(a[3], b[3]), "pools differ"
        assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]), "outputs differ"
    # against the oracle over the appended cache
    inp = oracle.PagedInputs.from_workload(w)
    k_ref, v_ref = oracle.append_kv(inp, new_k.cpu(), new_v.cpu())
    assert np.array_equal(results[2][2].cpu().numpy().view(np.uint16).ravel(), k_ref.ravel())
    w.k_pool = torch.from_numpy(k_ref.view(np.int16).reshape(tuple(w.k_pool.shape)))
    w.v_pool = torch.from_numpy(v_ref.view(np.int16).reshape(tuple(w.v_pool.shape)))
    ref_out, ref_lse = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w), run_mask=mask.cpu().numpy())
    assert_parity(results[3][0], results[3][1], ref_out, ref_lse)


def test_fused_write_is_refused_where_it_is_not_built():
    w = to_device(wl.config_tiny())
    nk = torch.zeros((4, 2, 64), dtype=torch.int16, device="cuda")
    out = torch.zeros((4, 8, 64), dtype=torch.float32, device="cuda")
    plan = da.decode_attn_plan(da.shape_of_workload(w), da.make_policy(kernel=da.DA_KERNEL_SIMT), w.seq_lens)
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device="cuda")
    args = (plan, w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, out, None, ws, plan.workspace_bytes)
    assert da.decode_attn_run(*args, new_k=nk, new_v=nk, check=False) == da.DA_ERR_UNSUPPORTED
    plan = da.decode_attn_plan(da.shape_of_workload(w), da.make_policy(), w.seq_lens)
    args = (plan,) + args[1:]
    assert da.decode_attn_run(*args, new_k=nk, new_v=None, check=False) == da.DA_ERR_INVALID_ARG


def test_run_args_without_the_new_fields_are_still_accepted():
    """A caller built against decode_attn_run_args_t as it was before new_k / new_v passes the
    shorter struct_size; whatever follows in memory must not be read."""
    import ctypes
    w = to_device(wl.config_tiny())
    plan = da.decode_attn_plan(da.shape_of_workload(w), da.make_policy(), w.seq_lens)
    out = torch.zeros((4, 8, 64), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device="cuda")
    a = da.RunArgs()
    a.struct_size = da.RunArgs.new_k.offset
    a.q, a.k_cache, a.v_cache = w.q_bits.data_ptr(), w.k_pool.data_ptr(), w.v_pool.data_ptr()
    a.block_table, a.seq_lens, a.out = w.block_table.data_ptr(), w.seq_lens.data_ptr(), out.data_ptr()
    a.workspace, a.workspace_bytes = ws.data_ptr(), plan.workspace_bytes
    a.new_k = a.new_v = 0xdead0                          # garbage behind the declared size
    before = w.k_pool.clone()
    assert da._lib.decode_attn_run_ex(plan.handle, ctypes.byref(a), torch.cuda.current_stream().cuda_stream) == da.DA_OK
    da.decode_attn_combine(plan, ws, out)
    assert da.decode_attn_last_device_status(plan) == da.DA_OK
    assert torch.equal(before, w.k_pool) and out.abs().sum() > 0
    a.struct_size = 80
    assert da._lib.decode_attn_run_ex(plan.handle, ctypes.byref(a), torch.cuda.current_stream().cuda_stream) == da.DA_ERR_INVALID_ARG
