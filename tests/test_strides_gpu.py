"""Pools with padding: K and V are addressed only through the strides of the
shape, which may differ between the two pools and leave gaps (filled with NaN
patterns here) after every row, head block and page; a combined K/V buffer
(V interleaved behind K in each token row) is one such case."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_37062_b200 import workloads as wl
from gpu_util import KERNELS, KERNEL_IDS, assert_parity, da

pytestmark = pytest.mark.gpu

NAN_BITS = 0x7FC0                  # a quiet NaN as bf16 and as fp16


def padded(pool, pad_h, pad_d):
    """[N, P, H, D] copied into a NaN-filled [N, P, H + pad_h, D + pad_d]; returns (buffer, strides)."""
    N, P, H, D = pool.shape
    buf = torch.full((N, P, H + pad_h, D + pad_d), NAN_BITS, dtype=torch.int16)
    buf[:, :, :H, :D] = pool
    Hs, Ds = H + pad_h, D + pad_d
    return buf, (P * Hs * Ds, Hs * Ds, Ds)


def run(w, shape, policy, k_buf, v_buf):
    dev = "cuda"
    plan = da.decode_attn_plan(shape, policy, w.seq_lens)
    out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device=dev)
    lse = torch.full((w.batch, w.num_q_heads), float("nan"), dtype=torch.float32, device=dev)
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device=dev)
    da.decode_attn_run(plan, w.q_bits.to(dev), k_buf, v_buf, w.block_table.to(dev), w.seq_lens.to(dev), out, lse, ws,
                       plan.workspace_bytes)
    if not policy.fuse_combine:
        da.decode_attn_combine(plan, ws, out, lse)
    torch.cuda.synchronize()
    assert da.decode_attn_last_device_status(plan) == da.DA_OK
    plan.destroy()
    return out, lse


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("d,ps", [(128, 16), (64, 16), (128, 64)])
def test_padded_pools_with_different_strides(kernel, d, ps):
    w = wl.make_workload("pad", [300, 17, 1025, 0, 64], 16, 4, d, seed=51, page_size=ps)
    k_buf, ks = padded(w.k_pool, 1, 8)
    v_buf, vs = padded(w.v_pool, 2, 24)
    shape = da.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, d, ps, w.max_pages_per_seq, w.num_pages, ks, vs)
    inp = oracle.PagedInputs(w.q_bits, k_buf, v_buf, w.block_table, w.seq_lens, ps, ks, w.num_kv_heads, v_strides=vs)
    ref_out, ref_lse = oracle.paged_decode_attention(inp)
    plain_out, plain_lse = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    assert np.array_equal(ref_out, plain_out)           # the oracle itself reads the same values through the strides
    for pol in (da.make_policy(kernel=kernel), da.make_policy(kernel=kernel, fuse_combine=1, chunk_tokens=64)):
        out, lse = run(w, shape, pol, k_buf.cuda(), v_buf.cuda())
        assert_parity(out, lse, ref_out, ref_lse, f"padded D={d} page={ps}")


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_interleaved_kv_buffer(kernel):
    """One buffer [N, P, 2, H, D]: K rows and V rows of a token side by side."""
    w = wl.make_workload("kv", [700, 33, 130], 32, 8, 128, seed=52)
    N, P, H, D = w.k_pool.shape
    both = torch.stack([w.k_pool, w.v_pool], dim=2).contiguous().cuda()     # [N, P, 2, H, D]
    strides = (P * 2 * H * D, 2 * H * D, D)
    shape = da.make_shape(w.batch, w.num_q_heads, H, D, P, w.max_pages_per_seq, N, strides, strides)
    k_view = both.view(-1)
    v_view = both.view(-1)[H * D:]                                            # V starts one K row block later
    ref_out, ref_lse = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    out, lse = run(w, shape, da.make_policy(kernel=kernel), k_view, v_view)
    assert_parity(out, lse, ref_out, ref_lse, "interleaved")
