"""Pages of 32, 64, 128 and 256 tokens: the kernels fetch 16-token tiles and
find each tile's page and slot offset from the block table, so every path
must give the oracle's result - and, since neither the plan nor the
arithmetic depends on the page size, the very bits it gives with 16-token
pages over the same logical cache."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_37062_b200 import workloads as wl
from gpu_util import KERNELS, KERNEL_IDS, assert_parity, da, oracle_of, to_device

pytestmark = pytest.mark.gpu

PAGE_SIZES = [32, 64, 128, 256]
LENS = [0, 1, 16, 17, 31, 33, 255, 257, 1000, 2049, 64, 4133]
POLICIES = [("auto", dict()),
            ("auto_fused", dict(fuse_combine=1, chunk_tokens=64)),
            ("fixed3", dict(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=3)),
            ("det48", dict(split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=48))]


def run(w_host, policy, **kw):
    out, lse = da.run_workload(to_device(w_host), policy, **kw)
    torch.cuda.synchronize()
    return out, lse


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("ps", PAGE_SIZES)
@pytest.mark.parametrize("name,pol", POLICIES, ids=[p[0] for p in POLICIES])
def test_parity_and_same_bits_as_16_token_pages(kernel, ps, name, pol):
    policy = da.make_policy(kernel=kernel, **pol)
    w16 = wl.make_workload("ps", LENS, 32, 8, 128, seed=41)
    wp = wl.make_workload("ps", LENS, 32, 8, 128, seed=41, page_size=ps)
    ref_out, ref_lse = oracle_of(wp)
    out, lse = run(wp, policy)
    assert_parity(out, lse, ref_out, ref_lse, f"{name} page_size={ps}")
    out16, lse16 = run(w16, policy)
    assert torch.equal(out, out16) and torch.equal(lse, lse16)


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("ps", [32, 128])
@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 64), (8, 8, 128), (40, 8, 128)])
def test_layouts_groups_and_head_dims(kernel, ps, hq, hkv, d):
    for layout in ("token_major", "head_major"):
        w = wl.make_workload("ps_l", [300, 5, 129, 1025], hq, hkv, d, seed=43, page_size=ps, layout=layout)
        k = kernel if hq // hkv > 1 else da.DA_KERNEL_SIMT
        ref_out, ref_lse = oracle_of(w)
        out, lse = run(w, da.make_policy(kernel=k, chunk_tokens=128))
        assert_parity(out, lse, ref_out, ref_lse, f"{layout} page_size={ps}")


@pytest.mark.parametrize("ps", [32, 64, 256])
def test_fp16_inputs(ps):
    w = wl.make_workload("ps_h", [700, 33, 2000], 32, 8, 128, seed=44, page_size=ps, dtype="fp16")
    ref_out, ref_lse = oracle_of(w)
    for kernel in KERNELS:
        out, lse = run(w, da.make_policy(kernel=kernel))
        assert_parity(out, lse, ref_out, ref_lse, f"fp16 page_size={ps}")


@pytest.mark.parametrize("kernel", [da.DA_KERNEL_MMA_TMA, da.DA_KERNEL_UMMA_PREFIX], ids=["mma", "umma"])
@pytest.mark.parametrize("ps,prefix", [(32, 480), (64, 640), (128, 1536), (256, 512)])
def test_shared_prefix(kernel, ps, prefix):
    lens = [prefix + n for n in (0, 1, 17, 200, 64, 255, 31, 16, 100, 3)]
    w = wl.make_workload("ps_p", lens, 32, 8, 128, seed=45, page_size=ps, shared_prefix_tokens=prefix)
    w16 = wl.make_workload("ps_p", lens, 32, 8, 128, seed=45, shared_prefix_tokens=prefix)
    s = da.shape_of_workload(w)
    assert da.decode_attn_validate_shared_prefix(s, prefix, w.seq_lens, w.block_table) == da.DA_OK
    policy = da.make_policy(kernel=kernel, shared_prefix_tokens=prefix)
    ref_out, ref_lse = oracle_of(w)
    out, lse = run(w, policy)
    assert_parity(out, lse, ref_out, ref_lse, f"prefix page_size={ps}")
    out16, lse16 = run(w16, policy)
    assert torch.equal(out, out16) and torch.equal(lse, lse16)


@pytest.mark.parametrize("ps", [32, 256])
def test_run_mask_and_output_types(ps):
    w = wl.make_workload("ps_m", [300, 300, 40, 1000, 9], 32, 8, 128, seed=46, page_size=ps)
    mask = [1, 0, 1, 0, 1]
    ref_out, ref_lse = oracle_of(w, run_mask=mask)
    dmask = torch.tensor(mask, dtype=torch.uint8, device="cuda")
    out, lse = run(w, da.make_policy(fuse_combine=1), run_mask=dmask)
    assert_parity(out, lse, ref_out, ref_lse, "masked")
    out_b, _ = run(w, da.make_policy(), out_dtype=da.DA_DTYPE_BF16, run_mask=dmask)
    assert np.abs(out_b.float().cpu().numpy() - ref_out).max() <= 2e-2


@pytest.mark.parametrize("ps", [32, 128])
def test_debug_gather_is_bit_exact(ps):
    w = wl.make_workload("ps_g", [17, 300, 1500], 8, 2, 64, seed=47, page_size=ps, layout="head_major")
    inp = oracle.PagedInputs.from_workload(w)
    wd = to_device(w)
    pol = da.make_policy(kernel=da.DA_KERNEL_MMA_TMA, split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=128)
    plan = da.decode_attn_plan(da.shape_of_workload(wd), pol, w.seq_lens)
    for b in range(w.batch):
        L = int(w.seq_lens[b])
        k_out = torch.full((L, w.num_kv_heads, w.head_dim), 0x1234, dtype=torch.int16, device="cuda")
        v_out = torch.full_like(k_out, 0x4321)
        da.decode_attn_debug_gather(plan, b, wd.k_pool, wd.v_pool, wd.block_table, k_out, v_out)
        assert da.decode_attn_last_device_status(plan) == da.DA_OK
        k_ref, v_ref = oracle.gather_kv(inp, b)
        assert np.array_equal(k_out.cpu().numpy().view(np.uint16), k_ref)
        assert np.array_equal(v_out.cpu().numpy().view(np.uint16), v_ref)
    plan.destroy()


@pytest.mark.parametrize("ps", [32, 64])
def test_append_writes_the_right_slot(ps):
    lens = [1, 16, 17, 300, 0, 1024, 1025, 77, ps, ps + 1]
    hq, hkv, d = 32, 8, 128
    w = wl.make_workload("ps_a", lens, hq, hkv, d, seed=48, page_size=ps)
    B = len(lens)
    new_k = wl.normal_bf16_bits(wl.stream_key(48, wl.TENSOR_NEW_K, 0), 0, B * hkv * d).view(B, hkv, d)
    new_v = wl.normal_bf16_bits(wl.stream_key(48, wl.TENSOR_NEW_V, 0), 0, B * hkv * d).view(B, hkv, d)
    k_ref, v_ref = oracle.append_kv(oracle.PagedInputs.from_workload(w), new_k, new_v)
    wd = to_device(w)
    da.decode_attn_append_kv(da.shape_of_workload(wd), new_k.cuda(), new_v.cuda(), wd.block_table, wd.seq_lens,
                             wd.k_pool, wd.v_pool)
    torch.cuda.synchronize()
    assert np.array_equal(wd.k_pool.cpu().numpy().view(np.uint16).ravel(), k_ref.ravel())
    assert np.array_equal(wd.v_pool.cpu().numpy().view(np.uint16).ravel(), v_ref.ravel())


def test_static_step_and_host_step(ps=64):
    w = wl.make_workload("ps_s", [900, 40, 333], 32, 8, 128, seed=49, page_size=ps)
    ref_out, ref_lse = oracle_of(w)
    wd = to_device(w)
    s = da.shape_of_workload(wd)
    out = torch.empty((w.batch, 32, 128), dtype=torch.float32, device="cuda")
    lse = torch.empty((w.batch, 32), dtype=torch.float32, device="cuda")
    da.decode_attn_step_static(s, w.seq_lens, wd.q_bits, wd.k_pool, wd.v_pool, wd.block_table, wd.seq_lens, out, lse)
    torch.cuda.synchronize()
    assert_parity(out, lse, ref_out, ref_lse, "static step")
    hout = torch.empty((w.batch, 32, 128), dtype=torch.float32).pin_memory()
    da.decode_attn_host_step(s, da.make_policy(), w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, hout)
    da.decode_attn_host_release()
    assert_parity(hout, None, ref_out, ref_lse, "host step")
