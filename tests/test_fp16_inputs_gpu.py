"""q, K and V in fp16 instead of bf16 (the paper serves one model family in
each, Section 4.1): same path, same oracle, same tolerance, on both kernels,
in every split mode, fused and separate merge, with a run mask, in both pool
layouts, with the own-layer KV write, and in shared-prefix plans on both
prefix kernels."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_37062_b200 import workloads as wl
from gpu_util import KERNELS, KERNEL_IDS, assert_parity, check_workload, da, oracle_of, to_device

pytestmark = pytest.mark.gpu

POLICIES = [("auto", dict()), ("auto_fused", dict(fuse_combine=1)),
            ("fixed5", dict(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=5)),
            ("det64", dict(split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=64)),
            ("det_default_fused", dict(split_mode=da.DA_SPLIT_DETERMINISTIC, fuse_combine=1))]


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("name,pol", POLICIES, ids=[p[0] for p in POLICIES])
def test_fp16_parity(kernel, name, pol):
    check_workload(wl.make_workload("tiny16", [17, 64, 129, 300], 8, 2, 64, seed=0, dtype="fp16"),
                   da.make_policy(kernel=kernel, **pol), what=name)
    check_workload(wl.make_workload("long16", [4133], 32, 8, 128, seed=1, dtype="fp16"),
                   da.make_policy(kernel=kernel, **pol), what=name)


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("hq,hkv,d", [(8, 8, 128), (16, 8, 64), (24, 8, 128), (40, 8, 64), (16, 2, 128)])
def test_fp16_group_sizes_head_dims_and_layouts(kernel, hq, hkv, d):
    lens = [1, 16, 33, 700, 2049, 0, 255]
    for layout in ("token_major", "head_major"):
        w = wl.make_workload("g16", lens, hq, hkv, d, seed=7, layout=layout, dtype="fp16")
        check_workload(w, da.make_policy(kernel=kernel if hq // hkv > 1 else da.DA_KERNEL_SIMT), what=f"G={hq // hkv} D={d}")


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_fp16_run_mask_and_full_size(kernel):
    w = wl.make_workload("m16", wl.lengths_short_chat(24, 2), 32, 8, 128, seed=2, dtype="fp16")
    mask = [i % 3 != 0 for i in range(24)]
    ref_out, ref_lse = oracle_of(w, run_mask=mask)
    out, lse = da.run_workload(to_device(w), da.make_policy(kernel=kernel),
                               run_mask=torch.tensor(mask, dtype=torch.uint8, device="cuda"))
    assert_parity(out, lse, ref_out, ref_lse)
    assert not out[0].any() and torch.isneginf(lse[0]).all()


def test_fp16_sharp_rows_keep_their_precision():
    """One dominant token per row: the weights' two-part split must hold in fp16 too."""
    w = wl.make_workload("s16", [1500, 900], 32, 8, 128, seed=3, dtype="fp16")
    ref_out, ref_lse = oracle_of(w, scale=1.0)
    out, lse = da.run_workload(to_device(w), da.make_policy(), sm_scale=1.0)
    diff = np.abs(out.double().cpu().numpy() - ref_out)
    assert diff.max() < 2e-4, diff.max()          # far inside the stated bar: a single-part fp16 P would sit near 1e-3


def test_fp16_append_then_attend():
    w = wl.make_workload("a16", [40, 17, 64, 1], 8, 2, 64, seed=4, dtype="fp16")
    inp = oracle.PagedInputs.from_workload(w)
    new_k = torch.randn(4, 2, 64).to(torch.float16).view(torch.int16)
    new_v = torch.randn(4, 2, 64).to(torch.float16).view(torch.int16)
    k_ref, v_ref = oracle.append_kv(inp, new_k, new_v)
    wd = to_device(w)
    da.decode_attn_append_kv(da.shape_of_workload(wd), new_k.cuda(), new_v.cuda(), wd.block_table, wd.seq_lens,
                             wd.k_pool, wd.v_pool)
    torch.cuda.synchronize()
    assert np.array_equal(wd.k_pool.cpu().numpy().view(np.uint16), k_ref.reshape(wd.k_pool.shape))
    assert np.array_equal(wd.v_pool.cpu().numpy().view(np.uint16), v_ref.reshape(wd.v_pool.shape))


@pytest.mark.parametrize("kernel", [da.DA_KERNEL_MMA_TMA, da.DA_KERNEL_UMMA_PREFIX], ids=["mma_sync", "tcgen05"])
def test_fp16_shared_prefix_plans(kernel):
    for batch, prefix in ((12, 512), (33, 1536), (5, 208)):
        w = wl.as_fp16(wl.config_shared_prefix(batch=batch, prefix=prefix))
        check_workload(w, da.make_policy(shared_prefix_tokens=prefix, kernel=kernel))
        check_workload(w, da.make_policy(shared_prefix_tokens=prefix, kernel=kernel, split_mode=da.DA_SPLIT_DETERMINISTIC,
                                         chunk_tokens=128))


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("fused", [0, 1])
def test_fp16_output_is_the_rounded_result(kernel, fused):
    """An fp16 `out` sits within one fp16 step of the oracle (its own rounding), whether it is
    written by the attention kernel (single split), the combine kernel or the merge blocks."""
    w = wl.make_workload("o16", [17, 64, 129, 900], 8, 2, 64, seed=6, dtype="fp16")
    ref_out, _ = oracle_of(w)
    out, _ = da.run_workload(to_device(w), da.make_policy(kernel=kernel, fuse_combine=fused, chunk_tokens=64),
                             out_dtype=da.DA_DTYPE_FP16)
    assert out.dtype == torch.float16
    got = out.float().cpu().numpy().astype(np.float64)
    step = np.maximum(np.abs(ref_out), 2.0 ** -14) * 2.0 ** -10
    assert (np.abs(got - ref_out) <= step + 1e-6).all()


def test_mixed_input_types_are_refused():
    w = wl.make_workload("p16", [600, 700], 32, 8, 128, seed=5, dtype="fp16")
    s = da.shape_of_workload(w)
    s.q_dtype = da.DA_DTYPE_BF16
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_plan(s, da.make_policy(), w.seq_lens)
    assert e.value.status == da.DA_ERR_UNSUPPORTED
