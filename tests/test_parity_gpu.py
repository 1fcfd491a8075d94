"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU
oracle on the same seeded bytes.  Tolerance: max-abs 2e-3 and mean-abs 2e-4
over all output elements of a case (bf16 K/V, fp32 accumulation, fp32 out)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_37062_b200 import workloads as wl
from gpu_util import (KERNELS, KERNEL_IDS, assert_parity, check_workload, da, errors, oracle_of, to_device)

pytestmark = pytest.mark.gpu

SPLITS = [("auto", dict()),
          ("auto_fused", dict(fuse_combine=1)),
          ("fixed1", dict(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=1)),
          ("fixed2", dict(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=2)),
          ("fixed3_fused", dict(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=3, fuse_combine=1)),
          ("fixed8", dict(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=8)),
          ("fixed64_fused", dict(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=64, fuse_combine=1)),
          ("det16", dict(split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=16)),
          ("det64_fused", dict(split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=64, fuse_combine=1)),
          ("det_default", dict(split_mode=da.DA_SPLIT_DETERMINISTIC))]


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("name,pol", SPLITS, ids=[s[0] for s in SPLITS])
def test_tiny_config(kernel, name, pol):
    check_workload(wl.config_tiny(), da.make_policy(kernel=kernel, **pol), what=name)


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_tiny_config_head_major_layout(kernel):
    check_workload(wl.config_tiny(layout="head_major"), da.make_policy(kernel=kernel))
    check_workload(wl.config_tiny(layout="head_major"),
                   da.make_policy(kernel=kernel, split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=3))


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("name,pol", [SPLITS[0], SPLITS[1], SPLITS[5], SPLITS[6], SPLITS[9]],
                         ids=["auto", "auto_fused", "fixed8", "fixed64_fused", "det_default"])
def test_long_sequence_reduced(kernel, name, pol):
    """Shape of the single-long-sequence configuration at 4,133 tokens: many
    tiles per unit and a ragged last page."""
    check_workload(wl.config_long(context=4133), da.make_policy(kernel=kernel, **pol), what=name)


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("fused", [0, 1])
def test_short_chat_mix_reduced(kernel, fused):
    check_workload(wl.config_short_chat(batch=24), da.make_policy(kernel=kernel, fuse_combine=fused))
    check_workload(wl.config_short_chat(batch=24),
                   da.make_policy(kernel=kernel, fuse_combine=fused, chunk_tokens=64, sm_count=16))


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_shared_prefix_reduced(kernel):
    w = wl.config_shared_prefix(batch=12, prefix=512)
    check_workload(w, da.make_policy(kernel=kernel, fuse_combine=1))
    check_workload(w, da.make_policy(kernel=kernel, split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=256))


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("hq,hkv,d", [(8, 8, 128), (16, 8, 64), (24, 8, 128), (32, 8, 64), (40, 8, 128),
                                      (12, 2, 64), (14, 2, 128), (16, 2, 128)])
def test_group_sizes_and_head_dims(kernel, hq, hkv, d):
    w = wl.make_workload("g", [200, 31, 1000], hq, hkv, d, seed=21)
    pol = da.make_policy(kernel=kernel if hq // hkv > 1 else da.DA_KERNEL_SIMT, fuse_combine=1, chunk_tokens=128)
    check_workload(w, pol, what=f"G={hq // hkv} D={d}")


EDGE_LENS = [0, 1, 15, 16, 17, 31, 32, 33, 63, 64, 65, 255, 256, 257, 1023, 1024, 1025]


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("name,pol", [SPLITS[0], SPLITS[4], SPLITS[7], SPLITS[9]],
                         ids=["auto", "fixed3_fused", "det16", "det_default"])
def test_edge_lengths_with_poisoned_padding(kernel, name, pol):
    """Lengths around page, tile and chunk boundaries; unused slots of the
    last page and unreferenced pages hold NaN bit patterns and must never
    reach the result.  A zero-length row gives zeros and lse = -inf."""
    w = wl.make_workload("edges", EDGE_LENS, 8, 2, 128, seed=5, pool_pages=400)
    ref_out, ref_lse = oracle_of(w)
    out, lse = da.run_workload(to_device(w), da.make_policy(kernel=kernel, **pol))
    assert_parity(out, lse, ref_out, ref_lse, name)
    assert not out[0].any() and torch.isneginf(lse[0]).all()


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_sharp_softmax_and_late_maximum(kernel):
    """q scaled by 16 (nearly one-hot softmax, the running max is rescued many
    times) and a sequence whose largest logit sits in the very last token."""
    w = wl.make_workload("sharp", [777, 2049], 8, 2, 128, seed=9)
    q = (w.q_bits.view(torch.bfloat16).float() * 16.0).to(torch.bfloat16)
    w.q_bits = q.view(torch.int16)
    b, L = 1, 2049
    page, slot = int(w.block_table[b, (L - 1) // 16]), (L - 1) % 16
    w.k_pool[page, slot] = (q[b, ::4] * 2).view(torch.int16)        # key aligned with each group's first query
    for name, pol in (SPLITS[0], SPLITS[6], SPLITS[7]):
        check_workload(w, da.make_policy(kernel=kernel, **pol), what=name)


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_explicit_scale(kernel):
    w = wl.config_tiny()
    ref_out, ref_lse = oracle_of(w, scale=float(np.float32(0.3)))
    out, lse = da.run_workload(to_device(w), da.make_policy(kernel=kernel), sm_scale=0.3)
    assert_parity(out, lse, ref_out, ref_lse)


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_bf16_output_is_the_rounded_result(kernel):
    """A bf16 `out` cannot meet the fp32 tolerance (its own rounding is
    larger); it must instead sit within one bf16 step of the rounded oracle."""
    w = wl.config_tiny()
    ref_out, _ = oracle_of(w)
    out, _ = da.run_workload(to_device(w), da.make_policy(kernel=kernel, fuse_combine=1), out_dtype=da.DA_DTYPE_BF16)
    assert out.dtype == torch.bfloat16
    got = out.float().cpu().numpy().astype(np.float64)
    ulp = np.maximum(np.abs(ref_out), 2.0 ** -126) * 2.0 ** -7
    assert (np.abs(got - ref_out) <= ulp + 1e-6).all()


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("fused", [0, 1])
def test_run_mask_rows_read_nothing_and_emit_zero(kernel, fused):
    """Algorithm 1 step 2: a Project-Only row reads no KV and emits zero."""
    w = wl.config_short_chat(batch=10)
    mask = [1, 0, 1, 1, 0, 0, 1, 1, 1, 0]
    ref_out, ref_lse = oracle_of(w, run_mask=mask)
    wd = to_device(w)
    # poison the masked rows' pages: if the kernel read them, NaN would surface
    for b, keep in enumerate(mask):
        if not keep:
            n = (int(w.seq_lens[b]) + 15) // 16
            wd.k_pool[wd.block_table[b, :n].long()] = 0x7FC0
            wd.v_pool[wd.block_table[b, :n].long()] = 0x7FC0
    dmask = torch.tensor(mask, dtype=torch.uint8, device="cuda")
    out, lse = da.run_workload(wd, da.make_policy(kernel=kernel, fuse_combine=fused, chunk_tokens=64), run_mask=dmask)
    assert_parity(out, lse, ref_out, ref_lse)
    for b, keep in enumerate(mask):
        if not keep:
            assert not out[b].any() and torch.isneginf(lse[b]).all()


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_one_hot_probes_pin_the_gather(kernel):
    """For each probed logical position t the key at t dominates (logit +1000
    against -1000), so `out` must equal the value row at t bit for bit: the K
    address decides which token wins, the V address decides what comes out.
    Covers every slot of several pages, both KV heads, a split boundary."""
    L, D, Hkv, G = 100, 128, 2, 4
    base = wl.make_workload("probe", [L], Hkv * G, Hkv, D, seed=13, pool_pages=16)
    q = torch.zeros((1, Hkv * G, D), dtype=torch.float32)
    q[:, :, 0] = 1.0 / float(np.float32(1.0) / np.sqrt(np.float32(D)))        # logit = k[0] up to rounding
    base.q_bits = q.to(torch.bfloat16).view(torch.int16)
    scale_q = float(q.to(torch.bfloat16)[0, 0, 0]) * float(np.float32(1.0) / np.sqrt(np.float32(D)))
    vals = base.v_pool.view(torch.bfloat16).float()
    for pol in (da.make_policy(kernel=kernel), da.make_policy(kernel=kernel, split_mode=da.DA_SPLIT_DETERMINISTIC,
                                                                chunk_tokens=48, fuse_combine=1)):
        for t in list(range(0, 34)) + [47, 48, 63, 64, 95, 96, 99]:
            w = to_device(base)
            kf = w.k_pool.view(torch.bfloat16)
            for tt in range(L):
                page, slot = int(base.block_table[0, tt // 16]), tt % 16
                kf[page, slot, :, 0] = 1000.0 if tt == t else -1000.0
            out, lse = da.run_workload(w, pol)
            page, slot = int(base.block_table[0, t // 16]), t % 16
            for h in range(Hkv * G):
                assert torch.equal(out[0, h].cpu(), vals[page, slot, h // G]), (t, h)
            assert abs(float(lse[0, 0]) - 1000.0 * scale_q) < 0.5


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_page_permutation_changes_nothing_within_tolerance(kernel):
    w = wl.config_tiny()
    ref_out, ref_lse = oracle_of(w)
    out, lse = da.run_workload(to_device(wl.permute_pages(w, seed=4)), da.make_policy(kernel=kernel))
    assert_parity(out, lse, ref_out, ref_lse)


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_block_table_rows_may_be_wider_than_needed(kernel):
    w = wl.make_workload("wide", [40, 333], 8, 2, 64, seed=3, max_pages_per_seq=77)
    check_workload(w, da.make_policy(kernel=kernel, fuse_combine=1, chunk_tokens=64))


@pytest.mark.parametrize("fused", [0, 1])
@pytest.mark.parametrize("frac", [0.1, 0.5, 0.9])
def test_run_mask_on_a_work_list_of_several_rounds(fused, frac):
    """More units than resident blocks and many masked rows: the masked variant of the tensor-core
    kernel deals the work list out again among its blocks (from three masked rows in ten); the
    result must not depend on which block attends which unit."""
    rng = np.random.default_rng(7)
    lens = [int(x) for x in rng.integers(1, 700, size=300)]
    w = wl.make_workload("m", lens, 32, 8, 128, seed=31)
    mask = (rng.random(len(lens)) >= frac).astype(np.uint8)
    ref_out, ref_lse = oracle_of(w, run_mask=mask)
    wd = to_device(w)
    dmask = torch.from_numpy(mask).cuda()
    pol = da.make_policy(kernel=da.DA_KERNEL_MMA_TMA, fuse_combine=fused, chunk_tokens=64)
    out, lse = da.run_workload(wd, pol, run_mask=dmask)
    assert_parity(out, lse, ref_out, ref_lse)
    # the same bits as row by row: a row's result does not depend on the mask of the others
    det = da.make_policy(kernel=da.DA_KERNEL_MMA_TMA, split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=128)
    out_m, _ = da.run_workload(wd, det, run_mask=dmask)
    out_all, _ = da.run_workload(wd, det)
    keep = torch.from_numpy(mask.astype(bool)).cuda()
    assert torch.equal(out_m[keep], out_all[keep])
    assert not out_m[~keep].any()

