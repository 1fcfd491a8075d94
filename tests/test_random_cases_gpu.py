"""Seeded random cases through the C ABI against the oracle: shapes, length
mixes with the awkward values (0, 1, page boundaries +-1), both kernels, all
split modes, fused and separate merge, run masks, both pool layouts, both
input types, page sizes, groups of up to 16 heads, and
shared-prefix plans on both prefix kernels.  What a case does not support is
refused with DA_ERR_UNSUPPORTED, never computed wrongly."""
import random

import numpy as np
import pytest
import torch

from paper_2609_37062_b200 import workloads as wl
from gpu_util import LSE_ABS, LSE_REL, MAX_ABS, MEAN_ABS, da, oracle_of, to_device

pytestmark = pytest.mark.gpu

LENGTHS = [0, 1, 15, 16, 17, 31, 33, 64, 100, 255, 256, 257, 500, 1000, 1500, 2049, 3000]


def one_case(rng, index, any_page_size=False, wide_groups=False):
    ps = rng.choice([16, 32, 64, 128, 256]) if any_page_size else 16
    D = rng.choice([64, 128])
    hkv = rng.choice([1, 2, 4, 8])
    G = rng.choice([9, 10, 11, 12, 13, 14, 15, 16, 4, 7]) if wide_groups else rng.choice([1, 2, 3, 4, 5, 8])
    B = rng.choice([1, 2, 3, 5, 9, 17])
    lens = [rng.choice(LENGTHS) for _ in range(B)]
    mode = rng.choice([da.DA_SPLIT_AUTO, da.DA_SPLIT_DETERMINISTIC, da.DA_SPLIT_FIXED_COUNT])
    pol = dict(kernel=rng.choice([da.DA_KERNEL_AUTO, da.DA_KERNEL_SIMT, da.DA_KERNEL_MMA_TMA]), split_mode=mode,
               fuse_combine=rng.choice([0, 1]))
    if mode == da.DA_SPLIT_FIXED_COUNT:
        pol["fixed_count"] = rng.choice([1, 2, 3, 4, 5, 7, 8, 9, 16, 33])
    if mode == da.DA_SPLIT_DETERMINISTIC:
        pol["chunk_tokens"] = rng.choice([16, 32, 64, 256, 1024])
    prefix = 0
    if rng.random() < 0.25:                       # (groups of 5+ heads: the tcgen05 prefix kernel only)
        prefix = (rng.choice([16, 128, 160, 512, 1040]) + ps - 1) // ps * ps
        lens = [prefix + n for n in lens]
        pol = dict(shared_prefix_tokens=prefix, split_mode=rng.choice([da.DA_SPLIT_AUTO, da.DA_SPLIT_DETERMINISTIC]),
                   kernel=rng.choice([da.DA_KERNEL_MMA_TMA, da.DA_KERNEL_UMMA_PREFIX]) if D == 128 else da.DA_KERNEL_MMA_TMA)
        if pol["split_mode"] == da.DA_SPLIT_DETERMINISTIC:
            pol["chunk_tokens"] = rng.choice([16, 64, 128, 1024])
    mask = [rng.choice([0, 1]) for _ in range(B)] if rng.random() < 0.3 else None
    layout = rng.choice(["token_major", "head_major"]) if not prefix else "token_major"
    dtype = rng.choice(["bf16", "fp16"])
    w = wl.make_workload("r", lens, hkv * G, hkv, D, seed=index, layout=layout, shared_prefix_tokens=prefix, dtype=dtype,
                         page_size=ps)
    return w, pol, mask


@pytest.mark.parametrize("seed", [11, 12, 13, 14, 15, 16, 17])
def test_random_cases(seed):
    rng = random.Random(seed)
    refused = 0
    for index in range(60):
        w, pol, mask = one_case(rng, index, any_page_size=seed >= 14, wide_groups=seed >= 16)
        ref, ref_lse = oracle_of(w, run_mask=mask)
        m = None if mask is None else torch.tensor(mask, dtype=torch.uint8, device="cuda")
        try:
            out, lse = da.run_workload(to_device(w), da.make_policy(**pol), run_mask=m)
        except da.DecodeAttnError as e:
            assert e.status == da.DA_ERR_UNSUPPORTED, (index, pol)
            refused += 1
            continue
        what = f"seed {seed} case {index}: {pol} {w.dtype} page {w.page_size} lens {w.seq_lens.tolist()} mask {mask}"
        diff = np.abs(out.double().cpu().numpy() - ref)
        assert diff.max() <= MAX_ABS and diff.mean() <= MEAN_ABS, what
        got = lse.double().cpu().numpy()
        fin = np.isfinite(ref_lse)
        assert np.array_equal(np.isneginf(got), np.isneginf(ref_lse)), what
        if fin.any():
            assert (np.abs(got[fin] - ref_lse[fin]) <= LSE_ABS + LSE_REL * np.abs(ref_lse[fin])).all(), what
    assert refused < (45 if seed >= 16 else 30)      # (wide groups: neither the CUDA-core kernel nor prefix plans)
