"""Helpers shared by the GPU tests: move a workload to the device, run the
library through its C ABI, and compare with the CPU oracle."""
import dataclasses

import numpy as np
import torch

import oracle
from paper_2609_37062_b200 import build as da_build

da_build.build()
from paper_2609_37062_b200 import binding as da  # noqa: E402

MAX_ABS = 2e-3    # bf16 KV, fp32 accumulate: the stated bar
MEAN_ABS = 2e-4
LSE_ABS = 1e-3    # plus LSE_REL * |lse|: an fp32 logit of magnitude x carries ~sqrt(D) ulps(x) of rounding
LSE_REL = 4e-6

KERNELS = [da.DA_KERNEL_SIMT, da.DA_KERNEL_MMA_TMA]
KERNEL_IDS = ["simt", "mma"]


def to_device(w, device="cuda"):
    return dataclasses.replace(
        w, seq_lens=w.seq_lens.to(device), block_table=w.block_table.to(device), q_bits=w.q_bits.to(device),
        k_pool=w.k_pool.to(device), v_pool=w.v_pool.to(device))


def to_host(w):
    return to_device(w, "cpu")


def oracle_of(w_host, scale=None, run_mask=None):
    return oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w_host), scale=scale, run_mask=run_mask)


def errors(out, ref):
    diff = np.abs(out.detach().float().cpu().numpy().astype(np.float64) - ref)
    return float(diff.max()) if diff.size else 0.0, float(diff.mean()) if diff.size else 0.0


def assert_parity(out, lse, ref_out, ref_lse, what=""):
    mx, mean = errors(out, ref_out)
    assert np.isfinite(out.detach().float().cpu().numpy()).all(), what
    assert mx <= MAX_ABS and mean <= MEAN_ABS, f"{what}: max-abs {mx:.3e} mean-abs {mean:.3e}"
    if lse is not None:
        got = lse.detach().cpu().numpy().astype(np.float64)
        fin = np.isfinite(ref_lse)
        assert np.array_equal(np.isneginf(got), np.isneginf(ref_lse)), what
        if fin.any():
            assert (np.abs(got[fin] - ref_lse[fin]) <= LSE_ABS + LSE_REL * np.abs(ref_lse[fin])).all(), what
    return mx, mean


def check_workload(w_host, policy=None, what="", **kw):
    ref_out, ref_lse = oracle_of(w_host, scale=kw.get("scale_ref"))
    w = to_device(w_host)
    out, lse = da.run_workload(w, policy, sm_scale=kw.get("sm_scale", 0.0))
    torch.cuda.synchronize()
    return assert_parity(out, lse, ref_out, ref_lse, what)
