"""Out-of-bounds writes: the workspace, the output and the LSE buffer sit
inside larger allocations whose margins hold a byte pattern; after run and
combine the margins must be untouched, for every kernel, fused or not, with
ragged lengths, empty and masked rows and every output type."""
import numpy as np
import pytest
import torch

from paper_2609_37062_b200 import workloads as wl
from gpu_util import assert_parity, da, oracle_of, to_device

pytestmark = pytest.mark.gpu

GUARD = 4096      # bytes on each side; a multiple of every alignment the library asks for
PATTERN = 0xA5


class Guarded:
    """`nbytes` usable bytes between two margins filled with PATTERN."""

    def __init__(self, nbytes, device="cuda"):
        self.nbytes = nbytes
        self.raw = torch.full((GUARD + nbytes + GUARD,), PATTERN, dtype=torch.uint8, device=device)

    def view(self, dtype, shape):
        return self.raw[GUARD:GUARD + self.nbytes].view(dtype).view(shape)

    def intact(self):
        return bool((self.raw[:GUARD] == PATTERN).all()) and bool((self.raw[GUARD + self.nbytes:] == PATTERN).all())


CASES = [
    ("simt_auto", dict(kernel=da.DA_KERNEL_SIMT)),
    ("simt_fused", dict(kernel=da.DA_KERNEL_SIMT, fuse_combine=1, chunk_tokens=64)),
    ("mma_auto", dict(kernel=da.DA_KERNEL_MMA_TMA)),
    ("mma_fused", dict(kernel=da.DA_KERNEL_MMA_TMA, fuse_combine=1, chunk_tokens=64)),
    ("mma_fixed7", dict(kernel=da.DA_KERNEL_MMA_TMA, split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=7)),
    ("mma_det", dict(kernel=da.DA_KERNEL_MMA_TMA, split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=48)),
]
OUT_TYPES = [(da.DA_DTYPE_FP32, torch.float32, 4), (da.DA_DTYPE_BF16, torch.bfloat16, 2),
             (da.DA_DTYPE_FP16, torch.float16, 2)]


def run_guarded(w_host, policy, out_dtype=da.DA_DTYPE_FP32, tdt=torch.float32, esize=4, run_mask=None):
    w = to_device(w_host)
    plan = da.decode_attn_plan(da.shape_of_workload(w, out_dtype=out_dtype), policy, w.seq_lens)
    try:
        n_out = w.batch * w.num_q_heads * w.head_dim
        g_out = Guarded(n_out * esize)
        g_lse = Guarded(w.batch * w.num_q_heads * 4)
        g_ws = Guarded(max(plan.workspace_bytes, 256))
        out = g_out.view(tdt, (w.batch, w.num_q_heads, w.head_dim))
        lse = g_lse.view(torch.float32, (w.batch, w.num_q_heads))
        ws = g_ws.raw[GUARD:GUARD + g_ws.nbytes]
        mask = None if run_mask is None else torch.as_tensor(run_mask, dtype=torch.uint8, device="cuda")
        da.decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, out, lse, ws,
                           plan.workspace_bytes, run_mask=mask)
        if not policy.fuse_combine:
            da.decode_attn_combine(plan, ws, out, lse)
        torch.cuda.synchronize()
        assert da.decode_attn_last_device_status(plan) == da.DA_OK
    finally:
        plan.destroy()
    assert g_out.intact(), "write outside out"
    assert g_lse.intact(), "write outside lse"
    assert g_ws.intact(), "write outside the workspace"
    return out, lse


@pytest.mark.parametrize("name,pol", CASES, ids=[c[0] for c in CASES])
def test_margins_untouched_ragged_batch(name, pol):
    w = wl.make_workload("guard", [0, 1, 17, 333, 1025, 64, 0, 2049], 32, 8, 128, seed=77)
    out, lse = run_guarded(w, da.make_policy(**pol))
    ref_out, ref_lse = oracle_of(w)
    assert_parity(out, lse, ref_out, ref_lse, name)


@pytest.mark.parametrize("odt,tdt,esize", OUT_TYPES, ids=["fp32", "bf16", "fp16"])
@pytest.mark.parametrize("fused", [0, 1])
def test_margins_untouched_every_output_type(odt, tdt, esize, fused):
    w = wl.make_workload("guard_t", [700, 5, 130], 16, 8, 64, seed=78)
    out, lse = run_guarded(w, da.make_policy(fuse_combine=fused, chunk_tokens=128), odt, tdt, esize)
    ref_out, _ = oracle_of(w)
    tol = 2e-3 if esize == 4 else 2e-2   # a 16-bit output rounds values of magnitude ~1 to 2^-8 / 2^-11
    assert np.abs(out.float().cpu().numpy() - ref_out).max() <= tol


def test_margins_untouched_masked_rows():
    w = wl.make_workload("guard_m", [300, 300, 40, 1000, 9], 32, 8, 128, seed=79)
    mask = [1, 0, 1, 0, 1]
    for fused in (0, 1):
        out, lse = run_guarded(w, da.make_policy(fuse_combine=fused), run_mask=mask)
        ref_out, ref_lse = oracle_of(w, run_mask=mask)
        assert_parity(out, lse, ref_out, ref_lse, "masked")


@pytest.mark.parametrize("kernel", [da.DA_KERNEL_MMA_TMA, da.DA_KERNEL_UMMA_PREFIX], ids=["mma", "umma"])
def test_margins_untouched_shared_prefix(kernel):
    w = wl.config_shared_prefix(batch=20, prefix=640)
    pol = da.make_policy(kernel=kernel, shared_prefix_tokens=w.shared_prefix_tokens)
    out, lse = run_guarded(w, pol)
    ref_out, ref_lse = oracle_of(w)
    assert_parity(out, lse, ref_out, ref_lse, "prefix")
