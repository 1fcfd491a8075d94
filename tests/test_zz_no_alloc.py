"""The allocation-free entry point (for callers that cannot use the CUDA
allocator at call time - an engine whose KV pool already owns all of HBM, or a
path that cannot take an allocation's device-wide sync) against the ordinary
plan / run / combine path it mirrors.  Collected last on purpose: if it fails,
a run that stops at the first failure has already been through everything
else.  Passes alone in a fresh process and after the other tests."""
import pytest
import torch

from paper_2609_37062_b200 import workloads as wl
from gpu_util import MAX_ABS, MEAN_ABS, da, errors, oracle_of, to_device

pytestmark = pytest.mark.gpu


def reference(w):
    """The existing entry points with the policy the static step uses."""
    out, lse = da.run_workload(w, da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC))
    return out, lse


def static_step(w):
    out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((w.batch, w.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    da.decode_attn_step_static(da.shape_of_workload(w), w.seq_lens, w.q_bits, w.k_pool, w.v_pool, w.block_table,
                               w.seq_lens, out, lse)
    torch.cuda.synchronize()
    return out, lse


def test_two_calls_in_a_row_match_the_planned_path():
    """Second call: other lengths, more splits - whatever the first call left
    in the shared scratch must not leak into it."""
    first = to_device(wl.make_workload("a", [3000, 17, 1024, 1025, 0, 2500], 32, 8, 128, seed=31))
    second = to_device(wl.make_workload("b", [5000, 4097, 900], 32, 8, 128, seed=32))
    for w in (first, second):
        ref_out, ref_lse = reference(w)
        out, lse = static_step(w)
        assert torch.isfinite(out).all()
        mx, mean = errors(out, ref_out.cpu().numpy().astype("float64"))
        assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
        assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)     # same kernels, same split policy
    # and against the oracle, for good measure
    host = to_device(second, "cpu")
    ref64, _ = oracle_of(host)
    mx, mean = errors(out, ref64)
    assert mx <= MAX_ABS and mean <= MEAN_ABS


def test_tiny_config_and_limits():
    w = to_device(wl.config_tiny())
    ref_out, ref_lse = reference(w)
    out, lse = static_step(w)
    assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)
    # beyond the built-in scratch: refused with a status, nothing launched
    big = da.shape_of_workload(w)
    big.batch = 2000
    out2 = torch.zeros(4, device="cuda")
    rc = da.decode_attn_step_static(big, [16] * 2000, w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, out2,
                                    check=False)
    assert rc == da.DA_ERR_WORKSPACE_TOO_SMALL
    long = wl.make_workload("long", [16], 32, 8, 128, seed=1, max_pages_per_seq=70000)
    s = da.shape_of_workload(long)
    s.batch = 200                                            # 200 x 32 splits x 8 heads: more units than it holds
    rc = da.decode_attn_step_static(s, [1_000_000] * 200, w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens,
                                    out2, check=False)
    assert rc == da.DA_ERR_WORKSPACE_TOO_SMALL
    torch.cuda.synchronize()
    assert not out2.any()
