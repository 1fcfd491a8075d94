"""decode_attn_step_static: a whole step whose scratch (work list, records)
is a static device array inside the library, for callers that cannot use the
CUDA allocator at call time - an engine whose KV pool already owns all of HBM,
or a path that cannot take an allocation's device-wide sync.  Held against the
ordinary plan / run / combine path it mirrors, bit for bit; free device memory
must not move across calls; device-detected conditions must be readable.
(The file name keeps it last in collection order, behind the tests of the
entry points it is compared with.)  Passes alone in a fresh process and after
the other tests."""
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


def test_calls_leave_free_device_memory_unchanged():
    """The point of the entry point: after the first call (which resolves the array's address and
    may load kernels) no call takes or returns device memory."""
    w = to_device(wl.make_workload("m", [3000, 700, 4097], 32, 8, 128, seed=33))
    out = torch.empty((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32, device="cuda")
    lse = torch.empty((w.batch, w.num_q_heads), dtype=torch.float32, device="cuda")
    shape = da.shape_of_workload(w)
    lens_host = w.seq_lens.cpu().numpy()
    call = lambda: da.decode_attn_step_static(shape, lens_host, w.q_bits, w.k_pool, w.v_pool, w.block_table,
                                              w.seq_lens, out, lse)
    call()
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        call()
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free0
    assert da.decode_attn_last_device_status(None) == da.DA_OK


def test_device_side_conditions_are_reported_and_capture_is_refused():
    w = to_device(wl.make_workload("s", [3000, 700, 4097], 32, 8, 128, seed=34))
    out = torch.empty((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32, device="cuda")
    shape = da.shape_of_workload(w)
    assert da.decode_attn_last_device_status(None) in (da.DA_OK, da.DA_ERR_STALE_PLAN, da.DA_ERR_BAD_PAGE)  # drain
    stale = w.seq_lens.clone()
    stale[1] += 1                                            # the device lengths are not the planned ones
    da.decode_attn_step_static(shape, w.seq_lens.cpu().numpy(), w.q_bits, w.k_pool, w.v_pool, w.block_table, stale, out)
    assert da.decode_attn_last_device_status(None) == da.DA_ERR_STALE_PLAN
    assert da.decode_attn_last_device_status(None) == da.DA_OK
    bt = w.block_table.clone()
    bt[0, 3] = w.num_pages
    da.decode_attn_step_static(shape, w.seq_lens.cpu().numpy(), w.q_bits, w.k_pool, w.v_pool, bt, w.seq_lens, out)
    assert da.decode_attn_last_device_status(None) == da.DA_ERR_BAD_PAGE
    # more than 8 KV heads are served like any other shape
    many = to_device(wl.make_workload("h", [2500, 90], 16, 16, 64, seed=35))
    ref_out, ref_lse = reference(many)
    got, got_lse = static_step(many)
    assert torch.equal(got, ref_out) and torch.equal(got_lse, ref_lse)
    # a capturing stream is refused: the call plans and uploads on the host every time
    lens_host = w.seq_lens.cpu().numpy()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            rc = da.decode_attn_step_static(shape, lens_host, w.q_bits, w.k_pool, w.v_pool, w.block_table,
                                            w.seq_lens, out, check=False)
    assert rc == da.DA_ERR_UNSUPPORTED
