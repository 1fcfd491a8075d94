"""Page gathering must be bit-exact: the TMA path's own view of the pools is
compared byte for byte with the CPU gather."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_37062_b200 import workloads as wl
from gpu_util import da, to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("layout", ["token_major", "head_major"])
@pytest.mark.parametrize("maker", [wl.config_tiny, lambda layout: wl.config_long(context=1500, layout=layout)],
                         ids=["tiny", "long1500"])
def test_debug_gather_matches_the_host_gather(layout, maker):
    w = maker(layout=layout)
    inp = oracle.PagedInputs.from_workload(w)
    wd = to_device(w)
    pol = da.make_policy(kernel=da.DA_KERNEL_MMA_TMA, split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=112)
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


def test_gather_probe_checksums_match_the_bytes_of_each_unit():
    """XOR of all 32-bit words of the K and V pages a unit streams."""
    w = wl.config_short_chat(batch=6)
    wd = to_device(w)
    plan = da.decode_attn_plan(da.shape_of_workload(wd), da.make_policy(kernel=da.DA_KERNEL_MMA_TMA, chunk_tokens=64),
                               w.seq_lens)
    units = da.decode_attn_plan_get_units(plan)
    chk = torch.full((len(units),), 0xFFFF, dtype=torch.int32, device="cuda")
    da.decode_attn_gather_probe(plan, wd.k_pool, wd.v_pool, wd.block_table, chk)
    assert da.decode_attn_last_device_status(plan) == da.DA_OK
    got = chk.cpu().numpy().view(np.uint32)
    kp = w.k_pool.numpy().view(np.uint16)
    vp = w.v_pool.numpy().view(np.uint16)
    for i, u in enumerate(units):
        acc = np.uint32(0)
        for page_idx in range(u.tok_begin // 16, (u.tok_end + 15) // 16):
            page = int(w.block_table[u.seq, page_idx])
            for pool in (kp, vp):
                words = np.ascontiguousarray(pool[page, :, u.kv_head, :]).view(np.uint32)
                acc ^= np.bitwise_xor.reduce(words.ravel())
        assert got[i] == acc, (i, u.seq, u.kv_head)
