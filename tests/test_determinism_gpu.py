"""Deterministic mode: split boundaries are a function of a sequence's own
length and the policy's chunk length, reductions run in logical token order
and the merge in ascending split order, so a sequence's output bits do not
depend on the batch it is served in, its position there, its neighbours'
lengths or where its pages live."""
import pytest
import torch

from paper_2609_37062_b200 import workloads as wl
from gpu_util import KERNELS, KERNEL_IDS, assert_parity, da, oracle_of, to_device

pytestmark = pytest.mark.gpu

HEADS = dict(num_q_heads=32, num_kv_heads=8, head_dim=128)


def run(lens, uids, policy, table_seed=None, pool_pages=None):
    w = wl.make_workload("det", lens, seed=4, seq_uids=uids, table_seed=table_seed, pool_pages=pool_pages,
                         device="cuda", **HEADS)
    out, lse = da.run_workload(w, policy)
    return out, lse, w


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("fused", [0, 1])
@pytest.mark.parametrize("chunk", [512, 0])
def test_bits_do_not_depend_on_batch_size_or_position(kernel, fused, chunk):
    pol = da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=chunk, kernel=kernel, fuse_combine=fused)
    L = 2500
    alone = {}
    for uid in (0, 3, 7):
        out, lse, w = run([L], [uid], pol)
        alone[uid] = (out[0].clone(), lse[0].clone())
    ref_out, ref_lse = oracle_of(to_device(w, "cpu"))
    assert_parity(out, lse, ref_out, ref_lse)
    for batch in (8, 64):
        uids = list(range(batch))
        out, lse, _ = run([L] * batch, uids, pol, table_seed=batch)
        for uid in (0, 3, 7):
            assert torch.equal(out[uid], alone[uid][0]) and torch.equal(lse[uid], alone[uid][1]), (batch, uid)
    # other positions in the batch
    uids = [11, 7, 12, 13, 3, 14, 0, 15]
    out, lse, _ = run([L] * 8, uids, pol, table_seed=5)
    for pos, uid in enumerate(uids):
        if uid in alone:
            assert torch.equal(out[pos], alone[uid][0]) and torch.equal(lse[pos], alone[uid][1])


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_bits_do_not_depend_on_neighbours_or_page_placement(kernel):
    pol = da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=256, kernel=kernel, fuse_combine=1)
    lens_a = [1000, 37, 4096, 513]
    uids_a = [20, 21, 22, 23]
    out_a, lse_a, _ = run(lens_a, uids_a, pol, table_seed=1)
    # same sequences, other neighbours (lengths and count), other page placement, a larger pool
    lens_b = [5, 513, 2000, 1000, 900, 4096, 64]
    uids_b = [30, 23, 31, 20, 32, 22, 33]
    out_b, lse_b, _ = run(lens_b, uids_b, pol, table_seed=2, pool_pages=3000)
    for pa, pb in ((0, 3), (2, 5), (3, 1)):
        assert torch.equal(out_a[pa], out_b[pb]) and torch.equal(lse_a[pa], lse_b[pb])


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_repeated_launches_give_the_same_bits(kernel):
    """No float atomics anywhere: AUTO mode is reproducible run to run too."""
    w = to_device(wl.config_short_chat(batch=32))
    pol = da.make_policy(kernel=kernel, fuse_combine=1)
    first, first_lse = da.run_workload(w, pol)
    for _ in range(3):
        again, again_lse = da.run_workload(w, pol)
        assert torch.equal(first, again) and torch.equal(first_lse, again_lse)


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_fused_and_separate_merge_give_the_same_bits(kernel):
    w = to_device(wl.config_long(context=6000))
    a, la = da.run_workload(w, da.make_policy(kernel=kernel, split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=512,
                                              fuse_combine=0))
    b, lb = da.run_workload(w, da.make_policy(kernel=kernel, split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=512,
                                              fuse_combine=1))
    assert torch.equal(a, b) and torch.equal(la, lb)


@pytest.mark.parametrize("splits", [2, 3, 4, 5, 8, 9, 13, 49, 300, 1024])
def test_every_merge_kernel_gives_the_fused_path_its_bits(splits):
    """The combine launch picks a kernel by the plan's largest split count (one thread per column
    up to 4 and up to 8 splits, the slice kernel beyond); all of them and the merge blocks of a
    fused launch add the same four chains in the same order."""
    w = to_device(wl.make_workload("m", [4000, 17, 900, 2500, 64], 32, 8, 128, seed=41))
    pol = dict(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=splits)
    a, la = da.run_workload(w, da.make_policy(fuse_combine=0, **pol))
    b, lb = da.run_workload(w, da.make_policy(fuse_combine=1, **pol))
    assert torch.equal(a, b) and torch.equal(la, lb)


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_sequences_beyond_the_default_split_bound(kernel):
    """Past 32,768 tokens the default bound of 32 splits lengthens the chunks (40,000 tokens: 1,264 each): still a
    function of the sequence's own length, so its bits do not change with the company it keeps."""
    pol = da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC, kernel=kernel)
    out_a, lse_a, w = run([40000], [50], pol)
    ref_out, ref_lse = oracle_of(to_device(w, "cpu"))
    assert_parity(out_a, lse_a, ref_out, ref_lse)
    out_b, lse_b, _ = run([700, 40000, 33000, 16], [51, 50, 52, 53], pol, table_seed=3)
    assert torch.equal(out_a[0], out_b[1]) and torch.equal(lse_a[0], lse_b[1])
    out_c, lse_c, _ = run([33000, 40000], [52, 50], pol, table_seed=4)
    assert torch.equal(out_b[2], out_c[0]) and torch.equal(out_a[0], out_c[1])
