"""Host-side checks that need no GPU: the library loads and exports what the
header declares, argument validation answers with status codes, and the
split planner's work lists cover every token exactly once."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2609_37062_b200 import build as da_build

da_build.build()
from paper_2609_37062_b200 import binding as da  # noqa: E402
from paper_2609_37062_b200 import workloads as wl  # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "decode_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(decode_attn_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 15
    lib = ctypes.CDLL(da.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(da.EXPORTED) == names


def test_version_and_strerror():
    assert "sm_100a" in da.decode_attn_version()
    assert da.decode_attn_strerror(da.DA_OK) == "ok"
    for code in range(-7, 0):
        assert da.decode_attn_strerror(code) != "unknown status"
    assert da.decode_attn_strerror(-99) == "unknown status"


def test_struct_sizes_match_the_header():
    assert ctypes.sizeof(da.Unit) == 32
    assert ctypes.sizeof(da.Policy) == 64 and da.Policy.shared_prefix_tokens.offset == 40
    assert ctypes.sizeof(da.Shape) == 96
    assert ctypes.sizeof(da.RunArgs) == 104 and da.RunArgs.new_k.offset == 88      # 88: the struct before new_k / new_v, still accepted


def shape(B=4, Hq=32, Hkv=8, D=128, mpp=8192, pages=1 << 20):
    return da.make_shape(B, Hq, Hkv, D, 16, mpp, pages, (16 * Hkv * D, Hkv * D, D))


def layout(lens, policy, sm=148, ctas=2, **kw):
    return da.decode_attn_plan_layout(shape(B=len(lens), **kw), policy, lens, sm, ctas)


def covered_exactly_once(units, lens, Hkv):
    """Every (sequence, KV head) token range is tiled by its units."""
    per = {}
    for u in units:
        per.setdefault((u.seq, u.kv_head), []).append(u)
    assert len(per) == len(lens) * Hkv
    for (b, g), us in per.items():
        us.sort(key=lambda u: u.split_index)
        assert [u.split_index for u in us] == list(range(len(us)))
        assert all(u.n_splits == len(us) and u.seq_len == lens[b] for u in us)
        pos = 0
        for u in us:
            assert u.tok_begin % 16 == 0
            if u.tok_end > u.tok_begin:
                assert u.tok_begin == pos
                pos = u.tok_end
            else:
                assert u.tok_end == u.tok_begin        # an empty split
        assert pos == lens[b]
        if len(us) == 1:
            assert us[0].slot == -1
        else:
            slots = [u.slot for u in us]
            assert slots == list(range(slots[0], slots[0] + len(us))) and slots[0] >= 0


@pytest.mark.parametrize("lens", [[17, 64, 129, 300], [32768], [0, 1, 15, 16, 17], [5000] * 64,
                                  wl.lengths_short_chat(64, 2), wl.lengths_shared_prefix(256, 3)])
@pytest.mark.parametrize("mode", [da.DA_SPLIT_AUTO, da.DA_SPLIT_DETERMINISTIC, da.DA_SPLIT_FIXED_COUNT])
def test_units_tile_every_sequence(lens, mode):
    pol = da.make_policy(split_mode=mode, fixed_count=3)
    units, splits, slot_base, n_slots, chunk = layout(lens, pol)
    covered_exactly_once(units, lens, 8)
    assert n_slots == sum(int(s) for s in splits if s > 1)
    costs = [u.tok_end - u.tok_begin for u in units]
    pages = [(c + 15) // 16 for c in costs]
    assert pages == sorted(pages, reverse=True)         # most expensive first
    for b, s in enumerate(splits):
        assert (slot_base[b] == -1) == (s == 1)


def test_auto_fills_the_machine_for_one_long_sequence():
    units, splits, _, n_slots, chunk = layout([32768], da.make_policy(), sm=148, ctas=2)
    assert 8 <= splits[0] <= 64
    assert len(units) <= 296 and len(units) > 296 - 8
    sizes = {u.tok_end - u.tok_begin for u in units}
    assert max(sizes) - min(sizes) <= 16                # near-equal cost
    assert chunk % 16 == 0 and chunk >= 256


def test_auto_never_goes_below_the_minimum_chunk():
    units, splits, _, _, chunk = layout([300, 200], da.make_policy())
    assert chunk == 256 and list(splits) == [2, 1]
    units, splits, _, _, chunk = layout([300, 200], da.make_policy(chunk_tokens=512))
    assert list(splits) == [1, 1]


def test_auto_uses_whole_waves_for_large_batches():
    lens = [512] * 256
    units, splits, _, n_slots, _ = layout(lens, da.make_policy())
    assert set(splits) == {1} and n_slots == 0 and len(units) == 2048


def test_auto_cuts_long_sequences_finer_when_whole_waves_do_not_divide():
    # 64 sequences x 8 heads = 512 units on 296 resident blocks: two units for most blocks, one for the rest.
    # Four splits of 32,768 tokens make 2,048 units, seven for most blocks: the heaviest block carries 12 % less.
    units, splits, _, _, chunk = layout([131072] * 64, da.make_policy(), mpp=8192)
    assert set(splits) == {4} and chunk == 32768 and len(units) == 2048
    covered_exactly_once(units, [131072] * 64, 8)
    units, splits, _, _, chunk = layout([8192] * 64, da.make_policy())
    assert set(splits) == {4} and chunk == 2048 and len(units) == 2048
    # never below the policy's own smallest chunk
    units, splits, _, _, chunk = layout([8192] * 64, da.make_policy(chunk_tokens=4096))
    assert set(splits) == {1} and chunk == 8192
    # units that a cut would bring under 2,048 tokens stay whole
    units, splits, _, _, chunk = layout([4096] * 64, da.make_policy())
    assert set(splits) == {1} and chunk == 4096 and len(units) == 512
    # waves that divide well enough are left alone (2,048 units on 296 blocks: 6.9 per block)
    units, splits, _, _, _ = layout([32768] * 256, da.make_policy())
    assert set(splits) == {1} and len(units) == 2048
    # one long sequence still fills the machine exactly
    units, splits, _, _, _ = layout([32768], da.make_policy())
    assert len(units) == 296


def test_auto_is_a_pure_function_of_its_inputs():
    lens = wl.lengths_short_chat(64, 2)
    a = layout(lens, da.make_policy())
    b = layout(lens, da.make_policy())
    assert [(u.seq, u.kv_head, u.tok_begin, u.tok_end, u.slot) for u in a[0]] == \
           [(u.seq, u.kv_head, u.tok_begin, u.tok_end, u.slot) for u in b[0]]
    c = layout(lens, da.make_policy(), sm=64)
    assert c[4] >= a[4]                                 # fewer SMs, never shorter chunks


def test_deterministic_boundaries_depend_on_the_length_alone():
    pol = da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=512)

    def cuts(lens, b, **kw):
        units = layout(lens, pol, **kw)[0]
        return sorted({(u.split_index, u.tok_begin, u.tok_end) for u in units if u.seq == b})

    alone = cuts([5000], 0)
    assert alone == [(i, 512 * i, min(512 * (i + 1), 5000)) for i in range(10)]
    assert cuts([77, 5000, 123456], 1) == alone
    assert cuts([5000] * 256, 200) == alone
    assert cuts([5000, 9], 0, sm=16, ctas=1) == alone
    assert layout([5000], da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC))[4] == 256


def test_fixed_count_gives_empty_trailing_splits():
    pol = da.make_policy(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=8)
    units, splits, _, n_slots, _ = layout([40], pol)
    assert list(splits) == [8] and n_slots == 8
    mine = sorted([u for u in units if u.kv_head == 0], key=lambda u: u.split_index)
    assert [(u.tok_begin, u.tok_end) for u in mine][:4] == [(0, 16), (16, 32), (32, 40), (48, 48)]
    assert all(u.tok_end == u.tok_begin for u in mine[3:])


def test_deterministic_default_bounds_the_splits_by_the_sequence_alone():
    """At most 32 splits by default: a longer sequence gets longer chunks, whatever else is in the batch."""
    det = da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC)
    expect = {32768: (32, 1024), 131072: (32, 4096), 40000: (32, 1264), 5000: (20, 256), 100: (1, 256),
              8192: (32, 256), 8200: (31, 272), 2048: (8, 256)}
    for batch in ([131072], [100, 40000, 131072, 5000, 32768], [32768] * 9 + [131072, 40000], [8192, 8200, 2048, 100]):
        units, splits, _, _, _ = layout(batch, det)
        covered_exactly_once(units, batch, 8)
        for b, L in enumerate(batch):
            n, chunk = expect[L]
            assert splits[b] == n
            mine = sorted([u for u in units if u.seq == b and u.kv_head == 0], key=lambda u: u.split_index)
            assert [u.tok_begin for u in mine] == [min(i * chunk, (L + 15) // 16 * 16) for i in range(n)]
    units, splits, _, _, _ = layout([131072], da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC, max_splits=512,
                                                             chunk_tokens=1024))
    assert splits[0] == 128                                   # fixed 1,024-token chunks on request


def test_max_splits_caps_the_split_count():
    units, splits, _, _, _ = layout([131072], da.make_policy(max_splits=16, chunk_tokens=16))
    assert splits[0] == 16


def test_groups_of_up_to_16_heads_plan_like_any_other():
    for hq in (72, 96, 128):                                  # groups of 9, 12, 16
        units, splits, _, _, _ = layout([5000, 100], da.make_policy(), Hq=hq, Hkv=8)
        covered_exactly_once(units, [5000, 100], 8)


def test_invalid_shapes_and_policies_are_rejected():
    L = [100]
    ok = da.make_policy()
    bad = [
        (dict(Hq=30), ok, da.DA_ERR_INVALID_ARG),           # heads do not divide
        (dict(Hq=136, Hkv=8), ok, da.DA_ERR_UNSUPPORTED),   # group of 17
        (dict(D=96), ok, da.DA_ERR_INVALID_ARG),            # stride rule holds but dim unsupported
        (dict(mpp=3), ok, da.DA_ERR_INVALID_ARG),           # block table row too short
        ({}, da.make_policy(split_mode=7), da.DA_ERR_INVALID_ARG),
        ({}, da.make_policy(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=0), da.DA_ERR_INVALID_ARG),
        ({}, da.make_policy(chunk_tokens=100), da.DA_ERR_INVALID_ARG),
        ({}, da.make_policy(kernel=9), da.DA_ERR_INVALID_ARG),
    ]
    for kw, pol, code in bad:
        with pytest.raises(da.DecodeAttnError) as e:
            layout(L, pol, **kw)
        if kw.get("D") == 96:
            assert e.value.status in (da.DA_ERR_INVALID_ARG, da.DA_ERR_UNSUPPORTED)
        else:
            assert e.value.status == code, (kw, e.value.status)
    for ps in (1, 8, 24, 48, 512):                           # pages hold 16, 32, 64, 128 or 256 tokens
        s = shape(B=1)
        s.page_size = ps
        with pytest.raises(da.DecodeAttnError) as e:
            da.decode_attn_plan_layout(s, ok, L, 148, 2)
        assert e.value.status == da.DA_ERR_UNSUPPORTED
    s = shape(B=1)
    s.k_stride_token = 100                                   # not a multiple of 8 elements
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_plan_layout(s, ok, L, 148, 2)
    assert e.value.status == da.DA_ERR_INVALID_ARG
    with pytest.raises(da.DecodeAttnError):
        layout([-1], ok)


def test_layout_does_not_depend_on_the_page_size():
    """The planner counts in 16-token tiles; the pool's page size only bounds the block table."""
    lens = [33, 1000, 4097, 0, 257]
    for pol in (da.make_policy(), da.make_policy(split_mode=da.DA_SPLIT_DETERMINISTIC, chunk_tokens=256),
                da.make_policy(split_mode=da.DA_SPLIT_FIXED_COUNT, fixed_count=5)):
        ref = None
        for ps in (16, 32, 64, 128, 256):
            s = da.make_shape(len(lens), 32, 8, 128, ps, 8192 * 16 // ps, 1 << 16, (ps * 8 * 128, 8 * 128, 128))
            units = da.decode_attn_plan_layout(s, pol, lens, 148, 2)[0]
            key = [(u.seq, u.kv_head, u.tok_begin, u.tok_end, u.slot, u.split_index, u.n_splits) for u in units]
            ref = ref or key
            assert key == ref
    # the block-table bound does use the page size
    s = da.make_shape(1, 32, 8, 128, 64, 4, 1 << 16, (64 * 8 * 128, 8 * 128, 128))
    da.decode_attn_plan_layout(s, da.make_policy(), [256], 148, 2)
    with pytest.raises(da.DecodeAttnError):
        da.decode_attn_plan_layout(s, da.make_policy(), [257], 148, 2)


def test_validate_block_table():
    w = wl.config_tiny()
    s = da.shape_of_workload(w)
    assert da.decode_attn_validate_block_table(s, w.seq_lens, w.block_table) == da.DA_OK
    bt = w.block_table.clone()
    bt[2, 3] = 64
    assert da.decode_attn_validate_block_table(s, w.seq_lens, bt) == da.DA_ERR_BAD_PAGE
    bt[2, 3] = -1
    assert da.decode_attn_validate_block_table(s, w.seq_lens, bt) == da.DA_ERR_BAD_PAGE
    bt = w.block_table.clone()
    bt[0, 2] = 1000                                          # beyond ceil(17/16) pages: never read
    assert da.decode_attn_validate_block_table(s, w.seq_lens, bt) == da.DA_OK


def test_compute_entry_points_fail_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    w = wl.config_tiny()
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_plan(da.shape_of_workload(w), da.make_policy(), w.seq_lens)
    assert e.value.status == da.DA_ERR_CUDA


def test_shared_prefix_layout_and_validation():
    lens = wl.lengths_shared_prefix(37, 3, prefix=1536)
    lens[5] = 1536                                            # a sequence that is nothing but the prefix
    pol = da.make_policy(shared_prefix_tokens=1536, kernel=da.DA_KERNEL_MMA_TMA)
    units, splits, slot_base, n_slots, _ = layout(lens, pol)
    prefix_units = [u for u in units if u.kv_head >> 16]
    own = [u for u in units if not (u.kv_head >> 16)]
    assert units[: len(prefix_units)] == prefix_units          # launched first
    blocks = (37 + 3) // 4
    chunks = len({u.split_index for u in prefix_units})
    assert len(prefix_units) == blocks * 8 * chunks
    for u in prefix_units:
        assert u.slot == -2 and 0 <= u.tok_begin < u.tok_end <= 1536 and 1 <= (u.kv_head >> 16) <= 4
    assert sorted({u.kv_head >> 16 for u in prefix_units}) == [1, 4]          # the last block holds one sequence
    # the prefix chunks tile [0, 1536) and every sequence's own units tile [1536, L)
    cuts = sorted({(u.tok_begin, u.tok_end) for u in prefix_units})
    assert cuts[0][0] == 0 and cuts[-1][1] == 1536 and all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
    for b, L in enumerate(lens):
        mine = sorted([u for u in own if u.seq == b and u.kv_head == 0], key=lambda u: u.split_index)
        assert splits[b] == chunks + len(mine) and slot_base[b] >= 0
        pos = 1536
        for i, u in enumerate(mine):
            assert u.tok_begin == pos and u.split_index == chunks + i and u.slot == slot_base[b] + chunks + i
            pos = u.tok_end
        assert pos == L
    assert n_slots == int(sum(splits))
    with pytest.raises(da.DecodeAttnError):
        layout([1000, 2000], pol)                             # shorter than the prefix
    with pytest.raises(da.DecodeAttnError) as e:
        layout(lens, da.make_policy(shared_prefix_tokens=1536, fuse_combine=1))
    assert e.value.status == da.DA_ERR_UNSUPPORTED
    w = wl.config_shared_prefix(batch=6, prefix=64)
    s = da.shape_of_workload(w)
    assert da.decode_attn_validate_shared_prefix(s, 64, w.seq_lens, w.block_table) == da.DA_OK
    bt = w.block_table.clone()
    bt[3, 2] = bt[3, 5]
    assert da.decode_attn_validate_shared_prefix(s, 64, w.seq_lens, bt) == da.DA_ERR_BAD_PAGE
    assert da.decode_attn_validate_shared_prefix(s, 60, w.seq_lens, w.block_table) == da.DA_ERR_INVALID_ARG


def test_tcgen05_prefix_layout():
    """The plan for the tcgen05 prefix kernel: 128 query rows per unit (128 / G sequences), chunks
    of whole 128-token tiles (AUTO), prefix units first; what follows the prefix is planned as before."""
    for hq, hkv, batch, prefix in ((32, 8, 70, 1536), (8, 8, 300, 1024), (16, 2, 40, 112 * 16)):
        G = hq // hkv
        lens = wl.lengths_shared_prefix(batch, 5, prefix=prefix)
        for mode, chunk in ((da.DA_SPLIT_AUTO, 0), (da.DA_SPLIT_DETERMINISTIC, 0), (da.DA_SPLIT_DETERMINISTIC, 128)):
            pol = da.make_policy(shared_prefix_tokens=prefix, kernel=da.DA_KERNEL_UMMA_PREFIX, split_mode=mode,
                                 chunk_tokens=chunk)
            units, splits, slot_base, n_slots, _ = layout(lens, pol, Hq=hq, Hkv=hkv, D=128)
            prefix_units = [u for u in units if u.kv_head >> 16]
            assert units[: len(prefix_units)] == prefix_units
            per_block = 128 // G
            blocks = -(-batch // per_block)
            chunks = len({u.split_index for u in prefix_units})
            assert len(prefix_units) == blocks * hkv * chunks
            for u in prefix_units:
                assert u.slot == -2 and u.seq % per_block == 0 and 1 <= (u.kv_head >> 16) <= per_block
                assert 0 < u.tok_end - u.tok_begin and u.tok_begin % 16 == 0 and u.tok_end % 16 == 0
                if mode == da.DA_SPLIT_AUTO:
                    assert u.tok_begin % 128 == 0 and (u.tok_end % 128 == 0 or u.tok_end == prefix)
            cuts = sorted({(u.tok_begin, u.tok_end) for u in prefix_units})
            assert cuts[0][0] == 0 and cuts[-1][1] == prefix and all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
            assert n_slots == int(sum(splits)) and all(s >= chunks for s in splits)
    # head_dim 64, or no shared prefix at all: not this kernel's
    with pytest.raises(da.DecodeAttnError) as e:
        layout([300, 400], da.make_policy(shared_prefix_tokens=256, kernel=da.DA_KERNEL_UMMA_PREFIX), Hq=8, Hkv=2, D=64)
    assert e.value.status == da.DA_ERR_UNSUPPORTED
    with pytest.raises(da.DecodeAttnError) as e:
        layout([300, 400], da.make_policy(kernel=da.DA_KERNEL_UMMA_PREFIX))
    assert e.value.status == da.DA_ERR_UNSUPPORTED
