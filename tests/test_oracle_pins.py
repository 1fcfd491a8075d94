"""Pins for the fp64 CPU oracle: everything here checks the oracle against
something other than itself - brute force over densely gathered arrays with a
library softmax, closed forms, invariants, and a library attention routine."""
import math

import numpy as np
import pytest
import scipy.special
import torch

import oracle
from paper_2609_37062_b200 import workloads as wl


def bits_to_f64(bits) -> np.ndarray:
    if hasattr(bits, "detach"):
        bits = bits.detach().cpu().numpy()
    u = np.ascontiguousarray(bits).view(np.uint16).astype(np.uint32) << 16
    return u.view(np.float32).astype(np.float64)


def f32_to_bits(x) -> np.ndarray:
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def dense_gather(w, b):
    """Independent gather: plain python indexing of the pool tensors."""
    L = int(w.seq_lens[b])
    P = w.page_size
    k = np.empty((L, w.num_kv_heads, w.head_dim))
    v = np.empty_like(k)
    kp, vp = bits_to_f64(w.k_pool), bits_to_f64(w.v_pool)
    for t in range(L):
        page = int(w.block_table[b, t // P])
        slot = t % P
        if w.layout == "token_major":
            k[t], v[t] = kp[page, slot], vp[page, slot]
        else:
            k[t], v[t] = kp[page, :, slot], vp[page, :, slot]
    return k, v


def brute_force(w, scale=None):
    """softmax(q k^T scale) v per head with scipy's softmax on dense arrays."""
    B, Hq, D = w.q_bits.shape
    G = Hq // w.num_kv_heads
    scale = oracle.default_scale(D) if scale is None else scale
    q = bits_to_f64(w.q_bits)
    out = np.zeros((B, Hq, D))
    lse = np.full((B, Hq), -np.inf)
    for b in range(B):
        if int(w.seq_lens[b]) == 0:
            continue
        k, v = dense_gather(w, b)
        for h in range(Hq):
            s = (k[:, h // G, :] @ q[b, h]) * scale
            out[b, h] = scipy.special.softmax(s) @ v[:, h // G, :]
            lse[b, h] = scipy.special.logsumexp(s)
    return out, lse


def small_workload(lens, Hq=4, Hkv=2, D=16, seed=11, layout="token_major", **kw):
    return wl.make_workload("small", lens, Hq, Hkv, D, seed=seed, layout=layout, **kw)


# --------------------------------------------------------------------------- brute force

@pytest.mark.parametrize("layout", ["token_major", "head_major"])
def test_matches_brute_force_on_tiny_inputs(layout):
    w = small_workload([1, 5, 16, 17, 33, 50], Hq=6, Hkv=2, D=16, layout=layout, pool_pages=40)
    out, lse = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    ref_out, ref_lse = brute_force(w)
    assert np.max(np.abs(out - ref_out)) < 1e-12
    assert np.max(np.abs(lse - ref_lse)) < 1e-12


def test_config1_against_library_attention():
    """Third opinion on the tiny configuration: torch's fp64 attention routine
    on the gathered dense arrays."""
    w = wl.config_tiny()
    out, _ = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    G = w.num_q_heads // w.num_kv_heads
    q = torch.from_numpy(bits_to_f64(w.q_bits))
    for b in range(w.batch):
        k, v = dense_gather(w, b)
        kt = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(G, dim=0)   # [Hq, L, D]
        vt = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(G, dim=0)
        ref = torch.nn.functional.scaled_dot_product_attention(
            q[b].unsqueeze(1), kt, vt, scale=oracle.default_scale(w.head_dim)).squeeze(1)
        assert np.max(np.abs(out[b] - ref.numpy())) < 1e-12


def test_explicit_scale_is_used():
    w = small_workload([40])
    out, _ = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w), scale=0.37)
    ref, _ = brute_force(w, scale=0.37)
    assert np.max(np.abs(out - ref)) < 1e-12
    other, _ = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w), scale=0.11)
    assert np.max(np.abs(out - other)) > 1e-3


def test_default_scale_is_fp32_inverse_sqrt():
    assert oracle.default_scale(64) == 0.125
    assert oracle.default_scale(128) == float(np.float32(1.0 / math.sqrt(128.0)))


# --------------------------------------------------------------------------- softmax invariants

def test_probabilities_sum_to_one_and_match_library():
    w = small_workload([7, 129])
    inp = oracle.PagedInputs.from_workload(w)
    q = bits_to_f64(w.q_bits)
    for b in range(2):
        k, _ = dense_gather(w, b)
        for h in range(4):
            p = oracle.attention_probs(inp, b, h)
            assert abs(p.sum() - 1.0) < 1e-12
            assert (p >= 0).all()
            ref = scipy.special.softmax((k[:, h // 2, :] @ q[b, h]) * oracle.default_scale(16))
            assert np.max(np.abs(p - ref)) < 1e-13


def test_output_is_a_convex_combination_of_values():
    w = small_workload([3, 48, 100])
    out, _ = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    for b in range(3):
        _, v = dense_gather(w, b)
        for h in range(4):
            lo, hi = v[:, h // 2, :].min(axis=0), v[:, h // 2, :].max(axis=0)
            assert (out[b, h] >= lo - 1e-12).all() and (out[b, h] <= hi + 1e-12).all()


def test_adding_a_constant_to_values_shifts_the_output():
    """Integer-valued V (exact in bf16) plus an integer constant stays exact,
    so out must move by exactly that constant (to fp64 rounding)."""
    rng = np.random.default_rng(5)
    w = small_workload([37])
    vi = rng.integers(-8, 9, size=tuple(w.v_pool.shape)).astype(np.float32)
    w.v_pool = torch.from_numpy(f32_to_bits(vi).view(np.int16))
    base, _ = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    w.v_pool = torch.from_numpy(f32_to_bits(vi + 3.0).view(np.int16))
    moved, _ = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    assert np.max(np.abs(moved - base - 3.0)) < 1e-12


# --------------------------------------------------------------------------- closed forms

def test_zero_query_gives_the_mean_of_values():
    w = small_workload([1, 19, 64])
    w.q_bits = torch.zeros_like(w.q_bits)
    out, lse = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    for b in range(3):
        _, v = dense_gather(w, b)
        L = int(w.seq_lens[b])
        for h in range(4):
            assert np.max(np.abs(out[b, h] - v[:, h // 2, :].mean(axis=0))) < 1e-13
            assert abs(lse[b, h] - math.log(L)) < 1e-13


def test_single_token_returns_its_value_exactly():
    w = small_workload([1, 1])
    inp = oracle.PagedInputs.from_workload(w)
    out, lse = oracle.paged_decode_attention(inp)
    q = bits_to_f64(w.q_bits)
    for b in range(2):
        k, v = dense_gather(w, b)
        for h in range(4):
            assert np.array_equal(out[b, h], v[0, h // 2, :])            # bit for bit
            assert abs(lse[b, h] - oracle.default_scale(16) * float(k[0, h // 2] @ q[b, h])) < 1e-13


def test_equal_keys_give_the_mean_of_values():
    w = small_workload([23], Hq=2, Hkv=1)
    kp = w.k_pool.clone()
    kp[:] = kp[int(w.block_table[0, 0]), 0, 0]        # every key row equals one row
    w.k_pool = kp
    out, lse = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    _, v = dense_gather(w, 0)
    k, _ = dense_gather(w, 0)
    q = bits_to_f64(w.q_bits)
    for h in range(2):
        assert np.max(np.abs(out[0, h] - v[:, 0, :].mean(axis=0))) < 1e-13
        s0 = oracle.default_scale(16) * float(k[0, 0] @ q[0, h])
        assert abs(lse[0, h] - (s0 + math.log(23))) < 1e-12


@pytest.mark.parametrize("winner", [0, 15, 16, 30, 44])
def test_one_dominant_key_selects_its_value_exactly(winner):
    """Key `winner` has logit +1000 and all others -1000, so every other
    weight underflows to zero and the value row comes out bit for bit: pins
    that K row t and V row t are fetched from the same (page, slot, head)."""
    L, D = 45, 16
    w = small_workload([L], Hq=2, Hkv=2, D=D)
    q = np.zeros((1, 2, D), dtype=np.float32)
    q[:, :, 0] = 4.0                                   # scale 0.25 -> logit = k[0]
    w.q_bits = torch.from_numpy(f32_to_bits(q).view(np.int16))
    kp = bits_to_f64(w.k_pool).astype(np.float32)
    for t in range(L):
        page, slot = int(w.block_table[0, t // 16]), t % 16
        kp[page, slot, :, 0] = 1000.0 if t == winner else -1000.0
    w.k_pool = torch.from_numpy(f32_to_bits(kp).view(np.int16))
    out, lse = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    _, v = dense_gather(w, 0)
    for h in range(2):
        assert np.array_equal(out[0, h], v[winner, h, :])
        assert lse[0, h] == 1000.0


def test_empty_and_masked_rows_emit_zero():
    """Algorithm 1 step 2: a Project-Only row reads no KV and emits zero; an
    empty row does the same."""
    w = small_workload([0, 20, 33], pool_pages=8)
    inp = oracle.PagedInputs.from_workload(w)
    out, lse = oracle.paged_decode_attention(inp)
    assert not out[0].any() and np.isneginf(lse[0]).all()
    ref, _ = brute_force(w)
    assert np.max(np.abs(out[1:] - ref[1:])) < 1e-12
    masked, mlse = oracle.paged_decode_attention(inp, run_mask=[1, 0, 1])
    assert not masked[1].any() and np.isneginf(mlse[1]).all()
    assert np.array_equal(masked[2], out[2]) and np.array_equal(mlse[2], lse[2])


def test_large_logits_do_not_overflow():
    w = small_workload([64])
    qs = bits_to_f64(w.q_bits).astype(np.float32) * 512.0
    w.q_bits = torch.from_numpy(f32_to_bits(qs).view(np.int16))
    out, lse = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    ref, ref_lse = brute_force(w)
    assert np.isfinite(out).all() and np.isfinite(lse).all()
    assert np.max(np.abs(out - ref)) < 1e-11 and np.max(np.abs(lse - ref_lse)) < 1e-9


# --------------------------------------------------------------------------- paging, heads

def test_page_permutation_leaves_every_bit_unchanged():
    w = wl.config_tiny()
    out, lse = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    w2 = wl.permute_pages(w, seed=99)
    assert not torch.equal(w.block_table, w2.block_table)
    out2, lse2 = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w2))
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def test_unused_slots_and_pages_are_never_read():
    """The generator poisons unused slots and unreferenced pages with NaN."""
    w = wl.config_tiny()
    assert torch.isnan(w.k_pool.view(torch.bfloat16).float()).any()
    out, lse = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    assert np.isfinite(out).all() and np.isfinite(lse).all()


def test_gather_is_bit_exact():
    w = small_workload([50, 3], Hq=4, Hkv=2, D=16, layout="head_major")
    inp = oracle.PagedInputs.from_workload(w)
    for b in range(2):
        k, v = oracle.gather_kv(inp, b)
        L = int(w.seq_lens[b])
        kref = wl.normal_bf16_bits(wl.stream_key(11, wl.TENSOR_K, b), 0, L * 2 * 16).view(L, 2, 16)
        vref = wl.normal_bf16_bits(wl.stream_key(11, wl.TENSOR_V, b), 0, L * 2 * 16).view(L, 2, 16)
        assert np.array_equal(k.view(np.int16), kref.numpy())
        assert np.array_equal(v.view(np.int16), vref.numpy())


def test_heads_of_one_group_with_equal_queries_agree():
    w = small_workload([41], Hq=8, Hkv=2)
    qb = w.q_bits.clone()
    qb[0, 1:4] = qb[0, 0]
    qb[0, 5:8] = qb[0, 4]
    w.q_bits = qb
    out, _ = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    for h in (1, 2, 3):
        assert np.array_equal(out[0, h], out[0, 0])
        assert np.array_equal(out[0, 4 + h], out[0, 4])
    assert not np.array_equal(out[0, 0], out[0, 4])


def test_swapping_kv_heads_swaps_group_outputs():
    w = small_workload([29], Hq=4, Hkv=2)
    qb = w.q_bits.clone()
    qb[0, 2:4] = qb[0, 0:2]                      # both groups ask the same questions
    w.q_bits = qb
    out, _ = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    w.k_pool = w.k_pool.flip(2)                   # token-major: dim 2 is the KV head
    w.v_pool = w.v_pool.flip(2)
    swapped, _ = oracle.paged_decode_attention(oracle.PagedInputs.from_workload(w))
    assert np.array_equal(swapped[0, 0:2], out[0, 2:4])
    assert np.array_equal(swapped[0, 2:4], out[0, 0:2])


# --------------------------------------------------------------------------- split / merge algebra

def test_split_and_merge_reproduces_full_attention_for_every_cut():
    w = small_workload([37], Hq=2, Hkv=1)
    inp = oracle.PagedInputs.from_workload(w)
    full, full_lse = oracle.paged_decode_attention(inp)
    for a in range(0, 38):                        # a = 0 and a = L leave one side empty
        o1, m1, l1 = oracle.partial_attention(inp, 0, 1, 0, a)
        o2, m2, l2 = oracle.partial_attention(inp, 0, 1, a, 37)
        merged, lse = oracle.merge_partials([o1, o2], [m1, m2], [l1, l2])
        assert np.max(np.abs(merged - full[0, 1])) < 1e-13
        assert abs(lse - full_lse[0, 1]) < 1e-13


def test_merge_of_many_parts_matches_direct_formula():
    """The merge against its definition written with library calls."""
    rng = np.random.default_rng(3)
    n, D = 7, 5
    o = rng.normal(size=(n, D))
    m = rng.normal(size=n) * 3
    l = rng.uniform(0.5, 20, size=n)
    l[2], m[2] = 0.0, -np.inf                     # an empty part
    out, lse = oracle.merge_partials(o, m, l)
    live = l > 0
    logw = m[live] + np.log(l[live])
    ref_lse = scipy.special.logsumexp(logw)
    ref = scipy.special.softmax(logw) @ o[live]
    assert np.max(np.abs(out - ref)) < 1e-13 and abs(lse - ref_lse) < 1e-13
    zero, zlse = oracle.merge_partials(o[:2], [-np.inf, -np.inf], [0.0, 0.0])
    assert not zero.any() and np.isneginf(zlse)


def test_threads_do_not_change_results():
    w = wl.config_tiny()
    inp = oracle.PagedInputs.from_workload(w)
    a, _ = oracle.paged_decode_attention(inp, num_threads=1)
    b, _ = oracle.paged_decode_attention(inp, num_threads=4)
    assert np.array_equal(a, b)


# --------------------------------------------------------------------------- own-layer KV write

def test_append_writes_the_last_position_and_nothing_else():
    """Invariant 1: position seq_len - 1 of the layer's cache holds the row's
    own K/V after the write; every other byte of the pools is untouched."""
    w = small_workload([1, 16, 17, 40, 0], Hq=4, Hkv=2, D=16, pool_pages=12)
    inp = oracle.PagedInputs.from_workload(w)
    new_k = wl.normal_bf16_bits(wl.stream_key(5, wl.TENSOR_NEW_K, 0), 0, 5 * 2 * 16).view(5, 2, 16)
    new_v = wl.normal_bf16_bits(wl.stream_key(5, wl.TENSOR_NEW_V, 0), 0, 5 * 2 * 16).view(5, 2, 16)
    k2, v2 = oracle.append_kv(inp, new_k, new_v)
    expected_k, expected_v = w.k_pool.numpy().copy(), w.v_pool.numpy().copy()
    for b, L in enumerate(w.seq_lens.tolist()):
        if L == 0:
            continue
        page, slot = int(w.block_table[b, (L - 1) // 16]), (L - 1) % 16
        expected_k[page, slot] = new_k[b].numpy()
        expected_v[page, slot] = new_v[b].numpy()
    assert np.array_equal(k2.view(np.int16).reshape(expected_k.shape), expected_k)
    assert np.array_equal(v2.view(np.int16).reshape(expected_v.shape), expected_v)
    # reading back through the gather gives the new rows at the last position
    w2 = wl.make_workload("small", [1, 16, 17, 40, 0], 4, 2, 16, seed=11, pool_pages=12)
    w2.k_pool = torch.from_numpy(k2.view(np.int16).reshape(expected_k.shape))
    w2.v_pool = torch.from_numpy(v2.view(np.int16).reshape(expected_v.shape))
    inp2 = oracle.PagedInputs.from_workload(w2)
    for b, L in enumerate(w.seq_lens.tolist()):
        if L:
            gk, gv = oracle.gather_kv(inp2, b)
            assert np.array_equal(gk[L - 1].view(np.int16), new_k[b].numpy())
            assert np.array_equal(gv[L - 1].view(np.int16), new_v[b].numpy())


def test_input_decoding_matches_the_library_for_every_bit_pattern():
    """bf16 and fp16 patterns -> fp64, all 65,536 of each, against numpy / torch's reading of the
    same bits (subnormals, signed zeros, infinities included; NaNs as NaNs)."""
    import torch
    bits = np.arange(65536, dtype=np.uint16)
    want16 = bits.view(np.float16).astype(np.float64)
    got16 = oracle.decode_bits(bits, in_fp16=True)
    nan = np.isnan(want16)
    assert np.array_equal(np.isnan(got16), nan) and np.array_equal(got16[~nan], want16[~nan])
    assert np.array_equal(np.signbit(got16[~nan]), np.signbit(want16[~nan]))
    wantb = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    gotb = oracle.decode_bits(bits, in_fp16=False)
    nan = np.isnan(wantb)
    assert np.array_equal(np.isnan(gotb), nan) and np.array_equal(gotb[~nan], wantb[~nan])


def test_fp16_inputs_go_through_the_same_definition():
    """The attention of fp16 inputs equals dense attention over the decoded values (brute force)."""
    w = wl.make_workload("h", [37, 5], 4, 2, 64, seed=21, dtype="fp16")
    inp = oracle.PagedInputs.from_workload(w)
    out, lse = oracle.paged_decode_attention(inp)
    q = w.q_bits.numpy().view(np.float16).astype(np.float64)
    for b, L in enumerate(w.seq_lens.tolist()):
        k, v = oracle.gather_kv(inp, b)
        k = k.view(np.float16).astype(np.float64)
        v = v.view(np.float16).astype(np.float64)
        for h in range(4):
            s = (k[:, h // 2, :] @ q[b, h]) * oracle.default_scale(64)
            p = np.exp(s - s.max())
            assert np.max(np.abs(out[b, h] - (p[:, None] * v[:, h // 2, :]).sum(0) / p.sum())) < 1e-12
            assert abs(lse[b, h] - (s.max() + np.log(p.sum()))) < 1e-12
