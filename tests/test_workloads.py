"""Checks of the seeded input generators (no attention arithmetic involved)."""
import os

import numpy as np
import torch

from paper_2609_37062_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _f32(bits):
    return bits.view(torch.bfloat16).float()


def test_values_look_standard_normal():
    x = _f32(wl.normal_bf16_bits(wl.stream_key(0, wl.TENSOR_K, 0), 0, 1 << 18))
    assert abs(float(x.mean())) < 0.01
    assert abs(float(x.std()) - 1.0) < 0.01
    assert float(x.abs().max()) < 7.0
    assert abs(float((x.abs() < 1.0).float().mean()) - 0.6827) < 0.01


def test_stream_is_counter_based():
    key = wl.stream_key(3, wl.TENSOR_V, 5)
    whole = wl.normal_bf16_bits(key, 0, 4096)
    part = wl.normal_bf16_bits(key, 1000, 96)
    assert torch.equal(whole[1000:1096], part)
    other = wl.normal_bf16_bits(wl.stream_key(3, wl.TENSOR_V, 6), 0, 4096)
    assert not torch.equal(whole, other)


def test_paper_kv_byte_accounting():
    """Appendix D: b = 4 KB per token per layer for 8 KV heads of 128 dims in a
    16-bit type; 128 KB over 32 layers (Appendix C)."""
    with open(os.path.join(GOLDEN, "kv_bytes_per_token.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for hkv, d, nbytes, layers, per_layer, per_token in rows:
        b = wl.kv_bytes_per_token(int(hkv), int(d), int(nbytes))
        assert b == int(per_layer)
        assert b * int(layers) == int(per_token)
    w = wl.config_long(context=64)
    assert w.kv_bytes_per_token == 4096 and w.logical_kv_bytes == 64 * 4096


def test_tiny_config_shape():
    w = wl.config_tiny()
    assert w.seq_lens.tolist() == [17, 64, 129, 300]
    assert (w.num_q_heads, w.num_kv_heads, w.head_dim, w.page_size, w.num_pages) == (8, 2, 64, 16, 64)
    used = []
    for b, L in enumerate(w.seq_lens.tolist()):
        n = (L + 15) // 16
        used += w.block_table[b, :n].tolist()
        assert (w.block_table[b, n:] == -1).all()
    assert len(used) == 34 and len(set(used)) == 34 and min(used) >= 0 and max(used) < 64
    assert used != sorted(used)                       # shuffled


def test_sequence_content_is_independent_of_batch():
    a = wl.config_sweep_cell(100, 1)
    b = wl.config_sweep_cell(100, 4)
    P = 16
    for layout_w in (a, b):
        assert layout_w.q_bits.shape[0] == layout_w.batch
    assert torch.equal(a.q_bits[0], b.q_bits[0])
    for t in (0, 17, 99):
        pa, pb = int(a.block_table[0, t // P]), int(b.block_table[0, t // P])
        assert torch.equal(a.k_pool[pa, t % P], b.k_pool[pb, t % P])
        assert torch.equal(a.v_pool[pa, t % P], b.v_pool[pb, t % P])


def test_layouts_hold_the_same_logical_rows():
    a = wl.make_workload("a", [40, 7], 4, 2, 16, seed=8, layout="token_major")
    b = wl.make_workload("b", [40, 7], 4, 2, 16, seed=8, layout="head_major")
    assert torch.equal(a.block_table, b.block_table)
    for s in range(2):
        for t in range(int(a.seq_lens[s])):
            page = int(a.block_table[s, t // 16])
            assert torch.equal(a.k_pool[page, t % 16], b.k_pool[page, :, t % 16])
    assert a.strides == (16 * 2 * 16, 2 * 16, 16) and b.strides == (2 * 16 * 16, 16, 16 * 16)


def test_shared_prefix_pages_are_shared():
    w = wl.config_shared_prefix(batch=8, prefix=64)
    first = w.block_table[0, :4]
    assert all(torch.equal(w.block_table[i, :4], first) for i in range(8))
    own = [set(w.block_table[i, 4:(int(w.seq_lens[i]) + 15) // 16].tolist()) for i in range(8)]
    for i in range(8):
        for j in range(i):
            assert not own[i] & own[j]
    assert w.unique_tokens == 64 + sum(int(l) - 64 for l in w.seq_lens)
    assert w.logical_tokens == int(w.seq_lens.sum())


def test_length_mixes():
    chat = wl.lengths_short_chat(4096, seed=2)
    assert min(chat) >= 1
    assert 350 < np.mean(chat) < 450                 # median 180 * exp(0.125) + 200.5 = 404
    pre = wl.lengths_shared_prefix(256, seed=3)
    assert min(pre) >= 1536 + 16 and max(pre) <= 1536 + 256


def test_alias_rule_reuses_pages():
    w = wl.config_sweep_cell(64, 6, alias_after=2)
    assert torch.equal(w.block_table[4], w.block_table[0])
    assert torch.equal(w.block_table[5], w.block_table[1])
    assert torch.equal(w.q_bits[4], w.q_bits[0])
    assert w.num_pages == 8 and w.unique_tokens == 128


def test_page_permutation_keeps_logical_content():
    w = wl.config_tiny()
    w2 = wl.permute_pages(w, seed=1)
    for b in range(4):
        for t in (0, 16, int(w.seq_lens[b]) - 1):
            p1, p2 = int(w.block_table[b, t // 16]), int(w2.block_table[b, t // 16])
            assert torch.equal(w.k_pool[p1, t % 16], w2.k_pool[p2, t % 16])
