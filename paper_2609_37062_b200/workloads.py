"""Seeded synthetic inputs for paged decode attention.

This module only *generates bytes*: bf16 bit patterns for q / K / V, length
mixes, block tables and physical page pools.  It contains none of the
attention arithmetic, so both the CPU oracle's tests and the CUDA path's tests
can feed on it without sharing any of the method's code.

Values are i.i.d. N(0,1) rounded to bf16 (round-to-nearest-even), drawn from a
counter-based generator keyed by (seed, tensor id, sequence uid, element
index).  A sequence's logical content therefore does not depend on which batch
it is placed in, nor on where its pages land in the physical pool; that is
what lets the deterministic-mode tests compare one sequence across batch
sizes.  Everything is written with torch integer / float ops so the same code
fills a small CPU pool for the oracle or a multi-GiB pool directly on the GPU.

The length mixes follow the shapes of the serving workloads of the paper's
Table 1 (short chat-style generations, few-shot prompts that share a long
cached prefix, long runaway generations); no dataset item is used.
"""
from __future__ import annotations

import math
import dataclasses
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import torch

TENSOR_Q = 1
TENSOR_K = 2
TENSOR_V = 3
TENSOR_NEW_K = 4
TENSOR_NEW_V = 5

_MASK64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Reinterpret an unsigned 64-bit python int as signed (torch has no uint64 math)."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


_C1 = _s64(0xBF58476D1CE4E5B9)
_C2 = _s64(0x94D049BB133111EB)
_GOLD = _s64(0x9E3779B97F4A7C15)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right on int64 tensors."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64_t(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser with wrap-around int64 arithmetic."""
    x = (x ^ _lsr(x, 30)) * _C1
    x = (x ^ _lsr(x, 27)) * _C2
    return x ^ _lsr(x, 31)


def _mix64_i(x: int) -> int:
    x &= _MASK64
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _MASK64
    return x ^ (x >> 31)


def stream_key(seed: int, tensor_id: int, uid: int) -> int:
    """Key of the value stream of one logical tensor of one sequence."""
    k = _mix64_i(seed * 0x9E3779B97F4A7C15 + tensor_id)
    return _mix64_i(k ^ ((uid + 1) * 0xD1342543DE82EF95))


def normal_bf16_bits(key: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """`count` N(0,1) samples as bf16 bit patterns (int16 tensor).

    Element i (global index start+i of the stream `key`) depends only on
    (key, start+i): Box-Muller on two 24-bit uniforms taken from one
    splitmix64 output.
    """
    if count == 0:
        return torch.empty(0, dtype=torch.int16, device=device)
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    h = _mix64_t(idx * _GOLD + _s64(key))
    u1 = (_lsr(h, 40).to(torch.float32) + 1.0) * (1.0 / 16777216.0)      # (0, 1]
    u2 = ((h >> 8) & 0xFFFFFF).to(torch.float32) * (1.0 / 16777216.0)    # [0, 1)
    z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
    return z.to(torch.bfloat16).view(torch.int16)


# ----------------------------------------------------------------------------
# length mixes
# ----------------------------------------------------------------------------

def _rng(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return g


def lengths_short_chat(batch: int, seed: int) -> List[int]:
    """prompt ~ lognormal(median 180, sigma 0.5) + generated ~ U{1..400}."""
    g = _rng(seed)
    prompt = torch.exp(math.log(180.0) + 0.5 * torch.randn(batch, generator=g, dtype=torch.float64))
    gen = torch.randint(1, 401, (batch,), generator=g)
    return [max(1, int(round(float(p))) + int(x)) for p, x in zip(prompt, gen)]


def lengths_shared_prefix(batch: int, seed: int, prefix: int = 1536, lo: int = 16, hi: int = 256) -> List[int]:
    """common prefix + per-sequence suffix ~ U{lo..hi}."""
    g = _rng(seed)
    suf = torch.randint(lo, hi + 1, (batch,), generator=g)
    return [prefix + int(x) for x in suf]


# ----------------------------------------------------------------------------
# a paged workload
# ----------------------------------------------------------------------------

@dataclass
class PagedWorkload:
    """Everything one decode-attention call reads, as raw tensors.

    q_bits        int16 [B, Hq, D]                   bf16 bit patterns
    k_pool/v_pool int16 [num_pages, P, Hkv, D] (token-major) or
                        [num_pages, Hkv, P, D] (head-major)
    block_table   int32 [B, max_pages_per_seq]
    seq_lens      int32 [B]
    strides are in elements: (page, token, head).
    """
    name: str
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    num_pages: int
    max_pages_per_seq: int
    seq_lens: torch.Tensor
    block_table: torch.Tensor
    q_bits: torch.Tensor
    k_pool: torch.Tensor
    v_pool: torch.Tensor
    layout: str = "token_major"
    seq_uids: List[int] = field(default_factory=list)
    shared_prefix_tokens: int = 0
    unique_tokens: int = 0
    dtype: str = "bf16"          # what the 16-bit patterns of q, k_pool and v_pool are: "bf16" or "fp16"

    @property
    def strides(self):
        P, H, D = self.page_size, self.num_kv_heads, self.head_dim
        if self.layout == "token_major":
            return (P * H * D, H * D, D)
        return (H * P * D, D, P * D)

    @property
    def logical_tokens(self) -> int:
        return int(self.seq_lens.sum().item())

    @property
    def kv_bytes_per_token(self) -> int:
        """K and V rows of every KV head in bf16: the per-token, per-layer byte
        count `b` of the paper's decode rule (Appendix D)."""
        return self.num_kv_heads * self.head_dim * 2 * 2

    @property
    def logical_kv_bytes(self) -> int:
        return self.logical_tokens * self.kv_bytes_per_token

    @property
    def unique_kv_bytes(self) -> int:
        return self.unique_tokens * self.kv_bytes_per_token


def kv_bytes_per_token(num_kv_heads: int, head_dim: int, bytes_per_elem: int = 2) -> int:
    return num_kv_heads * head_dim * 2 * bytes_per_elem


def _pages_of(length: int, page_size: int) -> int:
    return (length + page_size - 1) // page_size


def _fill_pages(pool: torch.Tensor, layout: str, page_ids: torch.Tensor, key: int,
                tok_begin: int, tok_end: int, P: int, H: int, D: int,
                chunk_tokens: int = 1 << 16) -> None:
    """Write logical tokens [tok_begin, tok_end) of stream `key` into the pages
    `page_ids` (page j holds tokens tok_begin + j*P ...).  tok_begin is the
    stream offset of the first token of page_ids[0]; slots past tok_end in the
    last page are left as they are."""
    dev = pool.device
    n_tok = tok_end - tok_begin
    done = 0
    while done < n_tok:
        n = min(chunk_tokens - chunk_tokens % P, n_tok - done)
        bits = normal_bf16_bits(key, (tok_begin + done) * H * D, n * H * D, dev).view(n, H, D)
        first_page = done // P
        full = n // P
        if full:
            blk = bits[: full * P].view(full, P, H, D)
            ids = page_ids[first_page: first_page + full].to(torch.int64)
            if layout == "token_major":
                pool[ids] = blk
            else:
                pool[ids] = blk.permute(0, 2, 1, 3)
        rem = n - full * P
        if rem:
            pid = int(page_ids[first_page + full])
            tail = bits[full * P:]
            if layout == "token_major":
                pool[pid, :rem] = tail
            else:
                pool[pid, :, :rem] = tail.permute(1, 0, 2)
        done += n


def make_workload(name: str, seq_lens: Sequence[int], num_q_heads: int, num_kv_heads: int,
                  head_dim: int, seed: int, page_size: int = 16, pool_pages: Optional[int] = None,
                  layout: str = "token_major", device="cpu", seq_uids: Optional[Sequence[int]] = None,
                  shared_prefix_tokens: int = 0, shuffle_pages: bool = True,
                  unused_fill_bits: int = 0x7FC0, max_pages_per_seq: Optional[int] = None,
                  alias_after: Optional[int] = None, table_seed: Optional[int] = None,
                  dtype: str = "bf16") -> PagedWorkload:
    """Build pools, block table and q for the given lengths.

    * `dtype` "fp16": the same values (and the same poison in unused slots) stored as fp16 bit
      patterns instead of bf16 (each bf16 sample converted, round to nearest);

    * physical pages: a seeded random permutation of the pool's page ids dealt
      to the sequences in order (prefix pages first when a prefix is shared);
    * `shared_prefix_tokens` > 0 (a multiple of the page size): the first
      tokens of every sequence are one common stream whose physical pages
      appear in every block-table row;
    * `unused_fill_bits`: bf16 bit pattern written everywhere first (default a
      quiet NaN), so slots past a sequence's end and unreferenced pages poison
      any result that touches them;
    * `alias_after` = K: sequences i >= K reuse the pages (and content) of
      sequence i mod K (for cells whose KV would not fit in memory);
    * `seq_uids`: content identity of each sequence (default: its index).
    """
    P, H, D = page_size, num_kv_heads, head_dim
    B = len(seq_lens)
    assert shared_prefix_tokens % P == 0
    uids = list(seq_uids) if seq_uids is not None else list(range(B))
    n_own = B if alias_after is None else min(B, alias_after)
    prefix_pages = shared_prefix_tokens // P
    need = prefix_pages
    for i in range(n_own):
        assert seq_lens[i] >= shared_prefix_tokens
        need += _pages_of(seq_lens[i], P) - prefix_pages
    num_pages = max(need, pool_pages or 0, 1)
    g = _rng((seed if table_seed is None else table_seed) * 7919 + 17)
    perm = torch.randperm(num_pages, generator=g) if shuffle_pages else torch.arange(num_pages)
    perm = perm.to(torch.int32)
    mpp = max([_pages_of(l, P) for l in seq_lens] + [1])
    if max_pages_per_seq is not None:
        assert max_pages_per_seq >= mpp
        mpp = max_pages_per_seq
    block_table = torch.full((B, mpp), -1, dtype=torch.int32)

    shape = (num_pages, P, H, D) if layout == "token_major" else (num_pages, H, P, D)
    fill = unused_fill_bits - (1 << 16) if unused_fill_bits >= (1 << 15) else unused_fill_bits
    k_pool = torch.full(shape, fill, dtype=torch.int16, device=device)
    v_pool = torch.full(shape, fill, dtype=torch.int16, device=device)

    cur = 0
    prefix_ids = perm[cur: cur + prefix_pages]
    cur += prefix_pages
    if prefix_pages:
        pk = stream_key(seed, TENSOR_K, 1_000_003)
        pv = stream_key(seed, TENSOR_V, 1_000_003)
        dev_ids = prefix_ids.to(device)
        _fill_pages(k_pool, layout, dev_ids, pk, 0, shared_prefix_tokens, P, H, D)
        _fill_pages(v_pool, layout, dev_ids, pv, 0, shared_prefix_tokens, P, H, D)
    unique_tokens = shared_prefix_tokens
    for i in range(B):
        L = int(seq_lens[i])
        npg = _pages_of(L, P)
        if i >= n_own:
            src = i % n_own
            assert seq_lens[src] == L
            block_table[i, :npg] = block_table[src, :npg]
            continue
        own = npg - prefix_pages
        ids = perm[cur: cur + own]
        cur += own
        block_table[i, :prefix_pages] = prefix_ids
        block_table[i, prefix_pages:npg] = ids
        if own:
            dev_ids = ids.to(device)
            _fill_pages(k_pool, layout, dev_ids, stream_key(seed, TENSOR_K, uids[i]),
                        shared_prefix_tokens, L, P, H, D)
            _fill_pages(v_pool, layout, dev_ids, stream_key(seed, TENSOR_V, uids[i]),
                        shared_prefix_tokens, L, P, H, D)
        unique_tokens += L - shared_prefix_tokens

    q = torch.empty((B, num_q_heads, D), dtype=torch.int16, device=device)
    for i in range(B):
        src_uid = uids[i if i < n_own else i % n_own]
        q[i] = normal_bf16_bits(stream_key(seed, TENSOR_Q, src_uid), 0, num_q_heads * D, device).view(num_q_heads, D)

    assert dtype in ("bf16", "fp16")
    if dtype == "fp16":
        as_fp16 = lambda t: t.view(torch.bfloat16).to(torch.float16).view(torch.int16)
        q, k_pool, v_pool = as_fp16(q), as_fp16(k_pool), as_fp16(v_pool)
    return PagedWorkload(
        name=name, batch=B, num_q_heads=num_q_heads, num_kv_heads=H, head_dim=D, page_size=P,
        num_pages=num_pages, max_pages_per_seq=mpp,
        seq_lens=torch.tensor(list(seq_lens), dtype=torch.int32).to(device),
        block_table=block_table.to(device), q_bits=q, k_pool=k_pool, v_pool=v_pool, layout=layout,
        seq_uids=uids, shared_prefix_tokens=shared_prefix_tokens, unique_tokens=unique_tokens, dtype=dtype)


# ----------------------------------------------------------------------------
# the five named configurations
# ----------------------------------------------------------------------------

def config_tiny(device="cpu", layout="token_major") -> PagedWorkload:
    """Batch 4, 8 query / 2 KV heads, head_dim 64, lengths {17, 64, 129, 300},
    34 pages dealt from a shuffled pool of 64, seed 0."""
    return make_workload("tiny", [17, 64, 129, 300], 8, 2, 64, seed=0, pool_pages=64,
                         layout=layout, device=device)


def config_long(device="cpu", context: int = 32768, layout="token_major", seed: int = 1,
                table_seed: Optional[int] = None, page_size: int = 16) -> PagedWorkload:
    """One sequence of `context` tokens, 32 query / 8 KV heads, head_dim 128."""
    return make_workload("long", [context], 32, 8, 128, seed=seed, layout=layout, device=device,
                         table_seed=table_seed, page_size=page_size)


def config_short_chat(device="cpu", batch: int = 64, layout="token_major", seed: int = 2,
                      table_seed: Optional[int] = None, page_size: int = 16) -> PagedWorkload:
    return make_workload("short_chat", lengths_short_chat(batch, seed), 32, 8, 128, seed=seed,
                         layout=layout, device=device, table_seed=table_seed, page_size=page_size)


def config_shared_prefix(device="cpu", batch: int = 256, layout="token_major", seed: int = 3,
                         prefix: int = 1536, table_seed: Optional[int] = None,
                         page_size: int = 16) -> PagedWorkload:
    return make_workload("shared_prefix", lengths_shared_prefix(batch, seed, prefix), 32, 8, 128,
                         seed=seed, layout=layout, device=device, shared_prefix_tokens=prefix,
                         table_seed=table_seed, page_size=page_size)


def config_sweep_cell(context: int, batch: int, device="cpu", layout="token_major", seed: int = 4,
                      alias_after: Optional[int] = None, table_seed: Optional[int] = None,
                      page_size: int = 16, num_q_heads: int = 32) -> PagedWorkload:
    """One cell of the length x batch sweep: `batch` sequences of `context`
    tokens; sequence i has the same content in every batch size."""
    return make_workload(f"sweep_{context}x{batch}", [context] * batch, num_q_heads, 8, 128, seed=seed,
                         layout=layout, device=device, alias_after=alias_after, table_seed=table_seed,
                         page_size=page_size)


def as_fp16(w: PagedWorkload) -> PagedWorkload:
    """The same workload with q, K and V stored as fp16 bit patterns (what `dtype="fp16"` of
    make_workload gives)."""
    if w.dtype == "fp16":
        return w
    cv = lambda t: t.view(torch.bfloat16).to(torch.float16).view(torch.int16)
    return dataclasses.replace(w, q_bits=cv(w.q_bits), k_pool=cv(w.k_pool), v_pool=cv(w.v_pool), dtype="fp16")


def permute_pages(w: PagedWorkload, seed: int) -> PagedWorkload:
    """The same logical workload with its physical pages moved: page p goes to
    sigma(p) in both pools and the block table is rewritten accordingly."""
    g = _rng(seed)
    sigma = torch.randperm(w.num_pages, generator=g)
    dev = w.k_pool.device
    inv_src = torch.empty_like(sigma)
    inv_src[sigma] = torch.arange(w.num_pages)
    k2 = w.k_pool[inv_src.to(dev)]
    v2 = w.v_pool[inv_src.to(dev)]
    bt = w.block_table.cpu().to(torch.int64)
    bt2 = torch.where(bt >= 0, sigma[bt.clamp(min=0)], bt).to(torch.int32)
    import dataclasses
    return dataclasses.replace(w, k_pool=k2, v_pool=v2, block_table=bt2.to(w.block_table.device))
