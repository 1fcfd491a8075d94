"""ctypes front end of the fp64 CPU oracle (test infrastructure only).

Only tests/, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It builds `paged_attention_oracle.c` with gcc on first use and
never touches the CUDA library; inputs are numpy / CPU torch arrays of bf16
(or, with in_fp16, fp16) bit patterns (uint16 / int16).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "paged_attention_oracle.c")
_LIB = os.path.join(_HERE, "libpaged_attention_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared library beside its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Shape(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
                ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("page_size", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32),
                ("k_stride_page", ctypes.c_int64), ("k_stride_token", ctypes.c_int64),
                ("k_stride_head", ctypes.c_int64), ("v_stride_page", ctypes.c_int64),
                ("v_stride_token", ctypes.c_int64), ("v_stride_head", ctypes.c_int64),
                ("in_fp16", ctypes.c_int32), ("pad", ctypes.c_int32)]


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_max_threads.restype = ctypes.c_int
    return _lib


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def _u16(a) -> np.ndarray:
    if hasattr(a, "detach"):
        a = a.detach().cpu().numpy()
    a = np.ascontiguousarray(a)
    assert a.dtype in (np.uint16, np.int16), a.dtype
    return a.view(np.uint16)


def _i32(a) -> np.ndarray:
    if hasattr(a, "detach"):
        a = a.detach().cpu().numpy()
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


class PagedInputs:
    """Host copies of one call's inputs, in the oracle's terms."""

    def __init__(self, q_bits, k_pool, v_pool, block_table, seq_lens, page_size: int,
                 strides: Tuple[int, int, int], num_kv_heads: int, v_strides=None, in_fp16: bool = False):
        self.q = _u16(q_bits)
        self.k = _u16(k_pool)
        self.v = _u16(v_pool)
        self.block_table = _i32(block_table)
        self.seq_lens = _i32(seq_lens)
        B, Hq, D = self.q.shape
        vs = v_strides or strides
        self.shape = _Shape(B, Hq, num_kv_heads, D, page_size, self.block_table.shape[1],
                            strides[0], strides[1], strides[2], vs[0], vs[1], vs[2], 1 if in_fp16 else 0, 0)
        self.B, self.Hq, self.Hkv, self.D, self.P = B, Hq, num_kv_heads, D, page_size

    @classmethod
    def from_workload(cls, w) -> "PagedInputs":
        return cls(w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, w.page_size, w.strides,
                   w.num_kv_heads, in_fp16=getattr(w, "dtype", "bf16") == "fp16")


def decode_bits(bits, in_fp16: bool) -> np.ndarray:
    """The oracle's reading of 16-bit input patterns, as fp64."""
    lib = _load()
    b = np.ascontiguousarray(np.asarray(bits).view(np.uint16)).ravel()
    out = np.empty(b.shape, dtype=np.float64)
    lib.oracle_decode_bits(ctypes.c_int(1 if in_fp16 else 0), _p(b), ctypes.c_int64(b.size), _p(out))
    return out


def default_scale(head_dim: int) -> float:
    """1/sqrt(D) evaluated in fp32 and promoted, the value a caller passing
    sm_scale = 0 gets."""
    return float(np.float32(1.0) / np.sqrt(np.float32(head_dim)))


def paged_decode_attention(inp: PagedInputs, scale: Optional[float] = None, run_mask=None,
                           num_threads: int = 0):
    """out [B,Hq,D] fp64 and lse [B,Hq] fp64."""
    lib = _load()
    scale = default_scale(inp.D) if scale is None else float(scale)
    out = np.empty((inp.B, inp.Hq, inp.D), dtype=np.float64)
    lse = np.empty((inp.B, inp.Hq), dtype=np.float64)
    mask = None
    if run_mask is not None:
        mask = np.ascontiguousarray(np.asarray(run_mask), dtype=np.uint8)
        assert mask.shape == (inp.B,)
    rc = lib.oracle_paged_decode_attention(ctypes.byref(inp.shape), _p(inp.q), _p(inp.k), _p(inp.v),
                                           _p(inp.block_table), _p(inp.seq_lens), _p(mask),
                                           ctypes.c_double(scale), _p(out), _p(lse),
                                           ctypes.c_int(num_threads))
    assert rc == 0
    return out, lse


def partial_attention(inp: PagedInputs, b: int, h: int, t_begin: int, t_end: int,
                      scale: Optional[float] = None):
    """(o [D] normalised, m, l) of tokens [t_begin, t_end) for one (b, h)."""
    lib = _load()
    scale = default_scale(inp.D) if scale is None else float(scale)
    o = np.empty(inp.D, dtype=np.float64)
    m = ctypes.c_double()
    l = ctypes.c_double()
    lib.oracle_partial_attention(ctypes.byref(inp.shape), _p(inp.q), _p(inp.k), _p(inp.v),
                                 _p(inp.block_table), ctypes.c_double(scale), b, h, t_begin, t_end,
                                 _p(o), ctypes.byref(m), ctypes.byref(l))
    return o, m.value, l.value


def attention_probs(inp: PagedInputs, b: int, h: int, scale: Optional[float] = None) -> np.ndarray:
    lib = _load()
    scale = default_scale(inp.D) if scale is None else float(scale)
    probs = np.empty(int(inp.seq_lens[b]), dtype=np.float64)
    lib.oracle_attention_probs(ctypes.byref(inp.shape), _p(inp.q), _p(inp.k), _p(inp.v),
                               _p(inp.block_table), _p(inp.seq_lens), ctypes.c_double(scale), b, h,
                               _p(probs))
    return probs


def merge_partials(o_parts, m_parts, l_parts):
    """LSE merge of partial results, ascending order: (out [D], lse)."""
    lib = _load()
    o_parts = np.ascontiguousarray(o_parts, dtype=np.float64)
    m_parts = np.ascontiguousarray(m_parts, dtype=np.float64)
    l_parts = np.ascontiguousarray(l_parts, dtype=np.float64)
    n, D = o_parts.shape
    out = np.empty(D, dtype=np.float64)
    lse = ctypes.c_double()
    lib.oracle_merge_partials(n, D, _p(o_parts), _p(m_parts), _p(l_parts), _p(out), ctypes.byref(lse))
    return out, lse.value


def gather_kv(inp: PagedInputs, b: int):
    """Logical K and V rows of sequence b as uint16 [L, Hkv, D]."""
    lib = _load()
    L = int(inp.seq_lens[b])
    k = np.empty((L, inp.Hkv, inp.D), dtype=np.uint16)
    v = np.empty((L, inp.Hkv, inp.D), dtype=np.uint16)
    lib.oracle_gather_kv(ctypes.byref(inp.shape), _p(inp.k), _p(inp.v), _p(inp.block_table),
                         _p(inp.seq_lens), b, _p(k), _p(v))
    return k, v


def append_kv(inp: PagedInputs, new_k, new_v):
    """Own-layer KV write: returns copies of the pools with every row's new K/V
    stored at logical position seq_len - 1 (Invariant 1)."""
    lib = _load()
    nk, nv = _u16(new_k), _u16(new_v)
    assert nk.shape == (inp.B, inp.Hkv, inp.D) and nv.shape == nk.shape
    k, v = inp.k.copy(), inp.v.copy()
    lib.oracle_append_kv(ctypes.byref(inp.shape), _p(nk), _p(nv), _p(inp.block_table), _p(inp.seq_lens), _p(k), _p(v))
    return k, v
