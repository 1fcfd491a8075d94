"""ctypes binding of libdecode_attn.so: the same entry points as
include/decode_attn.h, with argument marshalling only.

Tensors are torch tensors used for their device memory (`data_ptr()`); the
stream is `torch.cuda.current_stream().cuda_stream` unless one is given.
Every step of the path runs in the library's kernels.  If the library has not
been built, importing this module raises - there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# DECODE_ATTN_LIB: another build of the same library (a trace build, a variant under measurement)
LIB_PATH = os.environ.get("DECODE_ATTN_LIB") or os.path.join(_HERE, "libdecode_attn.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2609_37062_b200.build` "
        "(there is no CPU or eager fallback for the decode-attention path)")

_lib = ctypes.CDLL(LIB_PATH)

DA_OK = 0
DA_ERR_INVALID_ARG = -1
DA_ERR_UNSUPPORTED = -2
DA_ERR_WORKSPACE_TOO_SMALL = -3
DA_ERR_STALE_PLAN = -4
DA_ERR_CUDA = -5
DA_ERR_BAD_PAGE = -6
DA_ERR_TIMEOUT = -7

DA_DTYPE_BF16 = 1
DA_DTYPE_FP32 = 2
DA_DTYPE_FP16 = 3

DA_SPLIT_AUTO = 0
DA_SPLIT_FIXED_COUNT = 1
DA_SPLIT_DETERMINISTIC = 2

DA_KERNEL_AUTO = 0
DA_KERNEL_SIMT = 1
DA_KERNEL_MMA_TMA = 2
DA_KERNEL_UMMA_PREFIX = 3

EXPORTED = [
    "decode_attn_plan_layout", "decode_attn_plan", "decode_attn_plan_update", "decode_attn_plan_get_info",
    "decode_attn_plan_get_units", "decode_attn_plan_check", "decode_attn_plan_destroy", "decode_attn_run",
    "decode_attn_run_ex", "decode_attn_combine", "decode_attn_last_device_status",
    "decode_attn_validate_block_table", "decode_attn_debug_gather", "decode_attn_gather_probe",
    "decode_attn_host_step", "decode_attn_host_release", "decode_attn_strerror", "decode_attn_version",
    "decode_attn_step_static", "decode_attn_append_kv", "decode_attn_breakeven_tokens",
    "decode_attn_switch_thresholds", "decode_attn_switch_next", "decode_attn_validate_shared_prefix",
    "decode_attn_merge_shards", "decode_attn_append_kv_checked", "decode_attn_debug_expire_wait",
]


class Policy(ctypes.Structure):
    _fields_ = [("split_mode", ctypes.c_int32), ("fixed_count", ctypes.c_int32),
                ("chunk_tokens", ctypes.c_int32), ("max_splits", ctypes.c_int32),
                ("sm_count", ctypes.c_int32), ("kernel", ctypes.c_int32),
                ("fuse_combine", ctypes.c_int32), ("capacity_batch", ctypes.c_int32),
                ("capacity_tokens", ctypes.c_int32), ("ctas_per_sm", ctypes.c_int32),
                ("shared_prefix_tokens", ctypes.c_int32), ("reserved", ctypes.c_int32 * 5)]


class Shape(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
                ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("page_size", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32),
                ("num_pages", ctypes.c_int64),
                ("k_stride_page", ctypes.c_int64), ("k_stride_token", ctypes.c_int64),
                ("k_stride_head", ctypes.c_int64), ("v_stride_page", ctypes.c_int64),
                ("v_stride_token", ctypes.c_int64), ("v_stride_head", ctypes.c_int64),
                ("kv_dtype", ctypes.c_int32), ("q_dtype", ctypes.c_int32),
                ("out_dtype", ctypes.c_int32), ("sm_scale", ctypes.c_float)]


class Unit(ctypes.Structure):
    _fields_ = [("seq", ctypes.c_int32), ("kv_head", ctypes.c_int32), ("tok_begin", ctypes.c_int32),
                ("tok_end", ctypes.c_int32), ("slot", ctypes.c_int32), ("seq_len", ctypes.c_int32),
                ("split_index", ctypes.c_int32), ("n_splits", ctypes.c_int32)]


class PlanInfo(ctypes.Structure):
    _fields_ = [("n_units", ctypes.c_int64), ("grid", ctypes.c_int64), ("n_slots", ctypes.c_int64),
                ("workspace_bytes", ctypes.c_int64), ("chunk_tokens", ctypes.c_int32),
                ("kernel", ctypes.c_int32), ("ctas_per_sm", ctypes.c_int32), ("sm_count", ctypes.c_int32),
                ("fuse_combine", ctypes.c_int32), ("max_splits_used", ctypes.c_int32),
                ("block_threads", ctypes.c_int32), ("dynamic_smem_bytes", ctypes.c_int32)]


class RunArgs(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("flags", ctypes.c_uint32),
                ("q", ctypes.c_void_p), ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
                ("block_table", ctypes.c_void_p), ("seq_lens", ctypes.c_void_p),
                ("run_mask", ctypes.c_void_p), ("out", ctypes.c_void_p), ("lse", ctypes.c_void_p),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
                ("new_k", ctypes.c_void_p), ("new_v", ctypes.c_void_p)]


_vp = ctypes.c_void_p
_lib.decode_attn_plan_layout.argtypes = [ctypes.POINTER(Shape), ctypes.POINTER(Policy), _vp, ctypes.c_int32,
                                         ctypes.c_int32, _vp, ctypes.c_int64, ctypes.POINTER(ctypes.c_int64),
                                         _vp, _vp, ctypes.POINTER(ctypes.c_int64),
                                         ctypes.POINTER(ctypes.c_int32)]
_lib.decode_attn_plan.argtypes = [ctypes.POINTER(Shape), ctypes.POINTER(Policy), _vp, ctypes.POINTER(_vp),
                                  ctypes.POINTER(ctypes.c_size_t)]
_lib.decode_attn_plan_update.argtypes = [_vp, ctypes.c_int32, _vp, _vp]
_lib.decode_attn_plan_get_info.argtypes = [_vp, ctypes.POINTER(PlanInfo)]
_lib.decode_attn_plan_get_units.argtypes = [_vp, _vp, ctypes.c_int64]
_lib.decode_attn_plan_check.argtypes = [_vp, ctypes.c_int32, _vp]
_lib.decode_attn_plan_destroy.argtypes = [_vp]
_lib.decode_attn_run.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, ctypes.c_size_t, _vp]
_lib.decode_attn_run_ex.argtypes = [_vp, ctypes.POINTER(RunArgs), _vp]
_lib.decode_attn_combine.argtypes = [_vp, _vp, _vp, _vp, _vp]
_lib.decode_attn_last_device_status.argtypes = [_vp, _vp]
_lib.decode_attn_validate_block_table.argtypes = [ctypes.POINTER(Shape), _vp, _vp]
_lib.decode_attn_validate_shared_prefix.argtypes = [ctypes.POINTER(Shape), ctypes.c_int32, _vp, _vp]
_lib.decode_attn_debug_gather.argtypes = [_vp, ctypes.c_int32, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.decode_attn_gather_probe.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp]
_lib.decode_attn_host_step.argtypes = [ctypes.POINTER(Shape), ctypes.POINTER(Policy), _vp, _vp, _vp,
                                       ctypes.c_int64, _vp, _vp, _vp, _vp]
_lib.decode_attn_host_release.argtypes = []
_lib.decode_attn_step_static.argtypes = [ctypes.POINTER(Shape), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.decode_attn_append_kv.argtypes = [ctypes.POINTER(Shape), _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.decode_attn_append_kv_checked.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.decode_attn_debug_expire_wait.argtypes = [_vp, ctypes.POINTER(RunArgs), ctypes.c_int64, _vp]
_lib.decode_attn_merge_shards.argtypes = [ctypes.POINTER(Shape), ctypes.c_int32, _vp, _vp, _vp, _vp, _vp]
_lib.decode_attn_breakeven_tokens.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_int32,
                                              ctypes.c_double, ctypes.POINTER(ctypes.c_double)]
_lib.decode_attn_switch_thresholds.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.POINTER(ctypes.c_double),
                                               ctypes.POINTER(ctypes.c_double)]
_lib.decode_attn_switch_next.argtypes = [ctypes.c_int32, ctypes.c_double, ctypes.c_double, ctypes.c_double]
_lib.decode_attn_strerror.argtypes = [ctypes.c_int]
_lib.decode_attn_strerror.restype = ctypes.c_char_p
_lib.decode_attn_version.restype = ctypes.c_char_p


class DecodeAttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {decode_attn_strerror(status)} ({status})")


def decode_attn_strerror(status: int) -> str:
    return _lib.decode_attn_strerror(int(status)).decode()


def decode_attn_version() -> str:
    return _lib.decode_attn_version().decode()


def _check(status: int, where: str) -> None:
    if status != DA_OK:
        raise DecodeAttnError(status, where)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _host_i32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    return np.ascontiguousarray(np.asarray(x), dtype=np.int32)


def make_policy(split_mode: int = DA_SPLIT_AUTO, fixed_count: int = 0, chunk_tokens: int = 0,
                max_splits: int = 0, sm_count: int = 0, kernel: int = DA_KERNEL_AUTO, fuse_combine: int = 0,
                capacity_batch: int = 0, capacity_tokens: int = 0, ctas_per_sm: int = 0,
                shared_prefix_tokens: int = 0) -> Policy:
    p = Policy()
    p.split_mode, p.fixed_count, p.chunk_tokens, p.max_splits = split_mode, fixed_count, chunk_tokens, max_splits
    p.sm_count, p.kernel, p.fuse_combine = sm_count, kernel, fuse_combine
    p.capacity_batch, p.capacity_tokens, p.ctas_per_sm = capacity_batch, capacity_tokens, ctas_per_sm
    p.shared_prefix_tokens = shared_prefix_tokens
    return p


def make_shape(batch: int, num_q_heads: int, num_kv_heads: int, head_dim: int, page_size: int,
               max_pages_per_seq: int, num_pages: int, k_strides: Sequence[int],
               v_strides: Optional[Sequence[int]] = None, out_dtype: int = DA_DTYPE_FP32,
               sm_scale: float = 0.0, in_dtype: int = DA_DTYPE_BF16) -> Shape:
    s = Shape()
    s.batch, s.num_q_heads, s.num_kv_heads, s.head_dim = batch, num_q_heads, num_kv_heads, head_dim
    s.page_size, s.max_pages_per_seq, s.num_pages = page_size, max_pages_per_seq, num_pages
    s.k_stride_page, s.k_stride_token, s.k_stride_head = k_strides
    s.v_stride_page, s.v_stride_token, s.v_stride_head = v_strides or k_strides
    s.kv_dtype = s.q_dtype = in_dtype
    s.out_dtype = out_dtype
    s.sm_scale = sm_scale
    return s


def shape_of_workload(w, out_dtype: int = DA_DTYPE_FP32, sm_scale: float = 0.0) -> Shape:
    return make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.page_size, w.max_pages_per_seq,
                      w.num_pages, w.strides, out_dtype=out_dtype, sm_scale=sm_scale,
                      in_dtype=DA_DTYPE_FP16 if getattr(w, "dtype", "bf16") == "fp16" else DA_DTYPE_BF16)


def decode_attn_plan_layout(shape: Shape, policy: Policy, seq_lens, sm_count: int, ctas_per_sm: int):
    """Host-only planner: (units, splits[B], slot_base[B], n_slots, chunk_tokens)."""
    lens = _host_i32(seq_lens)
    n_units = ctypes.c_int64()
    n_slots = ctypes.c_int64()
    chunk = ctypes.c_int32()
    _check(_lib.decode_attn_plan_layout(ctypes.byref(shape), ctypes.byref(policy), _ptr(lens), sm_count,
                                        ctas_per_sm, None, 0, ctypes.byref(n_units), None, None,
                                        ctypes.byref(n_slots), ctypes.byref(chunk)), "decode_attn_plan_layout")
    units = (Unit * max(1, n_units.value))()
    splits = np.zeros(max(1, shape.batch), dtype=np.int32)
    slot_base = np.zeros(max(1, shape.batch), dtype=np.int32)
    _check(_lib.decode_attn_plan_layout(ctypes.byref(shape), ctypes.byref(policy), _ptr(lens), sm_count,
                                        ctas_per_sm, ctypes.addressof(units), n_units.value,
                                        ctypes.byref(n_units), _ptr(splits), _ptr(slot_base),
                                        ctypes.byref(n_slots), ctypes.byref(chunk)), "decode_attn_plan_layout")
    return ([units[i] for i in range(n_units.value)], splits[:shape.batch], slot_base[:shape.batch],
            n_slots.value, chunk.value)


class Plan:
    """Owner of one decode_attn_plan_t."""

    def __init__(self, handle: int, workspace_bytes: int, shape: Shape, policy: Policy):
        self.handle = handle
        self.workspace_bytes = workspace_bytes
        self.shape = shape
        self.policy = policy

    def info(self) -> PlanInfo:
        return decode_attn_plan_get_info(self)

    def destroy(self) -> None:
        if self.handle:
            _lib.decode_attn_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def decode_attn_plan(shape: Shape, policy: Policy, seq_lens_host) -> Plan:
    lens = _host_i32(seq_lens_host)
    handle = _vp()
    ws = ctypes.c_size_t()
    _check(_lib.decode_attn_plan(ctypes.byref(shape), ctypes.byref(policy), _ptr(lens), ctypes.byref(handle),
                                 ctypes.byref(ws)), "decode_attn_plan")
    return Plan(handle.value, ws.value, shape, policy)


def decode_attn_plan_update(plan: Plan, seq_lens_host, stream=None) -> None:
    lens = _host_i32(seq_lens_host)
    _check(_lib.decode_attn_plan_update(plan.handle, len(lens), _ptr(lens), _stream(stream)),
           "decode_attn_plan_update")
    plan.shape.batch = len(lens)


def decode_attn_plan_get_info(plan: Plan) -> PlanInfo:
    info = PlanInfo()
    _check(_lib.decode_attn_plan_get_info(plan.handle, ctypes.byref(info)), "decode_attn_plan_get_info")
    return info


def decode_attn_plan_get_units(plan: Plan):
    n = decode_attn_plan_get_info(plan).n_units
    units = (Unit * max(1, n))()
    _check(_lib.decode_attn_plan_get_units(plan.handle, ctypes.addressof(units), n), "decode_attn_plan_get_units")
    return [units[i] for i in range(n)]


def decode_attn_plan_check(plan: Plan, seq_lens_host) -> int:
    lens = _host_i32(seq_lens_host)
    return _lib.decode_attn_plan_check(plan.handle, len(lens), _ptr(lens))


def decode_attn_plan_destroy(plan: Plan) -> None:
    plan.destroy()


def decode_attn_run(plan: Plan, q, k_cache, v_cache, block_table, seq_lens, out, lse=None, workspace=None,
                    workspace_bytes: Optional[int] = None, stream=None, run_mask=None, check: bool = True,
                    new_k=None, new_v=None) -> int:
    """new_k / new_v: the rows' new K and V, written at position seq_len - 1 and attended in the same launch."""
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    if run_mask is None and new_k is None and new_v is None:
        rc = _lib.decode_attn_run(plan.handle, _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_table),
                                  _ptr(seq_lens), _ptr(out), _ptr(lse), _ptr(workspace), workspace_bytes,
                                  _stream(stream))
    else:
        a = RunArgs()
        a.struct_size = ctypes.sizeof(RunArgs)
        a.q, a.k_cache, a.v_cache = _ptr(q), _ptr(k_cache), _ptr(v_cache)
        a.block_table, a.seq_lens, a.run_mask = _ptr(block_table), _ptr(seq_lens), _ptr(run_mask)
        a.out, a.lse, a.workspace, a.workspace_bytes = _ptr(out), _ptr(lse), _ptr(workspace), workspace_bytes
        a.new_k, a.new_v = _ptr(new_k), _ptr(new_v)
        rc = _lib.decode_attn_run_ex(plan.handle, ctypes.byref(a), _stream(stream))
    if check:
        _check(rc, "decode_attn_run")
    return rc


def decode_attn_combine(plan: Plan, workspace, out, lse=None, stream=None, check: bool = True) -> int:
    rc = _lib.decode_attn_combine(plan.handle, _ptr(workspace), _ptr(out), _ptr(lse), _stream(stream))
    if check:
        _check(rc, "decode_attn_combine")
    return rc


def decode_attn_last_device_status(plan: Optional[Plan], stream=None) -> int:
    """plan None: the status word of decode_attn_step_static on the current device."""
    return _lib.decode_attn_last_device_status(plan.handle if plan is not None else None, _stream(stream))


def decode_attn_debug_expire_wait(plan: Plan, q, k_cache, v_cache, block_table, seq_lens, out, lse=None,
                                  workspace=None, workspace_bytes: Optional[int] = None, limit_cycles: int = 2_000_000,
                                  stream=None) -> int:
    """Test hook: the plan's partial kernel with its loads withheld and its waits cut to limit_cycles."""
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    a = RunArgs()
    a.struct_size = ctypes.sizeof(RunArgs)
    a.q, a.k_cache, a.v_cache = _ptr(q), _ptr(k_cache), _ptr(v_cache)
    a.block_table, a.seq_lens = _ptr(block_table), _ptr(seq_lens)
    a.out, a.lse, a.workspace, a.workspace_bytes = _ptr(out), _ptr(lse), _ptr(workspace), workspace_bytes
    return _lib.decode_attn_debug_expire_wait(plan.handle, ctypes.byref(a), int(limit_cycles), _stream(stream))


def decode_attn_validate_block_table(shape: Shape, seq_lens_host, block_table_host) -> int:
    lens = _host_i32(seq_lens_host)
    bt = _host_i32(block_table_host)
    return _lib.decode_attn_validate_block_table(ctypes.byref(shape), _ptr(lens), _ptr(bt))


def decode_attn_validate_shared_prefix(shape: Shape, shared_prefix_tokens: int, seq_lens_host, block_table_host) -> int:
    lens = _host_i32(seq_lens_host)
    bt = _host_i32(block_table_host)
    return _lib.decode_attn_validate_shared_prefix(ctypes.byref(shape), shared_prefix_tokens, _ptr(lens), _ptr(bt))


def decode_attn_debug_gather(plan: Plan, seq: int, k_cache, v_cache, block_table, k_out, v_out, stream=None) -> None:
    _check(_lib.decode_attn_debug_gather(plan.handle, seq, _ptr(k_cache), _ptr(v_cache), _ptr(block_table),
                                         _ptr(k_out), _ptr(v_out), _stream(stream)), "decode_attn_debug_gather")


def decode_attn_gather_probe(plan: Plan, k_cache, v_cache, block_table, checksum_out, stream=None) -> None:
    _check(_lib.decode_attn_gather_probe(plan.handle, _ptr(k_cache), _ptr(v_cache), _ptr(block_table),
                                         _ptr(checksum_out), _stream(stream)), "decode_attn_gather_probe")


def decode_attn_host_step(shape: Shape, policy: Policy, q_host, k_cache_host, v_cache_host, block_table_host,
                          seq_lens_host, out_host, lse_host=None) -> None:
    """Whole step from host tensors (CPU torch tensors or numpy arrays)."""
    pool_elems = k_cache_host.numel() if hasattr(k_cache_host, "numel") else k_cache_host.size
    _check(_lib.decode_attn_host_step(ctypes.byref(shape), ctypes.byref(policy), _ptr(q_host), _ptr(k_cache_host),
                                      _ptr(v_cache_host), pool_elems, _ptr(block_table_host), _ptr(seq_lens_host),
                                      _ptr(out_host), _ptr(lse_host)), "decode_attn_host_step")


def decode_attn_step_static(shape: Shape, seq_lens_host, q, k_cache, v_cache, block_table, seq_lens, out, lse=None,
                            stream=None, check: bool = True) -> int:
    """One whole step (partial + combine) that allocates nothing: for callers that cannot
    call the CUDA allocator.  Scratch is an 8 MiB array built into the library."""
    lens = _host_i32(seq_lens_host)
    rc = _lib.decode_attn_step_static(ctypes.byref(shape), _ptr(lens), _ptr(q), _ptr(k_cache), _ptr(v_cache),
                                      _ptr(block_table), _ptr(seq_lens), _ptr(out), _ptr(lse), _stream(stream))
    if check:
        _check(rc, "decode_attn_step_static")
    return rc


def decode_attn_append_kv(shape: Shape, new_k, new_v, block_table, seq_lens, k_cache, v_cache, stream=None,
                          check: bool = True) -> int:
    rc = _lib.decode_attn_append_kv(ctypes.byref(shape), _ptr(new_k), _ptr(new_v), _ptr(block_table), _ptr(seq_lens),
                                    _ptr(k_cache), _ptr(v_cache), _stream(stream))
    if check:
        _check(rc, "decode_attn_append_kv")
    return rc


def decode_attn_append_kv_checked(plan: Plan, new_k, new_v, block_table, seq_lens, k_cache, v_cache, stream=None,
                                  check: bool = True) -> int:
    rc = _lib.decode_attn_append_kv_checked(plan.handle, _ptr(new_k), _ptr(new_v), _ptr(block_table), _ptr(seq_lens),
                                            _ptr(k_cache), _ptr(v_cache), _stream(stream))
    if check:
        _check(rc, "decode_attn_append_kv_checked")
    return rc


def decode_attn_merge_shards(shape: Shape, n_shards: int, out_shards, lse_shards, out, lse=None, stream=None,
                             check: bool = True) -> int:
    rc = _lib.decode_attn_merge_shards(ctypes.byref(shape), int(n_shards), _ptr(out_shards), _ptr(lse_shards), _ptr(out),
                                       _ptr(lse), _stream(stream))
    if check:
        _check(rc, "decode_attn_merge_shards")
    return rc


def decode_attn_breakeven_tokens(tau_seconds: float, bandwidth_bytes_per_s: float, skip_fraction: float,
                                 routed_layers: int, kv_bytes_per_token_layer: float) -> float:
    v = ctypes.c_double()
    _check(_lib.decode_attn_breakeven_tokens(tau_seconds, bandwidth_bytes_per_s, skip_fraction, routed_layers,
                                             kv_bytes_per_token_layer, ctypes.byref(v)), "decode_attn_breakeven_tokens")
    return v.value


def decode_attn_switch_thresholds(v_star: float, round_to: float = 10_000.0):
    ex, en = ctypes.c_double(), ctypes.c_double()
    _check(_lib.decode_attn_switch_thresholds(v_star, round_to, ctypes.byref(ex), ctypes.byref(en)),
           "decode_attn_switch_thresholds")
    return ex.value, en.value


def decode_attn_switch_next(routed_now: bool, resident_tokens: float, exit_tokens: float, enter_tokens: float) -> bool:
    return bool(_lib.decode_attn_switch_next(int(bool(routed_now)), resident_tokens, exit_tokens, enter_tokens))


def decode_attn_host_release() -> None:
    _lib.decode_attn_host_release()


# ----------------------------------------------------------------------------
# convenience for tests, smoke and bench: one call over a device workload
# ----------------------------------------------------------------------------

def run_workload(w, policy: Optional[Policy] = None, out_dtype: int = DA_DTYPE_FP32, sm_scale: float = 0.0,
                 run_mask=None, want_lse: bool = True, return_plan: bool = False):
    """plan -> run -> (combine) on tensors that already live on the GPU.
    Returns (out, lse) as torch tensors; raises on any host or device status."""
    import torch
    policy = policy or make_policy()
    shape = shape_of_workload(w, out_dtype=out_dtype, sm_scale=sm_scale)
    plan = decode_attn_plan(shape, policy, w.seq_lens)
    dev = w.k_pool.device
    odt = {DA_DTYPE_FP32: torch.float32, DA_DTYPE_BF16: torch.bfloat16, DA_DTYPE_FP16: torch.float16}[out_dtype]
    out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=odt, device=dev)
    lse = torch.full((w.batch, w.num_q_heads), float("nan"), dtype=torch.float32, device=dev) if want_lse else None
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device=dev)
    decode_attn_run(plan, w.q_bits, w.k_pool, w.v_pool, w.block_table, w.seq_lens, out, lse, ws,
                    plan.workspace_bytes, run_mask=run_mask)
    if not policy.fuse_combine:
        decode_attn_combine(plan, ws, out, lse)
    st = decode_attn_last_device_status(plan)
    if st != DA_OK:
        plan.destroy()
        raise DecodeAttnError(st, "device status")
    if return_plan:
        return out, lse, plan
    plan.destroy()
    return out, lse
