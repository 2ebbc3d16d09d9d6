"""Thin ctypes binding of libfastkv_b200.so: argument marshalling only.

Function names mirror the C ABI (include/fastkv.h).  Tensors are torch CUDA tensors used purely
as device memory; every step of the path runs inside the library's kernels.  There is no CPU or
PyTorch fallback: if the library is missing or fails to load, importing the symbols raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

FASTKV_OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_DEVICE_INDEX = range(1, 7)
POOL_AVG, POOL_MAX = 0, 1
GROUP_THEN_POOL, POOL_THEN_GROUP = 0, 1
Q_FULL, Q_WINDOW = 0, 1

EXPORTS = ["fastkv_workspace_bytes", "fastkv_score", "fastkv_select_kv", "fastkv_select_tsp", "fastkv_select",
           "fastkv_compact", "fastkv_decode_attn_workspace_bytes", "fastkv_decode_attn", "fastkv_prefill_workspace_bytes",
           "fastkv_prefill_attention", "fastkv_device_status", "fastkv_layer_host_arena_bytes",
           "fastkv_layer_host", "fastkv_score_static", "fastkv_score_static_status", "fastkv_debug_set",
           "fastkv_debug_kernel_time",
           "fastkv_status_string", "fastkv_last_error", "fastkv_kernel_launches"]
_INT_RETURNING = [n for n in EXPORTS if n not in ("fastkv_status_string", "fastkv_last_error",
                                                  "fastkv_kernel_launches")]


class FastKVError(RuntimeError):
    def __init__(self, status: int, where: str):
        lib = _load()
        text = lib.fastkv_status_string(status).decode()
        detail = lib.fastkv_last_error().decode()
        super().__init__("%s: %s (%d)%s" % (where, text, status, ": " + detail if detail else ""))
        self.status = status


class Shape(ctypes.Structure):
    """fastkv_shape"""
    _fields_ = [("batch", ctypes.c_int32), ("total_len", ctypes.c_int32), ("max_len", ctypes.c_int32),
                ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("hidden_dim", ctypes.c_int32), ("window", ctypes.c_int32), ("pool_kernel", ctypes.c_int32),
                ("pool_mode", ctypes.c_int32), ("agg_order", ctypes.c_int32), ("force_window", ctypes.c_int32),
                ("q_layout", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
                ("cu_seqlens", ctypes.c_void_p),
                ("q_stride_tok", ctypes.c_int64), ("q_stride_head", ctypes.c_int64),
                ("k_stride_tok", ctypes.c_int64), ("k_stride_head", ctypes.c_int64),
                ("v_stride_tok", ctypes.c_int64), ("v_stride_head", ctypes.c_int64),
                ("hidden_stride_tok", ctypes.c_int64)]


class Budget(ctypes.Structure):
    """fastkv_budget"""
    _fields_ = [("k", ctypes.c_int32), ("total", ctypes.c_int32), ("cu_k", ctypes.c_void_p)]


_lib = None


def _load():
    global _lib
    if _lib is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            raise RuntimeError("libfastkv_b200.so is not built; run `python -m paper_2502_01068_b200.build` "
                               "(there is no fallback path)")
        lib = ctypes.CDLL(path)
        vp, sz = ctypes.c_void_p, ctypes.c_size_t
        ps, pb = ctypes.POINTER(Shape), ctypes.POINTER(Budget)
        lib.fastkv_workspace_bytes.argtypes = [ps, ctypes.POINTER(sz)]
        lib.fastkv_score.argtypes = [ps, vp, vp, vp, vp, vp, sz, vp]
        lib.fastkv_select_kv.argtypes = [ps, vp, pb, vp, vp, sz, vp]
        lib.fastkv_select_tsp.argtypes = [ps, vp, pb, vp, vp, sz, vp]
        lib.fastkv_select.argtypes = [ps, vp, pb, vp, vp, pb, vp, vp, sz, vp]
        lib.fastkv_compact.argtypes = [ps, vp, pb, vp, pb, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.fastkv_device_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
        lib.fastkv_layer_host_arena_bytes.argtypes = [ps, ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(sz)]
        lib.fastkv_layer_host.argtypes = [ps, ctypes.c_int32, ctypes.c_int32] + [vp] * 12 + [sz, vp]
        lib.fastkv_status_string.argtypes = [ctypes.c_int]
        lib.fastkv_status_string.restype = ctypes.c_char_p
        lib.fastkv_last_error.restype = ctypes.c_char_p
        lib.fastkv_kernel_launches.restype = ctypes.c_int64
        lib.fastkv_score_static.argtypes = [ps, vp, vp, vp, vp, vp]
        lib.fastkv_decode_attn_workspace_bytes.argtypes = [ps, ctypes.POINTER(sz)]
        lib.fastkv_decode_attn.argtypes = [ps, vp, vp, vp, pb, vp, vp, vp, sz, vp]
        lib.fastkv_prefill_workspace_bytes.argtypes = [ps, ctypes.POINTER(sz)]
        lib.fastkv_prefill_attention.argtypes = [ps, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.fastkv_score_static_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
        lib.fastkv_debug_set.argtypes = [ctypes.c_char_p, ctypes.c_int64]
        lib.fastkv_debug_kernel_time.argtypes = [ctypes.c_int32, ctypes.POINTER(ctypes.c_double),
                                                 ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_char_p)]
        for fn in _INT_RETURNING:
            getattr(lib, fn).restype = ctypes.c_int
        _lib = lib
    return _lib


def library_path() -> str:
    return _build.LIB_PATH


def _p(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    return t.ctypes.data          # numpy array (host entry points)


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


def _check(rc: int, where: str) -> None:
    if rc != FASTKV_OK:
        raise FastKVError(rc, where)


def make_shape(*, total_len: int, n_q_heads: int, n_kv_heads: int, head_dim: int, hidden_dim: int = 0,
               window: int = 8, pool_kernel: int = 7, pool_mode: int = POOL_AVG,
               agg_order: int = GROUP_THEN_POOL, force_window: bool = True, q_layout: int = Q_WINDOW,
               softmax_scale: float = 0.0, batch: int = 1, max_len: Optional[int] = None,
               cu_seqlens=None, q_stride_tok: Optional[int] = None, q_stride_head: Optional[int] = None,
               k_stride_tok: Optional[int] = None, k_stride_head: Optional[int] = None,
               v_stride_tok: Optional[int] = None, v_stride_head: Optional[int] = None,
               hidden_stride_tok: Optional[int] = None) -> Shape:
    """Fill a fastkv_shape; strides default to dense [tokens, heads, head_dim] tensors."""
    s = Shape()
    s.batch, s.total_len, s.max_len = batch, total_len, total_len if max_len is None else max_len
    s.n_q_heads, s.n_kv_heads, s.head_dim, s.hidden_dim = n_q_heads, n_kv_heads, head_dim, hidden_dim
    s.window, s.pool_kernel, s.pool_mode, s.agg_order = window, pool_kernel, pool_mode, agg_order
    s.force_window, s.q_layout, s.softmax_scale = int(force_window), q_layout, softmax_scale
    s.cu_seqlens = _p(cu_seqlens)
    s._keep_alive = cu_seqlens          # the struct only holds the address: the tensor must outlive it
    s.q_stride_head = head_dim if q_stride_head is None else q_stride_head
    s.q_stride_tok = n_q_heads * head_dim if q_stride_tok is None else q_stride_tok
    s.k_stride_head = head_dim if k_stride_head is None else k_stride_head
    s.k_stride_tok = n_kv_heads * head_dim if k_stride_tok is None else k_stride_tok
    s.v_stride_head = head_dim if v_stride_head is None else v_stride_head
    s.v_stride_tok = n_kv_heads * head_dim if v_stride_tok is None else v_stride_tok
    s.hidden_stride_tok = hidden_dim if hidden_stride_tok is None else hidden_stride_tok
    return s


def make_budget(k: int = 0, *, batch: int = 1, cu_k=None, total: Optional[int] = None) -> Budget:
    b = Budget()
    b.k = k
    b.cu_k = _p(cu_k)
    b._keep_alive = cu_k                # the struct only holds the address: the tensor must outlive it
    b.total = (k * batch) if total is None else total
    return b


def fastkv_workspace_bytes(shape: Shape) -> int:
    n = ctypes.c_size_t(0)
    _check(_load().fastkv_workspace_bytes(ctypes.byref(shape), ctypes.byref(n)), "fastkv_workspace_bytes")
    return int(n.value)


def fastkv_score(shape: Shape, q, k, scores_kv, scores_tsp, workspace, stream=None) -> None:
    _check(_load().fastkv_score(ctypes.byref(shape), _p(q), _p(k), _p(scores_kv), _p(scores_tsp), _p(workspace),
                                workspace.numel() * workspace.element_size(), _stream(stream)), "fastkv_score")


def fastkv_select_kv(shape: Shape, scores_kv, budget: Budget, idx_kv, workspace, stream=None) -> None:
    _check(_load().fastkv_select_kv(ctypes.byref(shape), _p(scores_kv), ctypes.byref(budget), _p(idx_kv),
                                    _p(workspace), workspace.numel() * workspace.element_size(),
                                    _stream(stream)), "fastkv_select_kv")


def fastkv_select_tsp(shape: Shape, scores_tsp, budget: Budget, idx_tsp, workspace, stream=None) -> None:
    _check(_load().fastkv_select_tsp(ctypes.byref(shape), _p(scores_tsp), ctypes.byref(budget), _p(idx_tsp),
                                     _p(workspace), workspace.numel() * workspace.element_size(),
                                     _stream(stream)), "fastkv_select_tsp")


def fastkv_select(shape: Shape, scores_kv, kv: Budget, idx_kv, scores_tsp, tsp: Budget, idx_tsp, workspace,
                  stream=None) -> None:
    _check(_load().fastkv_select(ctypes.byref(shape), _p(scores_kv), ctypes.byref(kv), _p(idx_kv), _p(scores_tsp),
                                 ctypes.byref(tsp), _p(idx_tsp), _p(workspace),
                                 workspace.numel() * workspace.element_size(), _stream(stream)), "fastkv_select")


def fastkv_compact(shape: Shape, idx_kv, kv: Optional[Budget], idx_tsp, tsp: Optional[Budget], k, v, hidden,
                   pos_ids, k_out, v_out, hidden_out, pos_out, workspace, stream=None) -> None:
    _check(_load().fastkv_compact(ctypes.byref(shape), _p(idx_kv), ctypes.byref(kv) if kv else None,
                                  _p(idx_tsp), ctypes.byref(tsp) if tsp else None, _p(k), _p(v), _p(hidden),
                                  _p(pos_ids), _p(k_out), _p(v_out), _p(hidden_out), _p(pos_out),
                                  _p(workspace), workspace.numel() * workspace.element_size(),
                                  _stream(stream)), "fastkv_compact")


def fastkv_decode_attn_workspace_bytes(shape: Shape) -> int:
    n = ctypes.c_size_t(0)
    _check(_load().fastkv_decode_attn_workspace_bytes(ctypes.byref(shape), ctypes.byref(n)),
           "fastkv_decode_attn_workspace_bytes")
    return int(n.value)


def fastkv_decode_attn(shape: Shape, q, k_cache, v_cache, kv: Budget, out, lse, workspace, stream=None) -> None:
    _check(_load().fastkv_decode_attn(ctypes.byref(shape), _p(q), _p(k_cache), _p(v_cache), ctypes.byref(kv), _p(out),
                                      _p(lse), _p(workspace), workspace.numel() * workspace.element_size(),
                                      _stream(stream)), "fastkv_decode_attn")


def fastkv_prefill_workspace_bytes(shape: Shape) -> int:
    n = ctypes.c_size_t(0)
    _check(_load().fastkv_prefill_workspace_bytes(ctypes.byref(shape), ctypes.byref(n)), "fastkv_prefill_workspace_bytes")
    return int(n.value)


def fastkv_prefill_attention(shape: Shape, q, k, v, out, scores_kv, scores_tsp, workspace, stream=None) -> None:
    _check(_load().fastkv_prefill_attention(ctypes.byref(shape), _p(q), _p(k), _p(v), _p(out), _p(scores_kv),
                                            _p(scores_tsp), _p(workspace), workspace.numel() * workspace.element_size(),
                                            _stream(stream)), "fastkv_prefill_attention")


def fastkv_device_status(workspace, stream=None):
    status, site = ctypes.c_int32(0), ctypes.c_int32(0)
    _check(_load().fastkv_device_status(_p(workspace), _stream(stream), ctypes.byref(status),
                                        ctypes.byref(site)), "fastkv_device_status")
    return int(status.value), int(site.value)


def fastkv_layer_host_arena_bytes(shape: Shape, k_kv: int, k_tsp: int) -> int:
    n = ctypes.c_size_t(0)
    _check(_load().fastkv_layer_host_arena_bytes(ctypes.byref(shape), k_kv, k_tsp, ctypes.byref(n)),
           "fastkv_layer_host_arena_bytes")
    return int(n.value)


def fastkv_layer_host(shape: Shape, k_kv: int, k_tsp: int, q, k, v, hidden, pos_ids, idx_kv, idx_tsp, k_out,
                      v_out, hidden_out, pos_out, arena, stream=None) -> None:
    """Host-buffer layer step: q..pos_out are host tensors/arrays, `arena` is a device tensor."""
    _check(_load().fastkv_layer_host(ctypes.byref(shape), k_kv, k_tsp, _p(q), _p(k), _p(v), _p(hidden),
                                     _p(pos_ids), _p(idx_kv), _p(idx_tsp), _p(k_out), _p(v_out),
                                     _p(hidden_out), _p(pos_out), _p(arena),
                                     arena.numel() * arena.element_size(), _stream(stream)),
           "fastkv_layer_host")


def fastkv_score_static(shape: Shape, q, k, scores_kv, scores_tsp, stream=None) -> None:
    """fastkv_score without a workspace argument: the scratch is a fixed 16 MiB array inside the
    library, for callers that cannot allocate device memory.  Shapes that need more raise
    FastKVError(ERR_WORKSPACE).  Calls on one device share the array: do not overlap them.
    fastkv_score_static_status() reads the device status word the call left behind."""
    _check(_load().fastkv_score_static(ctypes.byref(shape), _p(q), _p(k), _p(scores_kv), _p(scores_tsp),
                                       _stream(stream)), "fastkv_score_static")


def fastkv_score_static_status(stream=None):
    """(status, site) left by the last fastkv_score_static call on the current device."""
    status, site = ctypes.c_int32(0), ctypes.c_int32(0)
    _check(_load().fastkv_score_static_status(_stream(stream), ctypes.byref(status), ctypes.byref(site)),
           "fastkv_score_static_status")
    return int(status.value), int(site.value)


def fastkv_debug_set(key: str, value: int) -> None:
    """Test and tuning hooks of the library (process-wide); see include/fastkv.h for the keys."""
    _check(_load().fastkv_debug_set(key.encode(), int(value)), "fastkv_debug_set")


def fastkv_debug_kernel_time(kernel: int):
    """(name, total milliseconds, launches) recorded for one kernel class while the "time_kernels" hook was on."""
    ms, n, name = ctypes.c_double(0.0), ctypes.c_int64(0), ctypes.c_char_p()
    _check(_load().fastkv_debug_kernel_time(kernel, ctypes.byref(ms), ctypes.byref(n), ctypes.byref(name)),
           "fastkv_debug_kernel_time")
    return name.value.decode(), float(ms.value), int(n.value)


def fastkv_status_string(status: int) -> str:
    return _load().fastkv_status_string(status).decode()


def fastkv_last_error() -> str:
    return _load().fastkv_last_error().decode()


def fastkv_kernel_launches() -> int:
    return int(_load().fastkv_kernel_launches())
