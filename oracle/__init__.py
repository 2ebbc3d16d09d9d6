"""ctypes front end of the fp64 CPU oracle (TEST INFRASTRUCTURE ONLY).

Only `tests/`, the smoke check and the bench's CPU-baseline leg may import this
package.  The CUDA library and its Python binding never do, and this package
imports nothing from them.  `build()` compiles `fastkv_oracle.c` with gcc.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

POOL_AVG, POOL_MAX = 0, 1
GROUP_THEN_POOL, POOL_THEN_GROUP = 0, 1

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "fastkv_oracle.c")
_LIB = os.path.join(_DIR, "libfastkv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (fp64, -O2, OpenMP) if the library is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i64, i32, f64 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_double
        lib.oracle_window_attention.argtypes = [vp, i64, vp, i64, i32, i32, i32, i32, f64, vp]
        lib.oracle_full_attention_window.argtypes = [vp, vp, i64, i32, i32, i32, i32, f64, vp, vp]
        lib.oracle_pool1d.argtypes = [vp, i64, i64, i32, i32, vp]
        lib.oracle_scores.argtypes = [vp, i64, vp, i64, i32, i32, i32, i32, f64, i32, i32, i32,
                                      vp, vp, vp]
        lib.oracle_select.argtypes = [vp, i64, i64, i32, i32, vp, vp]
        lib.oracle_gather_rows.argtypes = [vp, i64, i64, vp, i64, vp]
        lib.oracle_decode_attention.argtypes = [vp, vp, vp, i64, i32, i32, i32, f64, vp, vp]
        lib.oracle_prefill_attention.argtypes = [vp, vp, vp, i64, i32, i32, i32, f64, vp]
        lib.oracle_num_threads.restype = i32
        _lib = lib
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a: np.ndarray) -> np.ndarray:
    assert a.dtype == np.uint16, "bf16 tensors are passed as uint16 bit patterns"
    return np.ascontiguousarray(a)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def window_attention(q: np.ndarray, q_first_pos: int, k: np.ndarray, w: int,
                     scale: Optional[float] = None) -> np.ndarray:
    """A[h, i] = sum over the w window rows of the causal softmax attention (Eq. 1, inner term)."""
    q, k = _u16(q), _u16(k)
    L, Hkv, d = k.shape
    H = q.shape[1]
    A = np.empty((H, L), dtype=np.float64)
    rc = _load().oracle_window_attention(_ptr(q), q_first_pos, _ptr(k), L, H, Hkv, d, w,
                                         (d ** -0.5) if scale is None else scale, _ptr(A))
    if rc:
        raise ValueError("oracle_window_attention rejected its arguments")
    return A


def full_attention_window(q_full: np.ndarray, k: np.ndarray, w: int, scale: Optional[float] = None,
                          want_matrix: bool = False) -> Tuple[np.ndarray, Optional[np.ndarray]]:
    q_full, k = _u16(q_full), _u16(k)
    L, Hkv, d = k.shape
    H = q_full.shape[1]
    A = np.empty((H, L), dtype=np.float64)
    att = np.empty((H, L, L), dtype=np.float64) if want_matrix else None
    rc = _load().oracle_full_attention_window(_ptr(q_full), _ptr(k), L, H, Hkv, d, w,
                                              (d ** -0.5) if scale is None else scale, _ptr(A),
                                              _ptr(att))
    if rc:
        raise ValueError("oracle_full_attention_window rejected its arguments")
    return A, att


def pool1d(x: np.ndarray, p: int, mode: int) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    x2 = x.reshape(-1, x.shape[-1])
    out = np.empty_like(x2)
    if _load().oracle_pool1d(_ptr(x2), x2.shape[0], x2.shape[1], p, mode, _ptr(out)):
        raise ValueError("oracle_pool1d rejected its arguments")
    return out.reshape(x.shape)


def scores(q: np.ndarray, q_first_pos: int, k: np.ndarray, w: int, pool_kernel: int,
           pool_mode: int = POOL_AVG, agg_order: int = GROUP_THEN_POOL,
           scale: Optional[float] = None, want_A: bool = False):
    """(S_kv [Hkv, L], S_tsp [L], A [H, L] or None) for one sequence of one layer."""
    q, k = _u16(q), _u16(k)
    L, Hkv, d = k.shape
    H = q.shape[1]
    S_kv = np.empty((Hkv, L), dtype=np.float64)
    S_tsp = np.empty((L,), dtype=np.float64)
    A = np.empty((H, L), dtype=np.float64) if want_A else None
    rc = _load().oracle_scores(_ptr(q), q_first_pos, _ptr(k), L, H, Hkv, d, w,
                               (d ** -0.5) if scale is None else scale, pool_kernel, pool_mode,
                               agg_order, _ptr(S_kv), _ptr(S_tsp), _ptr(A))
    if rc:
        raise ValueError("oracle_scores rejected its arguments")
    return S_kv, S_tsp, A


def select(S: np.ndarray, k: int, w: int, force_window: bool = True) -> Tuple[np.ndarray, float]:
    """Ascending indices of the k kept positions and tau, the score of the last ranked one kept."""
    S = np.ascontiguousarray(S, dtype=np.float64)
    idx = np.empty((k,), dtype=np.int64)
    tau = ctypes.c_double(0.0)
    rc = _load().oracle_select(_ptr(S), S.shape[0], k, w, int(force_window), _ptr(idx),
                               ctypes.cast(ctypes.byref(tau), ctypes.c_void_p))
    if rc:
        raise ValueError("oracle_select rejected its arguments")
    return idx, float(tau.value)


def gather_rows(src: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """dst[j] = src[idx[j]] as a byte copy; src is [rows, ...] with dense trailing dims."""
    assert src.strides[1:] == np.empty(src.shape[1:], src.dtype).strides, "trailing dims must be dense"
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    row_bytes = int(np.prod(src.shape[1:], dtype=np.int64)) * src.itemsize
    dst = np.empty((idx.shape[0],) + src.shape[1:], dtype=src.dtype)
    _load().oracle_gather_rows(_ptr(src), src.strides[0], row_bytes, _ptr(idx), idx.shape[0],
                               _ptr(dst))
    return dst


def decode_attention(q: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray, scale: Optional[float] = None):
    """One query token over a compressed cache: q [H, d], k_cache / v_cache [Hkv, k, d] (bf16 bits).
    Returns (out [H, d] fp64, lse [H] fp64)."""
    q, k_cache, v_cache = _u16(q), _u16(k_cache), _u16(v_cache)
    H, d = q.shape
    Hkv, k, _ = k_cache.shape
    out = np.empty((H, d), dtype=np.float64)
    lse = np.empty((H,), dtype=np.float64)
    rc = _load().oracle_decode_attention(_ptr(q), _ptr(k_cache), _ptr(v_cache), k, H, Hkv, d,
                                         (d ** -0.5) if scale is None else scale, _ptr(out), _ptr(lse))
    if rc:
        raise ValueError("oracle_decode_attention rejected its arguments")
    return out, lse


def prefill_attention(q_full: np.ndarray, k: np.ndarray, v: np.ndarray, scale: Optional[float] = None) -> np.ndarray:
    """Causal softmax attention of a whole prompt (the layer's own attention, Alg. 1): q_full [L, H, d],
    k / v [L, Hkv, d] (bf16 bits).  Returns O [L, H, d] fp64."""
    q_full, k, v = _u16(q_full), _u16(k), _u16(v)
    L, H, d = q_full.shape
    Hkv = k.shape[1]
    out = np.empty((L, H, d), dtype=np.float64)
    rc = _load().oracle_prefill_attention(_ptr(q_full), _ptr(k), _ptr(v), L, H, Hkv, d,
                                          (d ** -0.5) if scale is None else scale, _ptr(out))
    if rc:
        raise ValueError("oracle_prefill_attention rejected its arguments")
    return out
