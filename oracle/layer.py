"""One FastKV layer step on a packed (possibly ragged) batch, composed from the oracle's
routines in the order of Algorithm 1: scores -> KVCompress -> HiddenCompress -> update.

TEST INFRASTRUCTURE ONLY (see the package docstring).
"""
from __future__ import annotations

from typing import Dict, Optional, Sequence

import numpy as np

from . import GROUP_THEN_POOL, POOL_AVG, gather_rows, scores, select


def layer_step(q_win: np.ndarray, k: np.ndarray, v: Optional[np.ndarray],
               hidden: Optional[np.ndarray], pos: Optional[np.ndarray], cu_seqlens: np.ndarray,
               w: int, pool_kernel: int, k_kv: Sequence[int], k_tsp: Optional[Sequence[int]],
               pool_mode: int = POOL_AVG, agg_order: int = GROUP_THEN_POOL,
               force_window: bool = True, scale: Optional[float] = None,
               do_compact: bool = True) -> Dict[str, np.ndarray]:
    """q_win is [B*w, H, d] (last w query rows of each sequence); k, v are [total, Hkv, d];
    hidden is [total, hidden_dim]; pos is [total].  Index outputs are sequence-local."""
    B = len(cu_seqlens) - 1
    total, Hkv, d = k.shape
    S_kv = np.empty((Hkv, total), dtype=np.float64)
    S_tsp = np.empty((total,), dtype=np.float64)
    cu_k_kv = np.concatenate([[0], np.cumsum(k_kv)]).astype(np.int64)
    idx_kv = np.empty((Hkv, cu_k_kv[-1]), dtype=np.int64)
    tau_kv = np.empty((B, Hkv), dtype=np.float64)
    out: Dict[str, np.ndarray] = {}
    if k_tsp is not None:
        cu_k_tsp = np.concatenate([[0], np.cumsum(k_tsp)]).astype(np.int64)
        idx_tsp = np.empty((cu_k_tsp[-1],), dtype=np.int64)
        tau_tsp = np.empty((B,), dtype=np.float64)
    for b in range(B):
        lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        L = hi - lo
        s_kv, s_tsp, _ = scores(q_win[b * w:(b + 1) * w], L - w, k[lo:hi], w, pool_kernel,
                                pool_mode, agg_order, scale)
        S_kv[:, lo:hi] = s_kv
        S_tsp[lo:hi] = s_tsp
        for g in range(Hkv):                                    # KVCompress, per KV group
            idx, tau = select(s_kv[g], int(k_kv[b]), w, force_window)
            idx_kv[g, cu_k_kv[b]:cu_k_kv[b + 1]] = idx
            tau_kv[b, g] = tau
        if k_tsp is not None:                                   # HiddenCompress, once per layer
            idx, tau = select(s_tsp, int(k_tsp[b]), w, force_window)
            idx_tsp[cu_k_tsp[b]:cu_k_tsp[b + 1]] = idx
            tau_tsp[b] = tau
    out.update(S_kv=S_kv, S_tsp=S_tsp, idx_kv=idx_kv, tau_kv=tau_kv, cu_k_kv=cu_k_kv)
    if k_tsp is not None:
        out.update(idx_tsp=idx_tsp, tau_tsp=tau_tsp, cu_k_tsp=cu_k_tsp)
    if do_compact:
        k_out = np.empty((Hkv, cu_k_kv[-1], d), dtype=k.dtype)
        v_out = np.empty_like(k_out) if v is not None else None
        for b in range(B):
            lo = int(cu_seqlens[b])
            for g in range(Hkv):
                rows = lo + idx_kv[g, cu_k_kv[b]:cu_k_kv[b + 1]]
                k_out[g, cu_k_kv[b]:cu_k_kv[b + 1]] = gather_rows(k[:, g, :], rows)
                if v is not None:
                    v_out[g, cu_k_kv[b]:cu_k_kv[b + 1]] = gather_rows(v[:, g, :], rows)
        out.update(k_out=k_out)
        if v is not None:
            out.update(v_out=v_out)
        if k_tsp is not None:
            rows = np.concatenate([int(cu_seqlens[b]) + idx_tsp[cu_k_tsp[b]:cu_k_tsp[b + 1]]
                                   for b in range(B)])
            if hidden is not None:
                out.update(hidden_out=gather_rows(hidden, rows))
            if pos is not None:
                out.update(pos_out=gather_rows(pos, rows))
    return out
