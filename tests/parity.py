"""Test-side glue: run one layer through the C ABI on the GPU, run the oracle on the same bytes,
and apply the acceptance rules (scores within 2e-3 relative; index sets identical except at
boundary ties within 1e-6 relative of the threshold score; gathered rows bit-exact)."""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

from oracle.layer import layer_step
from paper_2502_01068_b200 import binding as B
from paper_2502_01068_b200 import workloads as W

SCORE_RTOL = 2e-3          # bf16 inputs, fp32 accumulation
SCORE_ATOL = 1e-12
TIE_RTOL = 1e-6            # a differing index must sit this close (relative) to the threshold


def dev(a: Optional[np.ndarray]):
    if a is None:
        return None
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda()
    return torch.from_numpy(a).cuda()


def host(t: torch.Tensor, dtype) -> np.ndarray:
    return t.cpu().numpy().view(dtype)


def gpu_layer(wl: W.Workload, x: W.LayerInputs, *, pool_mode=None, agg_order=B.GROUP_THEN_POOL,
              force_window=True, ragged_api=None, keep_device=False, fused_select=True,
              q_layout=B.Q_WINDOW) -> Dict[str, np.ndarray]:
    """score -> select_kv -> select_tsp -> compact through the binding.  `ragged_api` forces the
    cu_seqlens / cu_k form of the interface even for a single sequence; `q_layout` = Q_FULL hands the
    library the whole packed query tensor and lets it find the window rows itself."""
    lens = np.diff(x.cu_seqlens).tolist()
    Bn = len(lens)
    ragged = (Bn > 1) if ragged_api is None else ragged_api
    total = int(x.cu_seqlens[-1])
    d_cu = dev(x.cu_seqlens.astype(np.int32)) if ragged else None
    shape = B.make_shape(total_len=total, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
                         head_dim=wl.head_dim, hidden_dim=wl.hidden_dim, window=wl.window,
                         pool_kernel=wl.pool_kernel, pool_mode=wl.pool_mode if pool_mode is None else pool_mode,
                         agg_order=agg_order, force_window=force_window, q_layout=q_layout,
                         batch=Bn, max_len=max(lens), cu_seqlens=d_cu)
    q = dev(x.q_win if q_layout == B.Q_WINDOW else W.full_q(wl, x))
    k, v, hid, pos = dev(x.k), dev(x.v), dev(x.hidden), dev(x.pos)
    ws = torch.empty(B.fastkv_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    s_kv = torch.empty((wl.n_kv_heads, total), dtype=torch.float32, device="cuda")
    s_tsp = torch.empty((total,), dtype=torch.float32, device="cuda") if wl.k_tsp is not None else None
    B.fastkv_score(shape, q, k, s_kv, s_tsp, ws)
    uniform_kv = len(set(wl.k_kv)) == 1 and not (ragged_api and Bn == 1 and False)
    out: Dict[str, np.ndarray] = {}

    def budget(ks):
        if len(set(ks)) == 1 and ragged_api is not True:
            return B.make_budget(int(ks[0]), batch=Bn), None
        cu_k = np.concatenate([[0], np.cumsum(ks)]).astype(np.int32)
        d = dev(cu_k)
        return B.make_budget(0, cu_k=d, total=int(cu_k[-1])), d

    b_kv, keep1 = budget(wl.k_kv)
    idx_kv = torch.full((wl.n_kv_heads, b_kv.total), -1, dtype=torch.int32, device="cuda")
    b_tsp = idx_tsp = keep2 = None
    if wl.k_tsp is not None:
        b_tsp, keep2 = budget(wl.k_tsp)
        idx_tsp = torch.full((b_tsp.total,), -1, dtype=torch.int32, device="cuda")
    if fused_select and wl.k_tsp is not None:
        B.fastkv_select(shape, s_kv, b_kv, idx_kv, s_tsp, b_tsp, idx_tsp, ws)
    else:
        B.fastkv_select_kv(shape, s_kv, b_kv, idx_kv, ws)
        if wl.k_tsp is not None:
            B.fastkv_select_tsp(shape, s_tsp, b_tsp, idx_tsp, ws)
    k_out = torch.zeros((wl.n_kv_heads, b_kv.total, wl.head_dim), dtype=torch.int16, device="cuda")
    v_out = torch.zeros_like(k_out) if v is not None else None
    hid_out = pos_out = None
    if idx_tsp is not None and hid is not None:
        hid_out = torch.zeros((b_tsp.total, wl.hidden_dim), dtype=torch.int16, device="cuda")
    if idx_tsp is not None and pos is not None:
        pos_out = torch.full((b_tsp.total,), -7, dtype=torch.int32, device="cuda")
    B.fastkv_compact(shape, idx_kv, b_kv, idx_tsp, b_tsp, k, v, hid if hid_out is not None else None,
                     pos if pos_out is not None else None, k_out, v_out, hid_out, pos_out, ws)
    status, site = B.fastkv_device_status(ws)
    out["status"], out["site"] = status, site
    out["S_kv"] = s_kv.cpu().numpy()
    out["idx_kv"] = idx_kv.cpu().numpy()
    out["k_out"] = host(k_out, np.uint16)
    if v_out is not None:
        out["v_out"] = host(v_out, np.uint16)
    if s_tsp is not None:
        out["S_tsp"] = s_tsp.cpu().numpy()
        out["idx_tsp"] = idx_tsp.cpu().numpy()
    if hid_out is not None:
        out["hidden_out"] = host(hid_out, np.uint16)
    if pos_out is not None:
        out["pos_out"] = pos_out.cpu().numpy()
    if keep_device:
        out["_dev"] = dict(k=k, v=v, hidden=hid, pos=pos, idx_kv=idx_kv, idx_tsp=idx_tsp, k_out=k_out,
                           v_out=v_out, hidden_out=hid_out, pos_out=pos_out)
    return out


def host_layer(wl: W.Workload, x: W.LayerInputs, *, pinned=True) -> Dict[str, np.ndarray]:
    """The whole step from HOST buffers through fastkv_layer_host (uniform budgets only): inputs and
    outputs live in host memory, the library copies them through a caller-provided device arena.  For a
    batch, cu_seqlens is handed over as a HOST array, as that entry point specifies."""
    lens = np.diff(x.cu_seqlens).tolist()
    Bn = len(lens)
    total = int(x.cu_seqlens[-1])
    kk = int(wl.k_kv[0])
    kt = int(wl.k_tsp[0]) if wl.k_tsp is not None else 0
    assert len(set(wl.k_kv)) == 1 and (wl.k_tsp is None or len(set(wl.k_tsp)) == 1)
    cu_host = np.ascontiguousarray(x.cu_seqlens, dtype=np.int32)
    shape = B.make_shape(total_len=total, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                         hidden_dim=wl.hidden_dim, window=wl.window, pool_kernel=wl.pool_kernel,
                         pool_mode=wl.pool_mode, batch=Bn, max_len=max(lens),
                         cu_seqlens=cu_host if Bn > 1 else None)

    def hbuf(a):
        t = torch.from_numpy(np.ascontiguousarray(a.view(np.int16) if a.dtype == np.uint16 else a))
        return t.pin_memory() if pinned else t

    def hout(shape_, dtype):
        t = torch.full(shape_, -3, dtype=dtype)
        return t.pin_memory() if pinned else t

    hq, hk, hv = hbuf(x.q_win), hbuf(x.k), hbuf(x.v)
    hh = hbuf(x.hidden) if kt else None
    hp = hbuf(x.pos) if kt else None
    o_idx_kv = hout((wl.n_kv_heads, Bn * kk), torch.int32)
    o_k = hout((wl.n_kv_heads, Bn * kk, wl.head_dim), torch.int16)
    o_v = hout((wl.n_kv_heads, Bn * kk, wl.head_dim), torch.int16)
    o_idx_tsp = hout((Bn * kt,), torch.int32) if kt else None
    o_h = hout((Bn * kt, wl.hidden_dim), torch.int16) if kt else None
    o_p = hout((Bn * kt,), torch.int32) if kt else None
    arena = torch.empty(B.fastkv_layer_host_arena_bytes(shape, kk, kt), dtype=torch.uint8, device="cuda")
    B.fastkv_layer_host(shape, kk, kt, hq, hk, hv, hh, hp, o_idx_kv, o_idx_tsp, o_k, o_v, o_h, o_p, arena)
    out = {"status": 0, "site": 0, "idx_kv": o_idx_kv.numpy().copy(), "k_out": o_k.numpy().view(np.uint16).copy(),
           "v_out": o_v.numpy().view(np.uint16).copy()}
    if kt:
        out.update(idx_tsp=o_idx_tsp.numpy().copy(), hidden_out=o_h.numpy().view(np.uint16).copy(),
                   pos_out=o_p.numpy().copy())
    return out


def oracle_layer(wl: W.Workload, x: W.LayerInputs, *, pool_mode=None, agg_order=0, force_window=True,
                 do_compact=True):
    return layer_step(x.q_win, x.k, x.v, x.hidden, x.pos, x.cu_seqlens, wl.window, wl.pool_kernel,
                      wl.k_kv, wl.k_tsp, pool_mode=wl.pool_mode if pool_mode is None else pool_mode,
                      agg_order=agg_order, force_window=force_window, do_compact=do_compact)


def check_scores(got: np.ndarray, ref: np.ndarray, what: str) -> float:
    err = np.abs(got.astype(np.float64) - ref)
    bound = SCORE_RTOL * np.abs(ref) + SCORE_ATOL
    bad = err > bound
    assert not bad.any(), "%s: %d scores off, worst rel err %.3e" % (
        what, int(bad.sum()), float((err / np.maximum(np.abs(ref), 1e-300)).max()))
    return float((err / np.maximum(np.abs(ref), 1e-30)).max())


def check_index_set(got: np.ndarray, ref: np.ndarray, S_ref: np.ndarray, tau: float, L: int, w: int,
                    force_window: bool, what: str) -> int:
    """Size, order, range, window, and agreement with the oracle up to threshold ties."""
    k = len(ref)
    assert got.shape == (k,), what
    assert np.all(np.diff(got) > 0), what + ": not strictly ascending"
    assert got[0] >= 0 and got[-1] < L, what + ": index out of range"
    if force_window and w:
        assert got[-w:].tolist() == list(range(L - w, L)), what + ": window missing"
    diff = np.setxor1d(got, ref)
    if diff.size:
        gap = np.abs(S_ref[diff] - tau)
        assert np.all(gap <= TIE_RTOL * abs(tau)), "%s: %d indices differ beyond the tie band (worst gap %.3e rel)" % (
            what, diff.size, float(gap.max() / abs(tau)))
    return int(diff.size)


def check_layer(wl: W.Workload, x: W.LayerInputs, g: Dict[str, np.ndarray], o: Dict[str, np.ndarray],
                force_window=True, what="") -> Dict[str, float]:
    """Full acceptance check of one layer; returns a few statistics for reporting."""
    assert g["status"] == 0, "%s: device status %d at site %d" % (what, g["status"], g["site"])
    stats = {"score_err": check_scores(g["S_kv"], o["S_kv"], what + " S_kv") if "S_kv" in g else 0.0, "flips": 0}
    cu = x.cu_seqlens
    w = wl.window
    cu_k = o["cu_k_kv"]
    for b in range(len(cu) - 1):
        lo, hi = int(cu[b]), int(cu[b + 1])
        for h in range(wl.n_kv_heads):
            a, e = int(cu_k[b]), int(cu_k[b + 1])
            stats["flips"] += check_index_set(g["idx_kv"][h, a:e], o["idx_kv"][h, a:e], o["S_kv"][h, lo:hi],
                                              o["tau_kv"][b, h], hi - lo, w, force_window,
                                              "%s idx_kv[b=%d,h=%d]" % (what, b, h))
            rows = lo + g["idx_kv"][h, a:e]
            np.testing.assert_array_equal(g["k_out"][h, a:e], x.k[rows, h], err_msg=what + " k_out")
            if "v_out" in g:
                np.testing.assert_array_equal(g["v_out"][h, a:e], x.v[rows, h], err_msg=what + " v_out")
    if np.array_equal(g["idx_kv"], o["idx_kv"]) and "k_out" in o:
        np.testing.assert_array_equal(g["k_out"], o["k_out"])
        if "v_out" in g:
            np.testing.assert_array_equal(g["v_out"], o["v_out"])
    if "idx_tsp" in o:
        if "S_tsp" in g:
            stats["score_err"] = max(stats["score_err"], check_scores(g["S_tsp"], o["S_tsp"], what + " S_tsp"))
        cu_t = o["cu_k_tsp"]
        for b in range(len(cu) - 1):
            lo, hi = int(cu[b]), int(cu[b + 1])
            a, e = int(cu_t[b]), int(cu_t[b + 1])
            stats["flips"] += check_index_set(g["idx_tsp"][a:e], o["idx_tsp"][a:e], o["S_tsp"][lo:hi],
                                              o["tau_tsp"][b], hi - lo, w, force_window,
                                              "%s idx_tsp[b=%d]" % (what, b))
            rows = lo + g["idx_tsp"][a:e]
            if "hidden_out" in g:
                np.testing.assert_array_equal(g["hidden_out"][a:e], x.hidden[rows], err_msg=what + " hidden_out")
            if "pos_out" in g:
                np.testing.assert_array_equal(g["pos_out"][a:e], x.pos[rows], err_msg=what + " pos_out")
        if np.array_equal(g["idx_tsp"], o["idx_tsp"]):
            if "hidden_out" in g and "hidden_out" in o:
                np.testing.assert_array_equal(g["hidden_out"], o["hidden_out"])
            if "pos_out" in g and "pos_out" in o:
                np.testing.assert_array_equal(g["pos_out"], o["pos_out"])
    return stats
