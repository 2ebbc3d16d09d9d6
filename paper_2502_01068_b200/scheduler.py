"""Batched multi-request scheduling of the selection path.

The method is orthogonal to batching (Sec. 6: it composes with a serving framework's batching): the
score -> select -> compact step of one layer treats every sequence of a packed batch independently.
A server therefore does not run the step once per request; it packs the layers that are ready --
one per waiting request -- into a ragged batch and runs the three calls once.  This module is that
packing: a FIFO queue of per-request layer jobs, a greedy packer under a token budget, the assembly
of the packed tensors (`cu_seqlens`, per-sequence budgets as `cu_k` offsets) and the un-packing of
the results.

The step functions are passed in (`backend`), so the same scheduler drives the CUDA library
(`CudaBatchBackend`) and, in the CPU tests, a stand-in.  The scheduler itself does none of the
method's arithmetic.
"""
from __future__ import annotations

import dataclasses
from collections import deque
from typing import Any, Deque, Dict, List, Optional, Sequence, Tuple

import numpy as np


@dataclasses.dataclass(frozen=True)
class LayerGeometry:
    """What must agree between jobs that share a call: head shape, window, pooling, and whether the
    layer propagates tokens (TSP layer) or only compresses its KV cache."""
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    hidden_dim: int
    window: int
    pool_kernel: int
    pool_mode: int
    with_tsp: bool


@dataclasses.dataclass
class LayerJob:
    """One layer of one request: host arrays (bf16 as uint16 bit patterns), its budgets, and who asked."""
    request_id: Any
    geometry: LayerGeometry
    q_win: np.ndarray               # [w, Hq, d]
    k: np.ndarray                   # [L, Hkv, d]
    v: np.ndarray                   # [L, Hkv, d]
    hidden: Optional[np.ndarray]    # [L, hidden] on TSP layers
    pos: Optional[np.ndarray]       # [L] int32 on TSP layers
    k_kv: int
    k_tsp: int = 0

    @property
    def length(self) -> int:
        return int(self.k.shape[0])


@dataclasses.dataclass
class PackedBatch:
    """A ragged batch ready for one score / select / compact call sequence."""
    geometry: LayerGeometry
    jobs: List[LayerJob]
    q_win: np.ndarray               # [B * w, Hq, d]
    k: np.ndarray                   # [total, Hkv, d]
    v: np.ndarray
    hidden: Optional[np.ndarray]
    pos: Optional[np.ndarray]
    cu_seqlens: np.ndarray          # int32 [B + 1]
    k_kv: List[int]
    k_tsp: Optional[List[int]]

    @property
    def total_len(self) -> int:
        return int(self.cu_seqlens[-1])


@dataclasses.dataclass
class LayerResult:
    request_id: Any
    idx_kv: np.ndarray              # [Hkv, k_kv] sequence-local, ascending
    k_out: np.ndarray               # [Hkv, k_kv, d]
    v_out: np.ndarray
    idx_tsp: Optional[np.ndarray] = None
    hidden_out: Optional[np.ndarray] = None
    pos_out: Optional[np.ndarray] = None


def pack(jobs: Sequence[LayerJob]) -> PackedBatch:
    """Concatenate jobs of one geometry along the token axis."""
    if not jobs:
        raise ValueError("nothing to pack")
    geo = jobs[0].geometry
    if any(j.geometry != geo for j in jobs):
        raise ValueError("jobs of different geometry cannot share a batch")
    for j in jobs:
        if j.length < geo.window or not (geo.window <= j.k_kv <= j.length):
            raise ValueError("request %r: need window <= k_kv <= length" % (j.request_id,))
        if geo.with_tsp and not (geo.window <= j.k_tsp <= j.length):
            raise ValueError("request %r: need window <= k_tsp <= length" % (j.request_id,))
    lens = [j.length for j in jobs]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    cat = lambda xs: np.ascontiguousarray(np.concatenate(xs, axis=0))
    return PackedBatch(
        geometry=geo, jobs=list(jobs), q_win=cat([j.q_win for j in jobs]), k=cat([j.k for j in jobs]),
        v=cat([j.v for j in jobs]), hidden=cat([j.hidden for j in jobs]) if geo.with_tsp else None,
        pos=cat([j.pos for j in jobs]).astype(np.int32) if geo.with_tsp else None, cu_seqlens=cu,
        k_kv=[j.k_kv for j in jobs], k_tsp=[j.k_tsp for j in jobs] if geo.with_tsp else None)


def unpack(batch: PackedBatch, out: Dict[str, np.ndarray]) -> List[LayerResult]:
    """Split the packed outputs of one call sequence back into per-request results."""
    cu_kv = np.concatenate([[0], np.cumsum(batch.k_kv)])
    cu_t = np.concatenate([[0], np.cumsum(batch.k_tsp)]) if batch.k_tsp is not None else None
    results = []
    for b, job in enumerate(batch.jobs):
        a, e = int(cu_kv[b]), int(cu_kv[b + 1])
        r = LayerResult(job.request_id, out["idx_kv"][:, a:e].copy(), out["k_out"][:, a:e].copy(),
                        out["v_out"][:, a:e].copy())
        if cu_t is not None:
            a, e = int(cu_t[b]), int(cu_t[b + 1])
            r.idx_tsp, r.hidden_out, r.pos_out = (out["idx_tsp"][a:e].copy(), out["hidden_out"][a:e].copy(),
                                                  out["pos_out"][a:e].copy())
        results.append(r)
    return results


class BatchScheduler:
    """FIFO queue of layer jobs, packed greedily under a token budget.

    `next_batch()` takes the oldest waiting job and then, in arrival order, every later job of the same
    geometry that still fits `max_tokens` and `max_requests`; jobs that do not fit stay queued in order,
    so nothing is overtaken by more than one batch's worth of later arrivals.  A job longer than the
    token budget runs alone.  `run_all(backend)` drains the queue and returns the results by request id.
    """

    def __init__(self, max_tokens: int = 1 << 18, max_requests: int = 64):
        if max_tokens < 1 or max_requests < 1:
            raise ValueError("max_tokens and max_requests must be positive")
        self.max_tokens, self.max_requests = max_tokens, max_requests
        self._queue: Deque[LayerJob] = deque()
        self.batches_run = 0

    def submit(self, job: LayerJob) -> None:
        self._queue.append(job)

    def __len__(self) -> int:
        return len(self._queue)

    def next_batch(self) -> Optional[PackedBatch]:
        if not self._queue:
            return None
        head = self._queue.popleft()
        chosen, tokens = [head], head.length
        rest: Deque[LayerJob] = deque()
        while self._queue:
            j = self._queue.popleft()
            if (j.geometry == head.geometry and len(chosen) < self.max_requests and
                    tokens + j.length <= self.max_tokens):
                chosen.append(j)
                tokens += j.length
            else:
                rest.append(j)
        self._queue = rest
        return pack(chosen)

    def run_all(self, backend) -> Dict[Any, LayerResult]:
        done: Dict[Any, LayerResult] = {}
        while True:
            batch = self.next_batch()
            if batch is None:
                return done
            for r in unpack(batch, backend.layer(batch)):
                done[r.request_id] = r
            self.batches_run += 1


class CudaBatchBackend:
    """The three calls of the C ABI on a packed batch: host arrays in, host arrays out.  Device memory
    comes from torch; every step runs in the library's kernels."""

    def layer(self, batch: PackedBatch) -> Dict[str, np.ndarray]:
        import torch
        from . import binding as B
        geo, Bn, total = batch.geometry, len(batch.jobs), batch.total_len
        dev = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).cuda()
        d_cu = dev(batch.cu_seqlens)
        lens = np.diff(batch.cu_seqlens)
        shape = B.make_shape(total_len=total, n_q_heads=geo.n_q_heads, n_kv_heads=geo.n_kv_heads,
                             head_dim=geo.head_dim, hidden_dim=geo.hidden_dim, window=geo.window,
                             pool_kernel=geo.pool_kernel, pool_mode=geo.pool_mode, batch=Bn,
                             max_len=int(lens.max()), cu_seqlens=d_cu)
        q, k, v = dev(batch.q_win), dev(batch.k), dev(batch.v)
        ws = torch.empty(B.fastkv_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
        s_kv = torch.empty((geo.n_kv_heads, total), dtype=torch.float32, device="cuda")
        s_tsp = torch.empty((total,), dtype=torch.float32, device="cuda") if geo.with_tsp else None
        B.fastkv_score(shape, q, k, s_kv, s_tsp, ws)

        def budget(ks):
            cu_k = dev(np.concatenate([[0], np.cumsum(ks)]).astype(np.int32))
            return B.make_budget(0, cu_k=cu_k, total=int(sum(ks))), cu_k

        b_kv, keep_kv = budget(batch.k_kv)
        idx_kv = torch.empty((geo.n_kv_heads, b_kv.total), dtype=torch.int32, device="cuda")
        k_out = torch.empty((geo.n_kv_heads, b_kv.total, geo.head_dim), dtype=torch.int16, device="cuda")
        v_out = torch.empty_like(k_out)
        out: Dict[str, np.ndarray] = {}
        if geo.with_tsp:
            b_tsp, keep_tsp = budget(batch.k_tsp)
            hid, pos = dev(batch.hidden), dev(batch.pos)
            idx_tsp = torch.empty((b_tsp.total,), dtype=torch.int32, device="cuda")
            hid_out = torch.empty((b_tsp.total, geo.hidden_dim), dtype=torch.int16, device="cuda")
            pos_out = torch.empty((b_tsp.total,), dtype=torch.int32, device="cuda")
            B.fastkv_select(shape, s_kv, b_kv, idx_kv, s_tsp, b_tsp, idx_tsp, ws)
            B.fastkv_compact(shape, idx_kv, b_kv, idx_tsp, b_tsp, k, v, hid, pos, k_out, v_out, hid_out, pos_out, ws)
        else:
            B.fastkv_select_kv(shape, s_kv, b_kv, idx_kv, ws)
            B.fastkv_compact(shape, idx_kv, b_kv, None, None, k, v, None, None, k_out, v_out, None, None, ws)
        status, site = B.fastkv_device_status(ws)
        if status != 0:
            raise RuntimeError("device status %d at site %d" % (status, site))
        out.update(idx_kv=idx_kv.cpu().numpy(), k_out=k_out.cpu().numpy().view(np.uint16),
                   v_out=v_out.cpu().numpy().view(np.uint16))
        if geo.with_tsp:
            out.update(idx_tsp=idx_tsp.cpu().numpy(), hidden_out=hid_out.cpu().numpy().view(np.uint16),
                       pos_out=pos_out.cpu().numpy())
        return out
