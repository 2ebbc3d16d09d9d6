"""Seeded synthetic inputs for the FastKV score/select/compact path.

This module only *draws inputs*: bf16 Q/K/V/hidden tensors with the shapes,
sequence lengths and sparse heavy-hitter structure of the paper's workloads
(long prompts through a Llama-3.1-8B-shaped decoder; Section 3.2 describes the
few tokens that collect most of the attention mass).  It contains none of the
method's arithmetic (no softmax, pooling, ranking or gathering), so the CPU
oracle and the CUDA path can both be fed from it without sharing any code that
is under test.

All tensors are host numpy arrays.  bf16 values are carried as uint16 bit
patterns (numpy has no bf16), produced by round-to-nearest-even from float32
draws of `numpy.random.Generator(PCG64(SeedSequence([...])))`.
"""
from __future__ import annotations

import dataclasses
import os
from concurrent.futures import ThreadPoolExecutor
from typing import List, Optional, Sequence

import numpy as np

POOL_AVG = 0
POOL_MAX = 1
GROUP_THEN_POOL = 0
POOL_THEN_GROUP = 1

_T_Q, _T_K, _T_V, _T_HID, _T_PLANT, _T_LEN = range(6)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u >> np.uint32(16)) & np.uint32(1)
    r += np.uint32(0x7FFF)
    r += u
    r >>= np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence(list(key))))


_CHUNK_ELEMS = 1 << 22


def _normal_bf16(key: Sequence[int], shape) -> np.ndarray:
    """N(0,1) draws rounded to bf16.  Row chunk c is drawn from its own stream
    SeedSequence([*key, c]), so the result does not depend on how many threads fill it."""
    out = np.empty(shape, dtype=np.uint16)
    if out.size == 0:
        return out
    flat = out.reshape(shape[0], -1)
    rows_per = max(1, _CHUNK_ELEMS // flat.shape[1])
    starts = list(range(0, shape[0], rows_per))

    def fill(c: int) -> None:
        r0 = starts[c]
        r1 = min(shape[0], r0 + rows_per)
        x = _rng(*key, c).standard_normal((r1 - r0, flat.shape[1]), dtype=np.float32)
        flat[r0:r1] = f32_to_bf16_bits(x)

    if len(starts) == 1:
        fill(0)
    else:
        with ThreadPoolExecutor(max_workers=min(len(starts), os.cpu_count() or 1)) as ex:
            list(ex.map(fill, range(len(starts))))
    return out


@dataclasses.dataclass
class Workload:
    """Static description of one benchmark / parity configuration."""
    name: str
    cfg: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    hidden_dim: int
    window: int
    pool_kernel: int
    pool_mode: int
    seq_lens: List[int]
    k_kv: List[int]                 # per sequence KV budget (window included)
    k_tsp: Optional[List[int]]      # per sequence TSP budget, None on non-TSP layers
    plant: str = "uniform"          # "uniform" | "zipf" | "none"
    plant_frac: float = 0.01
    plant_count: Optional[int] = None
    plant_gain: float = 3.0
    plant_norm: str = "unit"        # "unit": +gain * unit mean-window-query direction
    n_sinks: int = 4
    zipf_alpha: float = 1.1

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def total_len(self) -> int:
        return int(sum(self.seq_lens))

    @property
    def batch(self) -> int:
        return len(self.seq_lens)

    def cu_seqlens(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.seq_lens)]).astype(np.int32)

    def with_lens(self, seq_lens: Sequence[int], k_kv: Sequence[int],
                  k_tsp: Optional[Sequence[int]]) -> "Workload":
        return dataclasses.replace(self, seq_lens=list(seq_lens), k_kv=list(k_kv),
                                   k_tsp=None if k_tsp is None else list(k_tsp))


@dataclasses.dataclass
class LayerInputs:
    """One layer's tensors, packed over the sequences of the batch."""
    q_win: np.ndarray               # uint16 [B*w, Hq, d]: the last w query rows of each sequence
    k: np.ndarray                   # uint16 [total, Hkv, d]
    v: Optional[np.ndarray]         # uint16 [total, Hkv, d]
    hidden: Optional[np.ndarray]    # uint16 [total, hidden]
    pos: np.ndarray                 # int32 [total]
    cu_seqlens: np.ndarray          # int32 [B+1]
    planted: List[np.ndarray]       # per sequence: sorted planted positions (sequence-local)


def _planted_positions(wl: Workload, rng: np.random.Generator, L: int) -> np.ndarray:
    w = wl.window
    hi = L - w                       # plants live in the prefix [0, L-w)
    if wl.plant == "none" or hi <= 0:
        return np.zeros(0, dtype=np.int64)
    sinks = np.arange(min(wl.n_sinks, hi), dtype=np.int64)
    n = wl.plant_count if wl.plant_count is not None else int(np.ceil(wl.plant_frac * L))
    if wl.plant == "uniform":
        lo = min(wl.n_sinks, hi)
        if hi - lo <= 0:
            return sinks
        n = min(n, hi - lo)
        extra = rng.choice(np.arange(lo, hi, dtype=np.int64), size=n, replace=False)
        return np.unique(np.concatenate([sinks, extra]))
    if wl.plant == "zipf":
        # truncated Zipf over position rank r = 1..hi: P(position = r-1) ~ r^-alpha,
        # drawn by inverse CDF and de-duplicated (so low positions form dense blocks)
        r = np.arange(1, hi + 1, dtype=np.float64)
        cdf = np.cumsum(r ** (-wl.zipf_alpha))
        cdf /= cdf[-1]
        draws = np.searchsorted(cdf, rng.random(n), side="left")
        return np.unique(np.minimum(draws, hi - 1).astype(np.int64))
    raise ValueError(wl.plant)


def make_layer(wl: Workload, layer: int = 0, *, with_v: bool = True, with_hidden: bool = True,
               seq_lens: Optional[Sequence[int]] = None,
               pos: Optional[np.ndarray] = None) -> LayerInputs:
    """Draw the tensors of one layer of `wl`.

    `seq_lens` overrides the workload's lengths (layers after the TSP layer run
    on the propagated length); `pos` overrides the default arange position ids
    (later layers receive the ids carried by the propagated tokens).
    """
    lens = list(wl.seq_lens if seq_lens is None else seq_lens)
    B, w, Hq, Hkv, d, G = len(lens), wl.window, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.group
    total = int(sum(lens))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    q_win = _normal_bf16((wl.cfg, layer, _T_Q), (B * w, Hq, d))
    k = _normal_bf16((wl.cfg, layer, _T_K), (total, Hkv, d))
    planted = []
    prng = _rng(wl.cfg, layer, _T_PLANT)
    qf = bf16_bits_to_f32(q_win).reshape(B, w, Hkv, G, d)
    for b, L in enumerate(lens):
        p = _planted_positions(wl, prng, L)
        planted.append(p)
        if p.size == 0:
            continue
        # mean of the G*w window-query vectors of each KV head's group
        m = qf[b].astype(np.float64).mean(axis=(0, 2))                  # [Hkv, d]
        if wl.plant_norm == "unit":
            m = m / np.maximum(np.linalg.norm(m, axis=-1, keepdims=True), 1e-30)
        rows = cu[b] + p
        kk = bf16_bits_to_f32(k[rows]).astype(np.float64) + wl.plant_gain * m[None, :, :]
        k[rows] = f32_to_bf16_bits(kk.astype(np.float32))
    v = _normal_bf16((wl.cfg, layer, _T_V), (total, Hkv, d)) if with_v else None
    hidden = (_normal_bf16((wl.cfg, layer, _T_HID), (total, wl.hidden_dim))
              if with_hidden else None)
    if pos is None:
        pos = np.concatenate([np.arange(L, dtype=np.int32) for L in lens]) if lens else \
            np.zeros(0, np.int32)
    return LayerInputs(q_win=q_win, k=k, v=v, hidden=hidden, pos=np.ascontiguousarray(pos, np.int32),
                       cu_seqlens=cu, planted=planted)


def full_q(wl: Workload, x: LayerInputs, layer: int = 0) -> np.ndarray:
    """The packed query tensor [total, Hq, d] of a layer: the rows the method reads (the last w of every
    sequence) are x.q_win, every other row is an independent N(0,1) draw that must not matter."""
    total = int(x.cu_seqlens[-1])
    q = _normal_bf16((wl.cfg, layer, _T_Q, 1), (total, wl.n_q_heads, wl.head_dim))
    w = wl.window
    for b in range(len(x.cu_seqlens) - 1):
        hi = int(x.cu_seqlens[b + 1])
        if hi - int(x.cu_seqlens[b]) >= w:
            q[hi - w:hi] = x.q_win[b * w:(b + 1) * w]
    return q


def _llama8b(name: str, cfg: int, seq_lens, k_kv, k_tsp, **kw) -> Workload:
    return Workload(name=name, cfg=cfg, n_q_heads=32, n_kv_heads=8, head_dim=128, hidden_dim=4096,
                    window=8, pool_kernel=7, pool_mode=POOL_AVG, seq_lens=list(seq_lens),
                    k_kv=list(k_kv), k_tsp=None if k_tsp is None else list(k_tsp), **kw)


def tiny() -> Workload:
    """Config 1: one layer, 4 query heads on 1 KV head, d=64, L=512, 4 sinks + 5 plants."""
    return Workload(name="tiny", cfg=0, n_q_heads=4, n_kv_heads=1, head_dim=64, hidden_dim=256,
                    window=8, pool_kernel=7, pool_mode=POOL_AVG, seq_lens=[512], k_kv=[128],
                    k_tsp=[128], plant="uniform", plant_count=5)


def llama8b_8k() -> Workload:
    """Config 2: Llama-3.1-8B head shape, L=8192, KV budget 2048, TSP keeps 20 %."""
    L = 8192
    return _llama8b("llama8b_8k", 1, [L], [2048], [L * 20 // 100])


def llama8b_32k_sweep() -> Workload:
    """Config 3: 32-layer sweep at L=32768; TSP at layer 15 keeps 20 %, later layers run on that."""
    L = 32768
    return _llama8b("llama8b_32k_sweep", 2, [L], [2048], [L * 20 // 100])


SWEEP_LAYERS = 32
SWEEP_TSP_LAYER = 15


def llama8b_128k() -> Workload:
    """Config 4: L=131072, KV retention 10 %, TSP keeps 20 %, Zipf-placed heavy hitters."""
    L = 131072
    return _llama8b("llama8b_128k", 3, [L], [L * 10 // 100], [L * 20 // 100], plant="zipf")


def ragged_lengths() -> List[int]:
    return [int(x) for x in _rng(4, 0, _T_LEN).integers(4096, 65536, size=8, endpoint=True)]


def llama8b_ragged() -> Workload:
    """Config 5: 8 sequences of 4K..64K tokens, per-sequence KV budget 2048, TSP keeps 20 %."""
    lens = ragged_lengths()
    return _llama8b("llama8b_ragged", 4, lens, [2048] * len(lens), [L * 20 // 100 for L in lens])


def all_workloads() -> List[Workload]:
    return [tiny(), llama8b_8k(), llama8b_32k_sweep(), llama8b_128k(), llama8b_ragged()]
