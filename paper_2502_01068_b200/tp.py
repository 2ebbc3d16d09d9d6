"""Tensor-parallel layer step: KV heads sharded over ranks, one all-reduce.

Scoring, KV selection and K/V compaction are independent per KV head (Eq. 1, App. B.1), so a rank
that holds `n_kv_heads / world` heads runs them locally.  The only quantity that needs every head
is the layer-level score of Eq. 2: each rank sums its own heads, the partial sums are all-reduced
(fp32, `total_len` values: 512 KB at 128K tokens), and every rank then runs the same deterministic
HiddenCompress selection on identical numbers and gathers the hidden rows (or its column shard of
them) with the shared index set.

The step functions are passed in (`backend`), so the same orchestration drives the CUDA library
(`CudaBackend`, one process per GPU, NCCL) and, in the CPU tests, a stand-in that checks the
sharding arithmetic with gloo.  Remote data is reduced into local memory by the collective; no
kernel of this library ever reads a peer's memory.
"""
from __future__ import annotations

import dataclasses
from typing import Any, Callable, Optional, Sequence

import torch
import torch.distributed as dist


@dataclasses.dataclass
class HeadShard:
    """Which KV heads (and, with them, which query heads) a rank owns."""
    rank: int
    world: int
    n_q_heads: int
    n_kv_heads: int

    def __post_init__(self):
        if self.n_kv_heads % self.world:
            raise ValueError("n_kv_heads must be divisible by the tensor-parallel world size")
        if self.n_q_heads % self.n_kv_heads:
            raise ValueError("n_q_heads must be a multiple of n_kv_heads")

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def local_kv_heads(self) -> int:
        return self.n_kv_heads // self.world

    @property
    def kv_range(self) -> range:
        return range(self.rank * self.local_kv_heads, (self.rank + 1) * self.local_kv_heads)

    @property
    def q_range(self) -> range:
        return range(self.kv_range.start * self.group, self.kv_range.stop * self.group)


def all_reduce_sum(t: torch.Tensor, group=None) -> torch.Tensor:
    """In-place sum over the tensor-parallel group (NCCL over NVLink on GPUs, gloo in the CPU tests)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return t


def tp_layer_step(backend: Any, shard: HeadShard, q_local, k_local, v_local, hidden, pos, k_kv, k_tsp,
                  group=None, reduce_fn: Optional[Callable[[torch.Tensor], torch.Tensor]] = None):
    """One layer on one rank.  q_local/k_local/v_local hold this rank's heads only; hidden and pos are
    replicated (or hidden is this rank's column shard).  Returns (idx_kv_local, idx_tsp, k_out, v_out,
    hidden_out, pos_out).  `reduce_fn` replaces the collective (used to emulate ranks in one process)."""
    s_kv, s_tsp_partial = backend.score(q_local, k_local)              # local heads; partial Eq. 2 sum
    s_tsp = (reduce_fn or (lambda t: all_reduce_sum(t, group)))(s_tsp_partial)
    idx_kv, idx_tsp = backend.select(s_kv, k_kv, s_tsp, k_tsp)         # identical idx_tsp on every rank
    k_out, v_out, hidden_out, pos_out = backend.compact(idx_kv, idx_tsp, k_local, v_local, hidden, pos)
    return idx_kv, idx_tsp, k_out, v_out, hidden_out, pos_out


class CudaBackend:
    """The three calls of the C ABI for one rank's shard of a single sequence (device tensors in, device
    tensors out).  bf16 tensors are int16 views, as everywhere in the binding."""

    def __init__(self, shard: HeadShard, total_len: int, head_dim: int, hidden_dim: int, window: int = 8,
                 pool_kernel: int = 7, pool_mode: int = 0, hidden_stride_tok: Optional[int] = None):
        from . import binding as B
        self.B, self.shard = B, shard
        self.total_len, self.head_dim, self.hidden_dim = total_len, head_dim, hidden_dim
        self.shape = B.make_shape(total_len=total_len, n_q_heads=shard.local_kv_heads * shard.group,
                                  n_kv_heads=shard.local_kv_heads, head_dim=head_dim, hidden_dim=hidden_dim,
                                  window=window, pool_kernel=pool_kernel, pool_mode=pool_mode,
                                  hidden_stride_tok=hidden_stride_tok)
        self.ws = torch.empty(B.fastkv_workspace_bytes(self.shape), dtype=torch.uint8, device="cuda")

    def score(self, q, k):
        s_kv = torch.empty((self.shard.local_kv_heads, self.total_len), dtype=torch.float32, device="cuda")
        s_tsp = torch.empty((self.total_len,), dtype=torch.float32, device="cuda")
        self.B.fastkv_score(self.shape, q, k, s_kv, s_tsp, self.ws)
        return s_kv, s_tsp

    def select(self, s_kv, k_kv, s_tsp, k_tsp):
        self.b_kv, self.b_tsp = self.B.make_budget(k_kv), self.B.make_budget(k_tsp)
        idx_kv = torch.empty((self.shard.local_kv_heads, k_kv), dtype=torch.int32, device="cuda")
        idx_tsp = torch.empty((k_tsp,), dtype=torch.int32, device="cuda")
        self.B.fastkv_select(self.shape, s_kv, self.b_kv, idx_kv, s_tsp, self.b_tsp, idx_tsp, self.ws)
        return idx_kv, idx_tsp

    def compact(self, idx_kv, idx_tsp, k, v, hidden, pos):
        n, kk, kt = self.shard.local_kv_heads, idx_kv.shape[1], idx_tsp.shape[0]
        k_out = torch.empty((n, kk, self.head_dim), dtype=torch.int16, device="cuda")
        v_out = torch.empty_like(k_out)
        hidden_out = torch.empty((kt, self.hidden_dim), dtype=torch.int16, device="cuda")
        pos_out = torch.empty((kt,), dtype=torch.int32, device="cuda")
        self.B.fastkv_compact(self.shape, idx_kv, self.b_kv, idx_tsp, self.b_tsp, k, v, hidden, pos, k_out, v_out,
                              hidden_out, pos_out, self.ws)
        return k_out, v_out, hidden_out, pos_out


def shard_heads(t: torch.Tensor, heads: Sequence[int]) -> torch.Tensor:
    """[tokens, heads, dim] -> the contiguous slice of `heads` (what a rank holds after a TP projection)."""
    return t[:, heads.start:heads.stop, :].contiguous()
