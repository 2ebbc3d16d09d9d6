"""Seeded random shapes through the scoring kernels' modes and the prefill attention, against the oracle: batch
size, head counts, head dimension, window, pooling, aggregation order and lengths (some shorter than a tile, some
spanning many) are drawn per case; every case runs the library's own choice of kernel and the parked kernel with
its partition mode forced on, forced off and left to the shape."""
import numpy as np
import pytest
import torch

import oracle
from paper_2502_01068_b200 import binding as B
from paper_2502_01068_b200 import workloads as W
from tests.parity import check_layer, check_scores, dev, gpu_layer, oracle_layer

pytestmark = pytest.mark.gpu


def draw(rng, it, max_len, long_len=None):
    Bn = int(rng.integers(1, 6))
    Hkv = int(rng.choice([1, 2, 4, 8])); G = int(rng.choice([1, 2, 4, 8])); d = int(rng.choice([64, 128])); w = int(rng.choice([4, 8, 16]))
    if G * w > 64:
        w = 64 // G
    lens = [int(rng.integers(w, max_len)) if long_len is None or rng.random() < 0.8 else int(rng.integers(max_len, long_len))
            for _ in range(Bn)]
    budgets = lambda: [int(rng.integers(w, max(w + 1, min(L, 3000)))) for L in lens]
    return W.Workload(name="random", cfg=7000 + it, n_q_heads=Hkv * G, n_kv_heads=Hkv, head_dim=d, hidden_dim=64, window=w,
                      pool_kernel=int(rng.choice([1, 3, 7, 9])), pool_mode=int(rng.choice([W.POOL_AVG, W.POOL_MAX])),
                      seq_lens=lens, k_kv=budgets(), k_tsp=budgets())


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_layers_through_every_mode_of_the_scoring_kernels(debug_hooks, seed):
    rng = np.random.default_rng(seed)
    for it in range(6):
        wl = draw(rng, seed * 100 + it, 30000, 120000)
        x = W.make_layer(wl)
        order = int(rng.choice([B.GROUP_THEN_POOL, B.POOL_THEN_GROUP]))
        o = oracle_layer(wl, x, agg_order=order)
        for path, part in ((0, 0), (3, 2), (3, 0), (3, 1), (2, 0)):
            debug_hooks("score_path", path)
            debug_hooks("score_partition", part)
            try:
                g = gpu_layer(wl, x, agg_order=order)
            except B.FastKVError as e:                     # a forced kernel that is not built for the shape
                assert e.status == B.ERR_UNSUPPORTED
                continue
            check_layer(wl, x, g, o, what="seed %d case %d path %d partition %d lens %s" % (seed, it, path, part, wl.seq_lens))


@pytest.mark.parametrize("seed", [21, 22])
def test_random_prompts_through_the_prefill_attention(seed):
    rng = np.random.default_rng(seed)
    for it in range(8):
        wl = draw(rng, seed * 100 + it, 1500)
        x = W.make_layer(wl)
        q_full = W.full_q(wl, x)
        total, Bn = wl.total_len, wl.batch
        order = int(rng.choice([B.GROUP_THEN_POOL, B.POOL_THEN_GROUP]))
        scale = float(rng.choice([0.0, 0.0, 0.5, 1.5]))
        d_cu = dev(x.cu_seqlens) if Bn > 1 else None
        shape = B.make_shape(total_len=total, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                             hidden_dim=64, window=wl.window, pool_kernel=wl.pool_kernel, pool_mode=wl.pool_mode,
                             agg_order=order, batch=Bn, max_len=max(wl.seq_lens), cu_seqlens=d_cu, q_layout=B.Q_FULL,
                             softmax_scale=scale)
        ws = torch.empty(B.fastkv_prefill_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
        out = torch.zeros((total, wl.n_q_heads, wl.head_dim), dtype=torch.int16, device="cuda")
        s_kv = torch.zeros((wl.n_kv_heads, total), dtype=torch.float32, device="cuda")
        s_tsp = torch.zeros((total,), dtype=torch.float32, device="cuda")
        B.fastkv_prefill_attention(shape, dev(q_full), dev(x.k), dev(x.v), out, s_kv, s_tsp, ws)
        assert B.fastkv_device_status(ws) == (0, 0)
        got = W.bf16_bits_to_f32(out.cpu().numpy().view(np.uint16)).astype(np.float64)
        what = "seed %d case %d lens %s scale %s" % (seed, it, wl.seq_lens, scale)
        for b in range(Bn):
            a, e = int(x.cu_seqlens[b]), int(x.cu_seqlens[b + 1])
            ref = oracle.prefill_attention(q_full[a:e], x.k[a:e], x.v[a:e], scale=None if scale == 0.0 else scale)
            assert np.all(np.abs(got[a:e] - ref) <= 1e-2 * np.abs(ref) + 1e-2), what
        if scale == 0.0:                                   # the scoring oracle uses the default scale
            o = oracle_layer(wl, x, agg_order=order, do_compact=False)
            check_scores(s_kv.cpu().numpy(), o["S_kv"], what)
            check_scores(s_tsp.cpu().numpy(), o["S_tsp"], what)
