"""GPU parity of the prefill attention with the saliency by-product: the attention output against the fp64
oracle of causal softmax attention, and the scores it hands out against the oracle of the scoring path (the
same bar as fastkv_score: 2e-3 relative), on lengths that span several tiles and a ragged tail."""
import numpy as np
import pytest
import torch

import oracle
from paper_2502_01068_b200 import binding as B
from paper_2502_01068_b200 import workloads as W
from tests.parity import check_scores, dev, oracle_layer

pytestmark = pytest.mark.gpu

# P is rounded to bf16 before it meets V (2^-9 relative per probability, independent signs) and the output is
# rounded to bf16 (2^-9 relative): with values ~ N(0,1) the error of an output element stays well inside
# 1e-2 * |O| + 1e-2 (observed worst cases are printed by the tests' assertion messages)
O_RTOL, O_ATOL = 1e-2, 1e-2


def small(name, cfg, lens, Hq=8, Hkv=2, d=128, w=8, p=7):
    return W.Workload(name=name, cfg=cfg, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, hidden_dim=64, window=w,
                      pool_kernel=p, pool_mode=W.POOL_AVG, seq_lens=list(lens), k_kv=[w] * len(lens),
                      k_tsp=[w] * len(lens))


def run_prefill(wl, x, q_full, *, pool_mode=None, agg_order=B.GROUP_THEN_POOL, want_scores=True):
    total, Bn = wl.total_len, wl.batch
    d_cu = dev(x.cu_seqlens) if Bn > 1 else None
    shape = B.make_shape(total_len=total, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                         hidden_dim=wl.hidden_dim, window=wl.window, pool_kernel=wl.pool_kernel,
                         pool_mode=wl.pool_mode if pool_mode is None else pool_mode, agg_order=agg_order, batch=Bn,
                         max_len=max(wl.seq_lens), cu_seqlens=d_cu, q_layout=B.Q_FULL)
    ws = torch.empty(B.fastkv_prefill_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    out = torch.full((total, wl.n_q_heads, wl.head_dim), -1, dtype=torch.int16, device="cuda")
    s_kv = torch.full((wl.n_kv_heads, total), -1.0, dtype=torch.float32, device="cuda") if want_scores else None
    s_tsp = torch.full((total,), -1.0, dtype=torch.float32, device="cuda") if want_scores else None
    B.fastkv_prefill_attention(shape, dev(q_full), dev(x.k), dev(x.v), out, s_kv, s_tsp, ws)
    assert B.fastkv_device_status(ws) == (0, 0)
    o = W.bf16_bits_to_f32(out.cpu().numpy().view(np.uint16)).astype(np.float64)
    return o, (s_kv.cpu().numpy() if want_scores else None), (s_tsp.cpu().numpy() if want_scores else None)


def check_output(got, wl, x, q_full, what):
    cu = x.cu_seqlens
    for b in range(wl.batch):
        a, e = int(cu[b]), int(cu[b + 1])
        ref = oracle.prefill_attention(q_full[a:e], x.k[a:e], x.v[a:e])
        err = np.abs(got[a:e] - ref)
        bad = err > O_RTOL * np.abs(ref) + O_ATOL
        assert not bad.any(), "%s seq %d: %d outputs off, worst abs err %.3e" % (what, b, int(bad.sum()), float(err.max()))


@pytest.mark.parametrize("L,d,Hq,Hkv,w", [(512, 64, 4, 1, 8), (100, 64, 4, 1, 8), (129, 128, 8, 2, 8), (1000, 128, 8, 2, 8),
                                           (777, 64, 16, 2, 8), (1030, 128, 4, 4, 8), (640, 128, 8, 2, 16), (8, 64, 4, 1, 8)])
def test_attention_output_and_scores_match_the_oracles(L, d, Hq, Hkv, w):
    wl = small("prefill", 900 + L, [L], Hq=Hq, Hkv=Hkv, d=d, w=w)
    x = W.make_layer(wl)
    q_full = W.full_q(wl, x)
    for pool_mode, order in ((B.POOL_AVG, B.GROUP_THEN_POOL), (B.POOL_MAX, B.POOL_THEN_GROUP)):
        o, s_kv, s_tsp = run_prefill(wl, x, q_full, pool_mode=pool_mode, agg_order=order)
        check_output(o, wl, x, q_full, "L=%d" % L)
        ref = oracle_layer(wl, x, pool_mode=pool_mode, agg_order=order, do_compact=False)
        check_scores(s_kv, ref["S_kv"], "S_kv from the attention, L=%d" % L)
        check_scores(s_tsp, ref["S_tsp"], "S_tsp from the attention, L=%d" % L)


def test_ragged_batch_and_attention_only():
    wl = small("prefill_ragged", 950, [300, 130, 1000, 64], Hq=8, Hkv=2, d=128)
    x = W.make_layer(wl)
    q_full = W.full_q(wl, x)
    o, s_kv, s_tsp = run_prefill(wl, x, q_full)
    check_output(o, wl, x, q_full, "ragged")
    ref = oracle_layer(wl, x, do_compact=False)
    check_scores(s_kv, ref["S_kv"], "S_kv, ragged")
    check_scores(s_tsp, ref["S_tsp"], "S_tsp, ragged")
    o2, none_kv, _ = run_prefill(wl, x, q_full, want_scores=False)
    assert none_kv is None
    np.testing.assert_array_equal(o2, o)                    # the by-product does not change the attention


def test_scores_from_the_attention_agree_with_the_scoring_path():
    """Same layer through fastkv_score (window queries x K) and through the attention's by-product."""
    from tests.parity import gpu_layer
    wl = small("prefill_vs_score", 960, [2500], Hq=8, Hkv=2, d=128)
    x = W.make_layer(wl)
    q_full = W.full_q(wl, x)
    _, s_kv, s_tsp = run_prefill(wl, x, q_full)
    g = gpu_layer(wl, x)
    np.testing.assert_allclose(s_kv, g["S_kv"], rtol=2e-3, atol=1e-12)
    np.testing.assert_allclose(s_tsp, g["S_tsp"], rtol=2e-3, atol=1e-12)


def test_peaked_and_wide_logits():
    """A large softmax scale: rows pick single keys and the running reference moves often (O is rescaled)."""
    wl = small("prefill_peaked", 970, [700], Hq=4, Hkv=2, d=64)
    x = W.make_layer(wl)
    q_full = W.full_q(wl, x)
    total = wl.total_len
    shape = B.make_shape(total_len=total, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                         window=wl.window, pool_kernel=wl.pool_kernel, q_layout=B.Q_FULL, softmax_scale=2.0)
    ws = torch.empty(B.fastkv_prefill_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    out = torch.zeros((total, wl.n_q_heads, wl.head_dim), dtype=torch.int16, device="cuda")
    B.fastkv_prefill_attention(shape, dev(q_full), dev(x.k), dev(x.v), out, None, None, ws)
    assert B.fastkv_device_status(ws) == (0, 0)
    got = W.bf16_bits_to_f32(out.cpu().numpy().view(np.uint16)).astype(np.float64)
    ref = oracle.prefill_attention(q_full, x.k, x.v, scale=2.0)
    err = np.abs(got - ref)
    assert np.all(err <= O_RTOL * np.abs(ref) + O_ATOL), float(err.max())


def test_long_prompts_on_sampled_rows():
    """Prompts of tens of key tiles (a single one that ends 77 tokens into a pair of query tiles, and a ragged
    batch): the oracle of the whole attention would take minutes, so sampled query rows -- the first rows, rows on
    both sides of the 128- and 256-row boundaries, rows deep in the prompt and the last rows -- are checked one by
    one against the oracle of a single query over its causal prefix (oracle.decode_attention: the same softmax
    attention of one token over keys 0 .. t)."""
    for lens, Hq, Hkv, d in (([16384 + 77], 8, 2, 128), ([5000, 129, 9000], 4, 1, 64)):
        wl = small("prefill_long", 990 + len(lens), lens, Hq=Hq, Hkv=Hkv, d=d)
        x = W.make_layer(wl)
        q_full = W.full_q(wl, x)
        got, _, _ = run_prefill(wl, x, q_full, want_scores=False)
        cu = x.cu_seqlens
        rng = np.random.default_rng(5)
        for b, L in enumerate(lens):
            a = int(cu[b])
            rows = {0, 1, 127, 128, 129, 255, 256, 257, 383, 384, L - 1, L - 2, L - 130} | set(int(t) for t in rng.integers(0, L, 12))
            for t in sorted(r for r in rows if 0 <= r < L):
                kc = np.ascontiguousarray(x.k[a:a + t + 1].transpose(1, 0, 2))     # [Hkv, t + 1, d]
                vc = np.ascontiguousarray(x.v[a:a + t + 1].transpose(1, 0, 2))
                ref, _ = oracle.decode_attention(q_full[a + t], kc, vc)
                err = np.abs(got[a + t] - ref)
                assert np.all(err <= O_RTOL * np.abs(ref) + O_ATOL), (lens, b, t, float(err.max()))
