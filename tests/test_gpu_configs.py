"""GPU parity on the benchmark configurations at their full sizes (configs 3, 4, 5), run through the same
call sequence and launch configuration the bench times."""
import dataclasses

import numpy as np
import pytest

from paper_2502_01068_b200 import workloads as W
from tests.parity import check_layer, gpu_layer, oracle_layer

pytestmark = pytest.mark.gpu


def test_llama8b_128k_tsp_layer_and_post_tsp_layer():
    wl = W.llama8b_128k()
    x = W.make_layer(wl)
    g = gpu_layer(wl, x)
    o = oracle_layer(wl, x, do_compact=False)
    st = check_layer(wl, x, g, o, what="128k tsp layer")
    print("128k: max rel score err %.3e, boundary flips %d" % (st["score_err"], st["flips"]))
    # the next layer runs on the propagated tokens with their carried position ids; its KV budget is
    # still 10 % of the original prompt
    L2 = wl.k_tsp[0]
    wl2 = dataclasses.replace(wl, seq_lens=[L2], k_tsp=None)
    x2 = W.make_layer(wl2, layer=1, with_hidden=False, pos=g["pos_out"])
    np.testing.assert_array_equal(x2.pos, g["idx_tsp"])          # position ids started as arange
    g2 = gpu_layer(wl2, x2)
    o2 = oracle_layer(wl2, x2, do_compact=False)
    check_layer(wl2, x2, g2, o2, what="128k post-tsp layer")


def test_llama8b_ragged_batch():
    wl = W.llama8b_ragged()
    x = W.make_layer(wl)
    g = gpu_layer(wl, x)
    o = oracle_layer(wl, x, do_compact=False)
    st = check_layer(wl, x, g, o, what="ragged")
    print("ragged: max rel score err %.3e, boundary flips %d" % (st["score_err"], st["flips"]))


def test_llama8b_32k_sweep():
    """32 layers with independent synthetic Q/K/V: layers 0..15 on the full prompt, TSP at layer 15,
    layers 16..31 on the propagated tokens with the carried position ids (Alg. 1's loop)."""
    wl = W.llama8b_32k_sweep()
    pos_g = pos_o = None
    flips = 0
    for layer in range(W.SWEEP_LAYERS):
        tsp_layer = layer == W.SWEEP_TSP_LAYER
        if layer <= W.SWEEP_TSP_LAYER:
            wll = wl if tsp_layer else dataclasses.replace(wl, k_tsp=None)
            x = W.make_layer(wll, layer=layer, with_hidden=tsp_layer)
        else:
            wll = dataclasses.replace(wl, seq_lens=[wl.k_tsp[0]], k_tsp=None)
            x = W.make_layer(wll, layer=layer, with_hidden=False, pos=pos_g)
        g = gpu_layer(wll, x)
        o = oracle_layer(wll, x, do_compact=tsp_layer)
        flips += check_layer(wll, x, g, o, what="sweep layer %d" % layer)["flips"]
        if tsp_layer:
            pos_g, pos_o = g["pos_out"], o["pos_out"]
            if np.array_equal(g["idx_tsp"], o["idx_tsp"]):
                np.testing.assert_array_equal(pos_g, pos_o)
    print("sweep: boundary flips over 32 layers: %d" % flips)


def test_llama8b_128k_prefill_attention_hands_out_the_layer_scores():
    """The 131072-token layer through the prefill attention in the launch configuration the bench times: the
    scores it hands out against the oracle of the scoring path (2e-3 relative, as for fastkv_score), and the
    attention output on sampled rows against the oracle of one query over its causal prefix."""
    import oracle
    from tests.test_gpu_prefill import O_ATOL, O_RTOL, run_prefill
    wl = W.llama8b_128k()
    x = W.make_layer(wl, with_hidden=False)
    q_full = W.full_q(wl, x)
    got, s_kv, s_tsp = run_prefill(wl, x, q_full)
    o = oracle_layer(wl, x, do_compact=False)
    np.testing.assert_allclose(s_kv, o["S_kv"], rtol=2e-3, atol=1e-12)
    np.testing.assert_allclose(s_tsp, o["S_tsp"], rtol=2e-3, atol=1e-12)
    L = wl.total_len
    rng = np.random.default_rng(9)
    rows = sorted({0, 255, 256, L // 2, L - 257, L - 256, L - 9, L - 1} | set(int(t) for t in rng.integers(0, L, 6)))
    worst = 0.0
    for t in rows:
        kc = np.ascontiguousarray(x.k[:t + 1].transpose(1, 0, 2))
        vc = np.ascontiguousarray(x.v[:t + 1].transpose(1, 0, 2))
        ref, _ = oracle.decode_attention(q_full[t], kc, vc)
        err = np.abs(got[t] - ref)
        worst = max(worst, float(err.max()))
        assert np.all(err <= O_RTOL * np.abs(ref) + O_ATOL), (t, float(err.max()))
    print("128k prefill attention: worst abs output error on %d sampled rows %.3e" % (len(rows), worst))
