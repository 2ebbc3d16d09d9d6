"""Pins for the fp64 oracle: each of its routines is checked against something that is not
itself -- a library routine on the plain definition, a closed form, an invariant, or brute
force on tiny inputs -- chosen so that a dropped term, a wrong index or sign, or a transposed
operand fails at least one of them."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle.layer import layer_step
from paper_2502_01068_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16(x):
    return W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def f64(bits):
    return W.bf16_bits_to_f32(bits).astype(np.float64)


def rand_qk(seed, L, H, Hkv, d):
    rng = np.random.default_rng(seed)
    return bf16(rng.standard_normal((L, H, d))), bf16(rng.standard_normal((L, Hkv, d)))


def torch_window_attention(q_bits, k_bits, w):
    """Eq. 1's inner term by the textbook route: full causal softmax attention matrix through
    torch.softmax (fp64), then the sum of its last w rows."""
    q = torch.from_numpy(f64(q_bits))                 # [L, H, d]
    k = torch.from_numpy(f64(k_bits))                 # [L, Hkv, d]
    L, H, d = q.shape
    G = H // k.shape[1]
    k = k.repeat_interleave(G, dim=1)                 # query head h reads KV head h // G
    logits = torch.einsum("thd,ihd->hti", q, k) / math.sqrt(d)
    mask = torch.ones(L, L, dtype=torch.bool).tril()
    att = torch.softmax(logits.masked_fill(~mask, float("-inf")), dim=-1)
    return att[:, L - w:, :].sum(dim=1).numpy(), att.numpy()


@pytest.mark.parametrize("L,H,Hkv,d,w", [(96, 4, 2, 16, 5), (40, 6, 3, 8, 8), (17, 2, 2, 32, 1),
                                         (9, 4, 1, 8, 9)])
def test_window_attention_matches_full_causal_softmax(L, H, Hkv, d, w):
    q, k = rand_qk(L * 7 + w, L, H, Hkv, d)
    ref, att = torch_window_attention(q, k, w)
    A_full = oracle.window_attention(q, 0, k, w)
    A_win = oracle.window_attention(q[L - w:], L - w, k, w)
    np.testing.assert_allclose(A_full, ref, rtol=0, atol=1e-13)
    np.testing.assert_array_equal(A_full, A_win)
    A_bf, att_bf = oracle.full_attention_window(q, k, w, want_matrix=True)
    np.testing.assert_allclose(A_bf, ref, rtol=0, atol=1e-13)
    np.testing.assert_allclose(att_bf, att, rtol=0, atol=1e-13)


def test_window_rows_sum_to_one_and_group_mass():
    L, H, Hkv, d, w = 300, 8, 2, 32, 8
    q, k = rand_qk(3, L, H, Hkv, d)
    A = oracle.window_attention(q[L - w:], L - w, k, w)
    np.testing.assert_allclose(A.sum(axis=1), w, rtol=0, atol=1e-12)
    S_kv, S_tsp, _ = oracle.scores(q[L - w:], L - w, k, w, 1)          # p = 1: no pooling
    np.testing.assert_allclose(S_kv.sum(axis=1), w * (H // Hkv), rtol=0, atol=1e-12)
    np.testing.assert_allclose(S_tsp.sum(), w * H, rtol=0, atol=1e-11)
    # causal mask inside the window: key L-1 is seen by the last query only, key L-w by all
    assert np.all(A[:, L - 1] <= 1.0) and np.all(A[:, L - 1] > 0)


def test_uniform_attention_closed_form_and_golden():
    """All keys equal => every visible key gets 1/(t+1) from query position t, so
    A[h,i] = sum_{j : t_j >= i} 1/(t_j+1) exactly (Eq. 1 with a flat softmax)."""
    L, H, Hkv, d, w = 16, 4, 2, 8, 4
    rng = np.random.default_rng(0)
    q = bf16(rng.standard_normal((L, H, d)))
    k = np.broadcast_to(bf16(rng.standard_normal((1, Hkv, d))), (L, Hkv, d)).copy()
    A = oracle.window_attention(q[L - w:], L - w, k, w)
    expect = np.array([float(sum(Fraction(1, t + 1) for t in range(L - w, L) if t >= i))
                       for i in range(L)])
    for h in range(H):
        np.testing.assert_allclose(A[h], expect, rtol=0, atol=1e-14)
    # the same closed form stored as exact rationals (written by tests/golden/make_uniform.py)
    with open(os.path.join(GOLDEN, "uniform_attention_L16_w4.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    gold = np.array([float(Fraction(r[1])) for r in rows])
    assert [int(r[0]) for r in rows] == list(range(L))
    np.testing.assert_allclose(A[0], gold, rtol=0, atol=1e-14)


def test_single_planted_key_closed_form():
    """Every window query equals u, one prefix key equals c*u, all other keys are zero:
    the logit is s = c*|u|^2/sqrt(d) at the plant and 0 elsewhere, so
    A[h, i*] = sum_j e^s / (e^s + t_j) and every other visible key gets 1 / (e^s + t_j)."""
    L, H, Hkv, d, w, istar, c = 64, 4, 2, 16, 8, 11, 2.0
    u = np.zeros(d); u[:4] = [1.0, -2.0, 0.5, 1.5]
    q = np.broadcast_to(bf16(u), (w, H, d)).copy()
    k = np.zeros((L, Hkv, d), dtype=np.uint16)
    k[istar] = bf16(c * u)
    A = oracle.window_attention(q, L - w, k, w)
    s = c * float(u @ u) / math.sqrt(d)
    ts = np.arange(L - w, L)
    np.testing.assert_allclose(A[:, istar], np.sum(np.exp(s) / (np.exp(s) + ts)), rtol=1e-13)
    np.testing.assert_allclose(A[:, 0], np.sum(1.0 / (np.exp(s) + ts)), rtol=1e-13)
    # last key is visible to the last query only
    np.testing.assert_allclose(A[:, L - 1], 1.0 / (np.exp(s) + (L - 1)), rtol=1e-13)
    # a strong plant takes all the mass: -> w
    k[istar] = bf16(40.0 * u)
    assert abs(oracle.window_attention(q, L - w, k, w)[0, istar] - w) < 1e-9


def test_softmax_shift_and_prefix_permutation_invariance():
    L, H, Hkv, d, w = 50, 4, 2, 8, 6
    rng = np.random.default_rng(5)
    qi = rng.integers(-3, 4, (w, H, d)).astype(np.float32)
    ki = rng.integers(-4, 5, (L, Hkv, d)).astype(np.float32)
    v = rng.integers(-2, 3, (1, Hkv, d)).astype(np.float32)      # small integers: exact in bf16
    A0 = oracle.window_attention(bf16(qi), L - w, bf16(ki), w)
    A1 = oracle.window_attention(bf16(qi), L - w, bf16(ki + v), w)
    np.testing.assert_allclose(A1, A0, rtol=0, atol=1e-12)
    perm = np.concatenate([rng.permutation(L - w), np.arange(L - w, L)])
    A2 = oracle.window_attention(bf16(qi), L - w, bf16(ki[perm]), w)
    np.testing.assert_allclose(A2, A0[:, perm], rtol=0, atol=1e-13)


def test_scale_argument_and_default():
    L, H, Hkv, d, w = 30, 2, 1, 16, 4
    q, k = rand_qk(9, L, H, Hkv, d)
    A_def = oracle.window_attention(q[L - w:], L - w, k, w)
    A_exp = oracle.window_attention(q[L - w:], L - w, k, w, scale=0.25)
    np.testing.assert_array_equal(A_def, A_exp)                 # default is 1/sqrt(d)
    A_zero = oracle.window_attention(q[L - w:], L - w, k, w, scale=0.0)
    expect = np.array([sum(1.0 / (t + 1) for t in range(L - w, L) if t >= i) for i in range(L)])
    np.testing.assert_allclose(A_zero[0], expect, rtol=0, atol=1e-14)


@pytest.mark.parametrize("p", [1, 3, 7, 9])
def test_pool_matches_library_pooling(p):
    rng = np.random.default_rng(p)
    x = rng.random((5, 41))
    t = torch.from_numpy(x)[None]
    avg = torch.nn.functional.avg_pool1d(t, p, stride=1, padding=p // 2, count_include_pad=True)[0]
    mx = torch.nn.functional.max_pool1d(t, p, stride=1, padding=p // 2)[0]
    np.testing.assert_allclose(oracle.pool1d(x, p, oracle.POOL_AVG), avg.numpy(), rtol=0, atol=1e-15)
    np.testing.assert_array_equal(oracle.pool1d(x, p, oracle.POOL_MAX), mx.numpy())
    if p == 1:
        np.testing.assert_array_equal(oracle.pool1d(x, 1, oracle.POOL_AVG), x)
        np.testing.assert_array_equal(oracle.pool1d(x, 1, oracle.POOL_MAX), x)


def test_pool_identities():
    rng = np.random.default_rng(2)
    L, p = 37, 7
    x = rng.random((3, L))
    avg = oracle.pool1d(x, p, oracle.POOL_AVG)
    # mass identity: interior positions are counted p times, the 3 at each edge 4, 5, 6 times
    c = np.full(L, float(p)); c[:3] = [4, 5, 6]; c[-3:] = [6, 5, 4]
    np.testing.assert_allclose(avg.sum(axis=1), (x * c).sum(axis=1) / p, rtol=1e-13)
    mx = oracle.pool1d(x, p, oracle.POOL_MAX)
    assert np.all(mx >= x)
    np.testing.assert_array_equal(oracle.pool1d(np.full((1, L), 0.3), p, oracle.POOL_MAX),
                                  np.full((1, L), 0.3))
    # an isolated spike spreads to exactly p positions under MAX and contributes 1/p under AVG
    e = np.zeros((1, L)); e[0, 10] = 2.0
    assert np.flatnonzero(oracle.pool1d(e, p, oracle.POOL_MAX)[0]).tolist() == list(range(7, 14))
    np.testing.assert_allclose(oracle.pool1d(e, p, oracle.POOL_AVG)[0, 7:14], 2.0 / p)


def test_scores_composition_and_order():
    L, H, Hkv, d, w, p = 120, 8, 2, 16, 8, 7
    G = H // Hkv
    q, k = rand_qk(11, L, H, Hkv, d)
    A = oracle.window_attention(q[L - w:], L - w, k, w)
    for mode in (oracle.POOL_AVG, oracle.POOL_MAX):
        S_kv, S_tsp, A_out = oracle.scores(q[L - w:], L - w, k, w, p, mode,
                                           oracle.GROUP_THEN_POOL, want_A=True)
        np.testing.assert_array_equal(A_out, A)
        a = A.reshape(Hkv, G, L).sum(axis=1)
        np.testing.assert_allclose(S_kv, oracle.pool1d(a, p, mode), rtol=0, atol=1e-15)
        np.testing.assert_allclose(S_tsp, S_kv.sum(axis=0), rtol=0, atol=1e-15)
        S_kv2, S_tsp2, _ = oracle.scores(q[L - w:], L - w, k, w, p, mode, oracle.POOL_THEN_GROUP)
        np.testing.assert_allclose(S_kv2, oracle.pool1d(A, p, mode).reshape(Hkv, G, L).sum(axis=1),
                                   rtol=0, atol=1e-15)
        if mode == oracle.POOL_AVG:      # linear pooling commutes with the group sum
            np.testing.assert_allclose(S_kv2, S_kv, rtol=0, atol=1e-14)
        else:                            # max of sums <= sum of maxes
            assert np.all(S_kv2 >= S_kv - 1e-15) and np.any(S_kv2 > S_kv + 1e-9)
    # a single KV head: the layer-level score is that head's score
    q1, k1 = rand_qk(12, L, 4, 1, d)
    S_kv, S_tsp, _ = oracle.scores(q1[L - w:], L - w, k1, w, p)
    np.testing.assert_array_equal(S_tsp, S_kv[0])


def brute_force_select(S, k, w, force_window):
    """Repeatedly take the best remaining candidate (largest score, lowest index on ties)."""
    L = len(S)
    cand = list(range(L - w)) if force_window else list(range(L))
    chosen = []
    for _ in range(k - w if force_window else k):
        best = cand[0]
        for i in cand:
            if S[i] > S[best]:
                best = i
        chosen.append(best)
        cand.remove(best)
    if force_window:
        chosen += list(range(L - w, L))
    return sorted(chosen), (S[chosen[(k - w if force_window else k) - 1]] if chosen else None)


@pytest.mark.parametrize("force_window", [True, False])
def test_select_matches_brute_force_with_ties(force_window):
    rng = np.random.default_rng(4)
    for trial in range(30):
        L = int(rng.integers(12, 60)); w = int(rng.integers(1, 6))
        S = rng.integers(0, 6, L).astype(np.float64) / 4.0          # many exact ties
        lo = w + 1 if force_window else 1
        k = int(rng.integers(lo, L + 1))
        idx, tau = oracle.select(S, k, w, force_window)
        ref, ref_tau = brute_force_select(S, k, w, force_window)
        assert idx.tolist() == ref
        assert tau == ref_tau
        assert len(set(idx.tolist())) == k and np.all(np.diff(idx) > 0)
        if force_window:
            assert idx[-w:].tolist() == list(range(L - w, L))


def test_select_special_cases():
    rng = np.random.default_rng(6)
    L, w = 50, 8
    S = rng.random(L)
    idx, tau = oracle.select(S, w, w, True)                         # k = w: the window alone
    assert idx.tolist() == list(range(L - w, L)) and tau == math.inf
    idx, _ = oracle.select(S, L, w, True)                           # k = L: identity
    assert idx.tolist() == list(range(L))
    idx, _ = oracle.select(np.full(L, 0.5), 20, w, True)            # all equal: lowest indices win
    assert idx.tolist() == list(range(12)) + list(range(L - w, L))
    # no ties: the definition is a stable argsort (library routine)
    k = 17
    idx, tau = oracle.select(S, k, w, False)
    order = np.argsort(-S, kind="stable")[:k]
    assert idx.tolist() == sorted(order.tolist()) and tau == S[order[-1]]
    # a window position with a huge score is not ranked when the window is forced in
    S2 = S.copy(); S2[L - 2] = 100.0
    idx_a, _ = oracle.select(S, 20, w, True)
    idx_b, _ = oracle.select(S2, 20, w, True)
    assert idx_a.tolist() == idx_b.tolist()
    with pytest.raises(ValueError):
        oracle.select(S, w - 1, w, True)
    with pytest.raises(ValueError):
        oracle.select(S, L + 1, w, False)


def test_gather_is_numpy_indexing():
    rng = np.random.default_rng(8)
    src = rng.integers(0, 65536, (40, 3, 16)).astype(np.uint16)
    idx = np.sort(rng.choice(40, 13, replace=False))
    np.testing.assert_array_equal(oracle.gather_rows(src, idx), src[idx])
    np.testing.assert_array_equal(oracle.gather_rows(src[:, 1, :], idx), src[idx, 1, :])   # strided rows
    np.testing.assert_array_equal(oracle.gather_rows(src, np.arange(40)), src)
    pos = np.arange(40, dtype=np.int32) * 3
    np.testing.assert_array_equal(oracle.gather_rows(pos, idx), pos[idx])


def test_layer_step_tiny_config_and_planted_recovery():
    wl = W.tiny()
    x = W.make_layer(wl)
    r = layer_step(x.q_win, x.k, x.v, x.hidden, x.pos, x.cu_seqlens, wl.window, wl.pool_kernel,
                   wl.k_kv, wl.k_tsp)
    L, w = wl.seq_lens[0], wl.window
    # one KV head and equal budgets: both selections are the same set
    np.testing.assert_array_equal(r["idx_kv"][0], r["idx_tsp"])
    assert r["idx_tsp"].shape == (128,) and np.all(np.diff(r["idx_tsp"]) > 0)
    assert r["idx_tsp"][-w:].tolist() == list(range(L - w, L))
    np.testing.assert_array_equal(r["k_out"][0], x.k[r["idx_kv"][0], 0])
    np.testing.assert_array_equal(r["v_out"][0], x.v[r["idx_kv"][0], 0])
    np.testing.assert_array_equal(r["hidden_out"], x.hidden[r["idx_tsp"]])
    np.testing.assert_array_equal(r["pos_out"], r["idx_tsp"].astype(np.int32))
    # a strong plant (several nats above the bulk) is always recovered, under both poolings
    import dataclasses
    strong = dataclasses.replace(wl, plant_gain=3.0 * math.sqrt(wl.head_dim))
    xs = W.make_layer(strong)
    for mode in (oracle.POOL_AVG, oracle.POOL_MAX):
        rs = layer_step(xs.q_win, xs.k, None, None, None, xs.cu_seqlens, w, wl.pool_kernel,
                        wl.k_kv, wl.k_tsp, pool_mode=mode, do_compact=False)
        assert np.isin(xs.planted[0], rs["idx_tsp"]).all()
        assert np.isin(xs.planted[0], rs["idx_kv"][0]).all()


def test_layer_step_ragged_batch_equals_per_sequence_runs():
    wl = W.Workload(name="r", cfg=77, n_q_heads=4, n_kv_heads=2, head_dim=16, hidden_dim=32,
                    window=4, pool_kernel=7, pool_mode=W.POOL_AVG, seq_lens=[37, 9, 64],
                    k_kv=[10, 5, 12], k_tsp=[8, 9, 20])
    x = W.make_layer(wl)
    r = layer_step(x.q_win, x.k, x.v, x.hidden, x.pos, x.cu_seqlens, wl.window, wl.pool_kernel,
                   wl.k_kv, wl.k_tsp)
    cu = x.cu_seqlens
    for b in range(3):
        lo, hi = cu[b], cu[b + 1]
        one = layer_step(x.q_win[b * 4:(b + 1) * 4], x.k[lo:hi], x.v[lo:hi], x.hidden[lo:hi],
                         x.pos[lo:hi], np.array([0, hi - lo]), wl.window, wl.pool_kernel,
                         [wl.k_kv[b]], [wl.k_tsp[b]])
        np.testing.assert_array_equal(r["S_kv"][:, lo:hi], one["S_kv"])
        a, e = r["cu_k_tsp"][b], r["cu_k_tsp"][b + 1]
        np.testing.assert_array_equal(r["idx_tsp"][a:e], one["idx_tsp"])
        np.testing.assert_array_equal(r["hidden_out"][a:e], one["hidden_out"])
        np.testing.assert_array_equal(r["pos_out"][a:e], one["pos_out"])
        a, e = r["cu_k_kv"][b], r["cu_k_kv"][b + 1]
        np.testing.assert_array_equal(r["k_out"][:, a:e], one["k_out"])


def test_decode_attention_matches_library_attention_and_closed_forms():
    """The decode step over the compressed cache is plain softmax attention of one query token: pinned
    against torch's scaled_dot_product_attention in fp64 and against two closed forms."""
    rng = np.random.default_rng(21)
    H, Hkv, d, k = 8, 2, 16, 37
    q = bf16(rng.standard_normal((H, d)))
    kc = bf16(rng.standard_normal((Hkv, k, d)))
    vc = bf16(rng.standard_normal((Hkv, k, d)))
    out, lse = oracle.decode_attention(q, kc, vc)
    G = H // Hkv
    tq = torch.from_numpy(f64(q))[None, :, None, :]                               # [1, H, 1, d]
    tk = torch.from_numpy(f64(kc)).repeat_interleave(G, dim=0)[None]              # head h reads group h // G
    tv = torch.from_numpy(f64(vc)).repeat_interleave(G, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[0, :, 0, :].numpy()
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-13)
    logits = torch.einsum("hd,hkd->hk", tq[0, :, 0, :], tk[0]) / math.sqrt(d)
    np.testing.assert_allclose(lse, torch.logsumexp(logits, dim=-1).numpy(), rtol=0, atol=1e-13)
    # all keys equal: the output is the mean of the values
    kc_same = np.broadcast_to(kc[:, :1, :], kc.shape).copy()
    out_u, lse_u = oracle.decode_attention(q, kc_same, vc)
    np.testing.assert_allclose(out_u, np.repeat(f64(vc).mean(axis=1), G, axis=0), rtol=0, atol=1e-13)
    # one key aligned with the query and far above the rest: the output is that key's value row
    kc_hot = np.zeros_like(kc); kc_hot[:, 5, :] = bf16(40.0 * f64(q)[::G])
    out_h, _ = oracle.decode_attention(q[::G].repeat(G, axis=0), kc_hot, vc)
    np.testing.assert_allclose(out_h, np.repeat(f64(vc)[:, 5, :], G, axis=0), rtol=0, atol=1e-9)
    # permuting cache entries (K and V together) changes nothing
    perm = rng.permutation(k)
    out_p, lse_p = oracle.decode_attention(q, kc[:, perm], vc[:, perm])
    np.testing.assert_allclose(out_p, out, rtol=0, atol=1e-13)
    np.testing.assert_allclose(lse_p, lse, rtol=0, atol=1e-13)


@pytest.mark.parametrize("L,H,Hkv,d", [(70, 4, 2, 16), (33, 6, 3, 8), (9, 2, 2, 32)])
def test_prefill_attention_matches_library_attention_and_closed_forms(L, H, Hkv, d):
    """The layer's own causal attention (whose matrix the saliency scores are read off): pinned against
    torch's scaled_dot_product_attention in fp64, against the matrix-times-values product of the
    brute-force attention matrix, and against closed forms."""
    rng = np.random.default_rng(100 + L)
    q, k = rand_qk(L + 3, L, H, Hkv, d)
    v = bf16(rng.standard_normal((L, Hkv, d)))
    O = oracle.prefill_attention(q, k, v)
    G = H // Hkv
    tq = torch.from_numpy(f64(q)).permute(1, 0, 2)[None]                          # [1, H, L, d]
    tk = torch.from_numpy(f64(k)).repeat_interleave(G, dim=1).permute(1, 0, 2)[None]
    tv = torch.from_numpy(f64(v)).repeat_interleave(G, dim=1).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(O, ref, rtol=0, atol=1e-13)
    # the same through the explicit attention matrix (torch.softmax route of the window pin)
    _, att = torch_window_attention(q, k, 1)                                       # [H, L, L]
    vv = f64(v).repeat(G, axis=1)                                                  # [L, H, d]
    np.testing.assert_allclose(O, np.einsum("hti,ihd->thd", att, vv), rtol=0, atol=1e-13)
    # the first token attends to itself only
    np.testing.assert_allclose(O[0], vv[0], rtol=0, atol=1e-15)
    # all value rows equal: the output is that row, whatever the weights
    v_same = np.broadcast_to(v[:1], v.shape).copy()
    np.testing.assert_allclose(oracle.prefill_attention(q, k, v_same), np.broadcast_to(vv[:1], O.shape), rtol=0, atol=1e-13)
    # zero queries: uniform causal weights, the output is the running mean of the values
    O_u = oracle.prefill_attention(np.zeros_like(q), k, v)
    run_mean = np.cumsum(vv, axis=0) / np.arange(1, L + 1)[:, None, None]
    np.testing.assert_allclose(O_u, run_mean, rtol=0, atol=1e-13)
    # a different scale changes the result the way the definition says (scale 0 = uniform weights)
    np.testing.assert_allclose(oracle.prefill_attention(q, k, v, scale=1e-30), run_mean, rtol=0, atol=1e-12)
    # one key far above the rest for every query after it: the output is that key's value row
    star = L // 3
    q_hot = np.broadcast_to(q[:1, ::G].repeat(G, axis=1), q.shape).copy()          # every position and every head of a group asks the same
    k_hot = np.zeros_like(k)
    k_hot[star] = bf16(60.0 * f64(q)[0, ::G])
    O_h = oracle.prefill_attention(q_hot, k_hot, v)
    np.testing.assert_allclose(O_h[star:], np.broadcast_to(vv[star], O_h[star:].shape), rtol=0, atol=1e-9)
    np.testing.assert_allclose(O_h[:star], run_mean[:star], rtol=0, atol=1e-13)   # before it: all logits are 0
