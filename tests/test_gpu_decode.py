"""GPU parity of the decode-time attention over the compact cache against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2502_01068_b200 import binding as B
from paper_2502_01068_b200 import workloads as W

pytestmark = pytest.mark.gpu

RTOL, ATOL = 2e-3, 2e-5      # bf16 inputs, fp32 accumulation; outputs are means of ~N(0,1) values


def run_decode(q, kc, vc, ks, Hq, Hkv, d, ragged, scale=0.0):
    Bn = len(ks)
    shape = B.make_shape(total_len=max(sum(ks), 8), n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, batch=Bn,
                         max_len=max(max(ks), 8) if Bn == 1 else max(ks),
                         cu_seqlens=torch.zeros(Bn + 1, dtype=torch.int32, device="cuda") if Bn > 1 else None,
                         softmax_scale=scale, force_window=False)
    t = lambda a: torch.from_numpy(a.view(np.int16)).cuda()
    if ragged:
        cu = torch.from_numpy(np.concatenate([[0], np.cumsum(ks)]).astype(np.int32)).cuda()
        bud = B.make_budget(0, cu_k=cu, total=int(sum(ks)))
    else:
        bud = B.make_budget(int(ks[0]), batch=Bn)
    ws = torch.zeros(B.fastkv_decode_attn_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    out = torch.full((Bn, Hq, d), 7.0, dtype=torch.float32, device="cuda")
    lse = torch.zeros((Bn, Hq), dtype=torch.float32, device="cuda")
    B.fastkv_decode_attn(shape, t(q), t(kc), t(vc), bud, out, lse, ws)
    assert B.fastkv_device_status(ws)[0] == 0
    return out.cpu().numpy(), lse.cpu().numpy()


@pytest.mark.parametrize("Hq,Hkv,d", [(32, 8, 128), (4, 1, 64), (8, 8, 128), (16, 2, 64), (6, 3, 128)])
@pytest.mark.parametrize("ks", [[13107], [1], [127], [129], [1000, 5, 128, 4097], [2048, 2048]])
def test_decode_attention_matches_the_oracle(Hq, Hkv, d, ks):
    rng = np.random.default_rng(Hq * 1000 + d + sum(ks))
    Bn, tot = len(ks), sum(ks)
    q = W.f32_to_bf16_bits(rng.standard_normal((Bn, Hq, d), dtype=np.float32))
    kc = W.f32_to_bf16_bits(rng.standard_normal((Hkv, tot, d), dtype=np.float32))
    vc = W.f32_to_bf16_bits(rng.standard_normal((Hkv, tot, d), dtype=np.float32))
    ragged = len(set(ks)) > 1
    got, got_lse = run_decode(q, kc, vc, ks, Hq, Hkv, d, ragged)
    cu = np.concatenate([[0], np.cumsum(ks)])
    for b in range(Bn):
        ref, ref_lse = oracle.decode_attention(q[b], kc[:, cu[b]:cu[b + 1]], vc[:, cu[b]:cu[b + 1]])
        assert np.all(np.abs(got[b] - ref) <= RTOL * np.abs(ref) + ATOL), np.abs(got[b] - ref).max()
        np.testing.assert_allclose(got_lse[b], ref_lse, rtol=1e-5, atol=1e-4)


def test_decode_attention_on_a_compacted_layer_and_with_peaked_softmax():
    """End to end: the cache is what fastkv_compact produced for the tiny config; and a large scale makes the
    softmax pick single keys (exercises the running-max rescaling across chunks)."""
    from tests.parity import gpu_layer
    wl = W.tiny()
    x = W.make_layer(wl)
    g = gpu_layer(wl, x)
    rng = np.random.default_rng(3)
    q = W.f32_to_bf16_bits(rng.standard_normal((1, wl.n_q_heads, wl.head_dim), dtype=np.float32))
    for scale in (0.0, 4.0):
        got, _ = run_decode(q, g["k_out"], g["v_out"], [128], wl.n_q_heads, wl.n_kv_heads, wl.head_dim, False, scale)
        ref, _ = oracle.decode_attention(q[0], g["k_out"], g["v_out"], scale=None if scale == 0.0 else scale)
        assert np.all(np.abs(got[0] - ref) <= RTOL * np.abs(ref) + ATOL)


def test_decode_attention_keeps_sequences_apart_when_a_neighbour_holds_nan():
    """A chunk of 16 cache rows can straddle two sequences: whatever the neighbour's rows hold (here NaN and
    infinity in K and V) must not reach this sequence's output."""
    Hq, Hkv, d, ks = 8, 2, 128, [21, 40, 3]
    rng = np.random.default_rng(77)
    q = W.f32_to_bf16_bits(rng.standard_normal((3, Hq, d), dtype=np.float32))
    kf = rng.standard_normal((Hkv, sum(ks), d), dtype=np.float32)
    vf = rng.standard_normal((Hkv, sum(ks), d), dtype=np.float32)
    kf[:, 21:61], vf[:, 21:61] = np.nan, np.inf          # the middle sequence is poisoned
    kc, vc = W.f32_to_bf16_bits(kf), W.f32_to_bf16_bits(vf)
    got, got_lse = run_decode(q, kc, vc, ks, Hq, Hkv, d, True)
    for b, (lo, hi) in ((0, (0, 21)), (2, (61, 64))):
        ref, ref_lse = oracle.decode_attention(q[b], kc[:, lo:hi], vc[:, lo:hi])
        assert np.all(np.abs(got[b] - ref) <= RTOL * np.abs(ref) + ATOL)
        np.testing.assert_allclose(got_lse[b], ref_lse, rtol=1e-5, atol=1e-4)


@pytest.mark.parametrize("seed", [31, 32, 33])
def test_decode_attention_on_random_shapes(seed):
    """Seeded random caches: KV heads, group size (1..8, odd ones included), head dimension, batch size and kept
    entries per sequence (empty caches, caches shorter than one 16-entry chunk, caches of thousands of entries), a
    random softmax scale; every sequence against its own oracle run."""
    rng = np.random.default_rng(seed)
    for it in range(6):
        Hkv = int(rng.choice([1, 2, 3, 8])); G = int(rng.integers(1, 9)); d = int(rng.choice([64, 128]))
        Bn = int(rng.integers(1, 6))
        ks = [int(rng.choice([0, 1, 15, 16, 17, int(rng.integers(18, 400)), int(rng.integers(400, 6000))])) for _ in range(Bn)]
        if sum(ks) == 0:
            ks[0] = 33
        if Bn == 1 or len(set(ks)) == 1:
            ks = [max(ks[0], 1)] * Bn                      # the uniform form of the budget
        scale = float(rng.choice([0.0, 0.05, 0.5]))
        Hq, tot = Hkv * G, sum(ks)
        q = W.f32_to_bf16_bits(rng.standard_normal((Bn, Hq, d), dtype=np.float32))
        kc = W.f32_to_bf16_bits(rng.standard_normal((Hkv, tot, d), dtype=np.float32))
        vc = W.f32_to_bf16_bits(rng.standard_normal((Hkv, tot, d), dtype=np.float32))
        ragged = len(set(ks)) > 1
        got, got_lse = run_decode(q, kc, vc, ks, Hq, Hkv, d, ragged, scale)
        cu = np.concatenate([[0], np.cumsum(ks)])
        for b in range(Bn):
            if ks[b] == 0:
                assert np.all(got[b] == 0.0), (seed, it, b)   # an empty cache: the output is defined as zero
                continue
            ref, ref_lse = oracle.decode_attention(q[b], kc[:, cu[b]:cu[b + 1]], vc[:, cu[b]:cu[b + 1]],
                                                   scale=None if scale == 0.0 else scale)
            err = np.abs(got[b] - ref)
            assert np.all(err <= RTOL * np.abs(ref) + ATOL), (seed, it, b, Hkv, G, d, ks, float(err.max()))
            np.testing.assert_allclose(got_lse[b], ref_lse, rtol=1e-5, atol=1e-4)
