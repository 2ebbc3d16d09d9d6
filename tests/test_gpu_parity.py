"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle on the same seeded bytes."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2502_01068_b200 import binding as B
from paper_2502_01068_b200 import workloads as W
from tests.parity import check_layer, gpu_layer, oracle_layer

pytestmark = pytest.mark.gpu


def small(name, cfg, lens, k_kv, k_tsp, Hq=8, Hkv=2, d=128, hidden=256, w=8, p=7, **kw):
    return W.Workload(name=name, cfg=cfg, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, hidden_dim=hidden,
                      window=w, pool_kernel=p, pool_mode=W.POOL_AVG, seq_lens=list(lens), k_kv=list(k_kv),
                      k_tsp=None if k_tsp is None else list(k_tsp), **kw)


@pytest.mark.parametrize("pool_mode", [B.POOL_AVG, B.POOL_MAX])
@pytest.mark.parametrize("agg_order", [B.GROUP_THEN_POOL, B.POOL_THEN_GROUP])
def test_tiny_config(pool_mode, agg_order):
    wl = W.tiny()
    x = W.make_layer(wl)
    g = gpu_layer(wl, x, pool_mode=pool_mode, agg_order=agg_order)
    o = oracle_layer(wl, x, pool_mode=pool_mode, agg_order=agg_order)
    check_layer(wl, x, g, o, what="tiny")
    # one KV head and equal budgets: KV selection and TSP selection coincide
    np.testing.assert_array_equal(g["idx_kv"][0], g["idx_tsp"])


@pytest.mark.parametrize("L,d,Hq,Hkv,w", [(100, 64, 4, 1, 8), (129, 128, 8, 2, 8), (1000, 128, 8, 2, 8),
                                           (777, 64, 16, 2, 8), (2500, 128, 8, 8, 8), (640, 128, 8, 2, 16),
                                           (300, 128, 4, 4, 8), (515, 64, 6, 2, 5), (8, 64, 4, 1, 8)])
def test_odd_shapes(L, d, Hq, Hkv, w):
    k_kv = max(w, min(L, L // 3 + w))
    wl = small("odd", 100 + L, [L], [k_kv], [max(w, L // 5)], Hq=Hq, Hkv=Hkv, d=d, w=w)
    x = W.make_layer(wl)
    g = gpu_layer(wl, x)
    o = oracle_layer(wl, x)
    check_layer(wl, x, g, o, what="odd L=%d" % L)


def test_no_forced_window_and_pool_kernels():
    for p in (1, 3, 9):
        wl = small("nofw", 300 + p, [1500], [400], [123], p=p)
        x = W.make_layer(wl)
        for fw in (True, False):
            g = gpu_layer(wl, x, force_window=fw, pool_mode=B.POOL_MAX)
            o = oracle_layer(wl, x, force_window=fw, pool_mode=B.POOL_MAX)
            check_layer(wl, x, g, o, force_window=fw, what="p=%d fw=%d" % (p, fw))


def test_ragged_batch_small():
    lens = [700, 8, 129, 2048, 300]
    wl = small("rag", 400, lens, [64, 8, 100, 256, 77], [140, 8, 25, 409, 60])
    x = W.make_layer(wl)
    g = gpu_layer(wl, x)
    o = oracle_layer(wl, x)
    check_layer(wl, x, g, o, what="ragged")
    # the cu_seqlens / cu_k form of the interface on a single sequence gives the same answer
    wl1 = small("rag1", 401, [900], [100], [180])
    x1 = W.make_layer(wl1)
    g1 = gpu_layer(wl1, x1, ragged_api=True)
    g0 = gpu_layer(wl1, x1, ragged_api=False)
    for key in ("S_kv", "idx_kv", "idx_tsp", "k_out", "hidden_out", "pos_out"):
        np.testing.assert_array_equal(g1[key], g0[key])


def test_deterministic_across_runs():
    wl = small("det", 500, [5000], [700], [1000])
    x = W.make_layer(wl)
    a = gpu_layer(wl, x)
    b = gpu_layer(wl, x, fused_select=False)        # separate select calls give the same indices
    for key in ("S_kv", "S_tsp", "idx_kv", "idx_tsp", "k_out", "v_out", "hidden_out", "pos_out"):
        np.testing.assert_array_equal(a[key], b[key])


def test_llama8b_8k():
    wl = W.llama8b_8k()
    x = W.make_layer(wl)
    g = gpu_layer(wl, x)
    o = oracle_layer(wl, x)
    st = check_layer(wl, x, g, o, what="8k")
    assert st["score_err"] < 2e-3


@pytest.mark.parametrize("path", [1, 2, 3])
def test_every_scoring_kernel_matches(debug_hooks, path):
    """The library picks one of three scoring kernels by shape: (3) logits parked in tensor memory,
    (2) K read a second time from L2, (1) fp32 logits buffered in the workspace.  Each of them, forced
    through the score_path hook, must match the oracle on the same layers."""
    debug_hooks("score_path", path)
    for wl in (W.tiny(), small("buf", 600, [3000, 130, 1000], [300, 64, 200], [500, 20, 100])):
        x = W.make_layer(wl)
        for order in (B.GROUP_THEN_POOL, B.POOL_THEN_GROUP):
            g = gpu_layer(wl, x, pool_mode=B.POOL_MAX, agg_order=order)
            o = oracle_layer(wl, x, pool_mode=B.POOL_MAX, agg_order=order)
            check_layer(wl, x, g, o, what="path %d" % path)


def test_sequence_longer_than_half_the_tensor_memory_ring(debug_hooks):
    """L = 160 000: a CTA owns 9 tiles per phase, more than half of the 16 parked slots, so the statistics of a
    phase cannot hide behind a whole next phase; the library still picks the parked kernel (it is the faster one up
    to the ring), and every scoring kernel, forced, gives the same result up to rounding."""
    wl = small("long", 601, [160000], [4000], [8000], Hq=4, Hkv=1, d=64, hidden=64)
    x = W.make_layer(wl)
    o = oracle_layer(wl, x)
    check_layer(wl, x, gpu_layer(wl, x), o, what="160k")
    for path in (3, 2):
        debug_hooks("score_path", path)
        check_layer(wl, x, gpu_layer(wl, x), o, what="160k, path %d" % path)


def test_parked_kernel_at_the_edge_of_its_ring(debug_hooks):
    """148 CTAs x 16 slots x 128 keys = 303 104 keys is the most the parked kernel can hold per phase:
    every slot of the ring is in use at once."""
    debug_hooks("score_path", 3)
    wl = small("edge", 602, [303000], [4000], [8000], Hq=4, Hkv=1, d=64, hidden=64)
    x = W.make_layer(wl)
    g = gpu_layer(wl, x)
    o = oracle_layer(wl, x)
    check_layer(wl, x, g, o, what="303k parked")
    # beyond that the parked kernel cannot run: refused on the host
    shape = B.make_shape(total_len=310000, n_q_heads=4, n_kv_heads=1, head_dim=64)
    with pytest.raises(B.FastKVError) as e:
        B.fastkv_workspace_bytes(shape)
    assert e.value.status == B.ERR_UNSUPPORTED


def test_batch_scored_side_by_side_in_several_waves(debug_hooks):
    """A batch on the parked kernel: its sequences are scored side by side, each by its share of the CTAs, in as
    many waves as the tensor-memory ring needs (here three: {0, 1}, {2, 3}, {4}); one sequence is much shorter
    than the others, one wave has CTAs left over."""
    lens = [150000, 90000, 200000, 4000, 120000]
    wl = small("waves", 603, lens, [4000] * 5, [8000, 8000, 8000, 800, 8000], Hq=4, Hkv=1, d=64, hidden=64)
    x = W.make_layer(wl)
    o = oracle_layer(wl, x)
    check_layer(wl, x, gpu_layer(wl, x), o, what="five sequences, the library's choice")
    debug_hooks("score_path", 3)
    check_layer(wl, x, gpu_layer(wl, x), o, what="five sequences, parked kernel")


@pytest.mark.parametrize("L", [700, 40000, 100000])
def test_single_sequence_with_its_heads_side_by_side(debug_hooks, L):
    """The parked kernel with one KV head per share of the CTAs (what the library picks for 24K .. 113K tokens at
    the 8B head shape), forced on short, middling and long single sequences; G = 2, four KV heads."""
    debug_hooks("score_path", 3)
    debug_hooks("score_partition", 2)
    wl = small("heads_side_by_side", 604, [L], [2000 if L > 2000 else 300], [4000 if L > 4000 else 200], Hq=8, Hkv=4, d=64, hidden=64)
    x = W.make_layer(wl)
    for order in (B.GROUP_THEN_POOL, B.POOL_THEN_GROUP):
        check_layer(wl, x, gpu_layer(wl, x, agg_order=order), oracle_layer(wl, x, agg_order=order), what="L=%d order %d" % (L, order))


@pytest.mark.parametrize("path", [2, 3])
def test_group_sizes_and_wide_windows_on_the_persistent_kernels(debug_hooks, path):
    debug_hooks("score_path", path)
    for Hq, Hkv, w in [(8, 8, 8), (16, 8, 8), (16, 2, 8), (8, 2, 16), (4, 1, 16), (12, 4, 8)]:
        wl = small("grp", 700 + Hq + Hkv + w, [2000], [300], [400], Hq=Hq, Hkv=Hkv, w=w)
        x = W.make_layer(wl)
        for order in (B.GROUP_THEN_POOL, B.POOL_THEN_GROUP):
            g = gpu_layer(wl, x, agg_order=order, pool_mode=B.POOL_MAX)
            o = oracle_layer(wl, x, agg_order=order, pool_mode=B.POOL_MAX)
            check_layer(wl, x, g, o, what="G=%d w=%d order=%d" % (Hq // Hkv, w, order))


@pytest.mark.parametrize("path", [2, 3])
@pytest.mark.parametrize("scale", [0.5, 2.0])
def test_wide_logit_range_exercises_reference_rescaling(debug_hooks, scale, path):
    """With a large softmax scale the logits span far more than the slack the kernel allows between a
    lane's reference and its running maximum, so stored exponentials get rescaled mid-phase.  Scores
    only (most of them underflow to zero on both sides, which makes the selection a tie lottery)."""
    import oracle
    from tests.parity import SCORE_RTOL, dev
    debug_hooks("score_path", path)
    for L, Hq, Hkv, d, w in [(5000, 8, 2, 128, 8), (1500, 4, 1, 64, 8), (20000, 8, 2, 128, 16)]:
        wl = small("wide", 800 + L, [L], [w], [w], Hq=Hq, Hkv=Hkv, d=d, w=w)
        x = W.make_layer(wl, with_v=False, with_hidden=False)
        shape = B.make_shape(total_len=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, window=w, softmax_scale=scale)
        ws = torch.empty(B.fastkv_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
        s_kv = torch.empty((Hkv, L), dtype=torch.float32, device="cuda")
        s_tsp = torch.empty((L,), dtype=torch.float32, device="cuda")
        B.fastkv_score(shape, dev(x.q_win), dev(x.k), s_kv, s_tsp, ws)
        assert B.fastkv_device_status(ws)[0] == 0
        ref_kv, ref_tsp, _ = oracle.scores(x.q_win, L - w, x.k, w, 7, scale=scale)
        got = s_kv.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - ref_kv) <= SCORE_RTOL * np.abs(ref_kv) + 1e-12)
        np.testing.assert_allclose(got.sum(axis=1), ref_kv.sum(axis=1), rtol=1e-5)
        assert np.all(np.abs(s_tsp.cpu().numpy() - ref_tsp) <= SCORE_RTOL * np.abs(ref_tsp) + 1e-12)


@pytest.mark.parametrize("heads,lead", [(1, 2), (2, 1000), (3, 2), (8, 3)])
def test_phase_shapes_of_the_rereading_kernel(debug_hooks, heads, lead):
    """The kernel that reads K twice cuts its work into phases of `heads` KV heads and lets pass 1 run
    `lead` phases ahead; the result must not depend on either (tuning hooks of the library)."""
    debug_hooks("score_path", 2)
    debug_hooks("fused_heads", heads)
    debug_hooks("fused_lead", lead)
    wl = small("phases", 900, [20000, 3000], [500, 100], [2000, 300], Hq=32, Hkv=8)
    x = W.make_layer(wl, with_hidden=False)
    g = gpu_layer(wl, x)
    o = oracle_layer(wl, x, do_compact=False)
    check_layer(wl, x, g, o, what="heads=%d lead=%d" % (heads, lead))


def test_sequence_shorter_than_the_window_is_reported_not_scored():
    """In a batch, a sequence with fewer tokens than the observation window has no defined scores: the
    scoring kernel skips it and raises the status word; the other sequences are unaffected."""
    lens = [300, 5, 700]
    wl = small("short", 950, lens, [40, 8, 60], [50, 8, 90])
    x = W.make_layer(wl, with_hidden=False)
    from tests.parity import dev
    cu = dev(x.cu_seqlens.astype(np.int32))
    shape = B.make_shape(total_len=sum(lens), n_q_heads=8, n_kv_heads=2, head_dim=128, batch=3, max_len=700,
                         cu_seqlens=cu)
    ws = torch.empty(B.fastkv_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    s_kv = torch.zeros((2, sum(lens)), dtype=torch.float32, device="cuda")
    B.fastkv_score(shape, dev(x.q_win), dev(x.k), s_kv, None, ws)
    status, site = B.fastkv_device_status(ws)
    assert status == B.ERR_INVALID_ARG
    import oracle
    got = s_kv.cpu().numpy()
    for b in (0, 2):
        lo, hi = int(x.cu_seqlens[b]), int(x.cu_seqlens[b + 1])
        ref, _, _ = oracle.scores(x.q_win[b * 8:(b + 1) * 8], hi - lo - 8, x.k[lo:hi], 8, 7)
        assert np.all(np.abs(got[:, lo:hi] - ref) <= 2e-3 * np.abs(ref) + 1e-12)


@pytest.mark.parametrize("path", [0, 1, 2, 3])
def test_full_query_tensor_layout(debug_hooks, path):
    """q_layout = FASTKV_Q_FULL: the caller hands over the whole packed query tensor [total, Hq, d] and the
    library reads rows cu_seqlens[b+1]-w .. cu_seqlens[b+1]-1 itself (Eq. 1's Att[h, N_I-n, .] rows).  Every
    other query row is random and must not matter: same oracle result as with the window-only layout."""
    debug_hooks("score_path", path)
    cases = [small("qfull1", 1100, [3000], [400], [600]),
             small("qfull2", 1101, [700, 8, 129, 2048, 300], [64, 8, 100, 256, 77], [140, 8, 25, 409, 60]),
             small("qfull3", 1102, [513], [100], [100], Hq=4, Hkv=1, d=64, w=5)]
    for wl in cases:
        x = W.make_layer(wl)
        o = oracle_layer(wl, x)
        g = gpu_layer(wl, x, q_layout=B.Q_FULL)
        check_layer(wl, x, g, o, what="%s Q_FULL path %d" % (wl.name, path))
        gw = gpu_layer(wl, x, q_layout=B.Q_WINDOW)
        np.testing.assert_array_equal(g["S_kv"], gw["S_kv"])          # same rows read, same arithmetic


def test_full_query_tensor_layout_at_8k():
    wl = W.llama8b_8k()
    x = W.make_layer(wl)
    g = gpu_layer(wl, x, q_layout=B.Q_FULL)
    o = oracle_layer(wl, x)
    check_layer(wl, x, g, o, what="8k Q_FULL")
