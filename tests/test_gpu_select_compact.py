"""GPU tests of the selection and compaction kernels on their own, fed with scores / indices chosen to
stress ties, budgets at their limits, ragged offsets, strides and bad indices.  Selection on fp32
scores is integer work: results must equal the oracle's full-sort definition bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2502_01068_b200 import binding as B

pytestmark = pytest.mark.gpu


def run_select(S: np.ndarray, lens, ks, w, force_window=True, rows=1, ragged=None):
    """S is [rows, total] fp32; returns idx [rows, sum k] from fastkv_select_kv (rows > 1) or _tsp."""
    total = int(sum(lens))
    Bn = len(lens)
    ragged = (Bn > 1) if ragged is None else ragged
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    d_cu = torch.from_numpy(cu).cuda() if ragged else None
    shape = B.make_shape(total_len=total, n_q_heads=rows, n_kv_heads=rows, head_dim=128, window=w,
                         force_window=force_window, batch=Bn, max_len=max(lens), cu_seqlens=d_cu)
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    dS = torch.from_numpy(np.ascontiguousarray(S, dtype=np.float32)).cuda()
    if len(set(ks)) == 1 and not ragged:
        bud, keep = B.make_budget(int(ks[0]), batch=Bn), None
    else:
        cu_k = np.concatenate([[0], np.cumsum(ks)]).astype(np.int32)
        keep = torch.from_numpy(cu_k).cuda()
        bud = B.make_budget(0, cu_k=keep, total=int(cu_k[-1]))
    idx = torch.full((rows, bud.total), -1, dtype=torch.int32, device="cuda")
    if rows == 1:
        B.fastkv_select_tsp(shape, dS, bud, idx, ws)
    else:
        B.fastkv_select_kv(shape, dS, bud, idx, ws)
    status, site = B.fastkv_device_status(ws)
    return idx.cpu().numpy(), status


def oracle_select_batch(S, lens, ks, w, force_window):
    rows = S.shape[0]
    cu = np.concatenate([[0], np.cumsum(lens)])
    out = [[] for _ in range(rows)]
    for r in range(rows):
        for b, (L, k) in enumerate(zip(lens, ks)):
            idx, _ = oracle.select(S[r, cu[b]:cu[b + 1]].astype(np.float64), int(k), w, force_window)
            out[r].append(idx)
    return np.stack([np.concatenate(o) for o in out]).astype(np.int32)


@pytest.mark.parametrize("L,k,w", [(512, 128, 8), (100, 8, 8), (100, 100, 8), (131072, 13107, 8), (131072, 26214, 8),
                                   (300001, 50000, 8), (9, 9, 8), (65537, 1000, 16), (1000, 999, 1)])
@pytest.mark.parametrize("kind", ["random", "ties", "equal", "maxpool", "signed"])
def test_select_is_the_full_sort_definition(L, k, w, kind):
    rng = np.random.default_rng(L * 31 + k)
    if kind == "random":
        S = rng.random(L, dtype=np.float32) ** 8
    elif kind == "ties":
        S = (rng.integers(0, 7, L) / 8.0).astype(np.float32)
    elif kind == "equal":
        S = np.full(L, 0.125, dtype=np.float32)
    elif kind == "maxpool":                            # runs of 7 equal values, like MAX pooling gives
        base = rng.random(L, dtype=np.float32) ** 4
        S = np.max(np.lib.stride_tricks.sliding_window_view(np.pad(base, 3), 7), axis=1).astype(np.float32)
    else:                                              # negatives, zeros of both signs, tiny values
        S = rng.standard_normal(L).astype(np.float32)
        S[rng.integers(0, L, L // 4)] = 0.0
        S[rng.integers(0, L, L // 4)] = -0.0
        S[rng.integers(0, L, L // 8)] = 1e-40
    for fw in (True, False):
        got, status = run_select(S[None], [L], [k], w, fw)
        assert status == 0
        ref = oracle_select_batch(S[None], [L], [k], w, fw)
        np.testing.assert_array_equal(got, ref)


def test_select_kv_rows_and_ragged_offsets():
    rng = np.random.default_rng(7)
    lens = [5000, 8, 129, 70000, 4097]
    ks = [600, 8, 129, 7000, 9]
    total = sum(lens)
    S = (rng.integers(0, 50, (8, total)) / 64.0).astype(np.float32)
    got, status = run_select(S, lens, ks, 8, True, rows=8)
    assert status == 0
    np.testing.assert_array_equal(got, oracle_select_batch(S, lens, ks, 8, True))
    # uniform budget over a batch
    lens2, ks2 = [3000, 2000, 2500], [256, 256, 256]
    S2 = rng.random((2, sum(lens2)), dtype=np.float32)
    got, status = run_select(S2, lens2, ks2, 8, True, rows=2)
    np.testing.assert_array_equal(got, oracle_select_batch(S2, lens2, ks2, 8, True))


def test_select_reports_budget_outside_the_sequence():
    rng = np.random.default_rng(9)
    lens, ks = [1000, 50], [100, 100]                  # second sequence is shorter than its budget
    S = rng.random((1, 1050), dtype=np.float32)
    got, status = run_select(S, lens, ks, 8, True)
    assert status == B.ERR_DEVICE_INDEX
    np.testing.assert_array_equal(got[0, :100], oracle_select_batch(S[:, :1000], [1000], [100], 8, True)[0])


def make_compact_case(rng, lens, ks_kv, ks_tsp, Hkv, d, hidden, k_tok_stride=None, hidden_stride=None):
    total = sum(lens)
    kt = Hkv * d if k_tok_stride is None else k_tok_stride
    hs = hidden if hidden_stride is None else hidden_stride
    kbuf = rng.integers(0, 65536, (total, kt)).astype(np.uint16)
    vbuf = rng.integers(0, 65536, (total, kt)).astype(np.uint16)
    hbuf = rng.integers(0, 65536, (total, hs)).astype(np.uint16)
    pos = rng.integers(0, 1 << 30, total).astype(np.int32)
    idx_kv = np.concatenate([np.stack([rng.choice(L, k, replace=False) for _ in range(Hkv)])
                             for L, k in zip(lens, ks_kv)], axis=1).astype(np.int32)
    idx_tsp = np.concatenate([np.sort(rng.choice(L, k, replace=False)) for L, k in zip(lens, ks_tsp)]).astype(np.int32)
    return kbuf, vbuf, hbuf, pos, idx_kv, idx_tsp


def run_compact(lens, ks_kv, ks_tsp, Hkv, d, hidden, kbuf, vbuf, hbuf, pos, idx_kv, idx_tsp, ragged,
                k_tok_stride=None, hidden_stride=None):
    total, Bn = sum(lens), len(lens)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    d_cu = torch.from_numpy(cu).cuda() if (ragged or Bn > 1) else None
    shape = B.make_shape(total_len=total, n_q_heads=Hkv, n_kv_heads=Hkv, head_dim=d, hidden_dim=hidden, batch=Bn,
                         max_len=max(lens), cu_seqlens=d_cu, k_stride_tok=k_tok_stride, v_stride_tok=k_tok_stride,
                         hidden_stride_tok=hidden_stride)
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    t = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).cuda()
    keep = []

    def bud(ks):
        if not ragged:
            return B.make_budget(int(ks[0]), batch=Bn)
        c = torch.from_numpy(np.concatenate([[0], np.cumsum(ks)]).astype(np.int32)).cuda()
        keep.append(c)
        return B.make_budget(0, cu_k=c, total=int(sum(ks)))

    bkv, bt = bud(ks_kv), bud(ks_tsp)
    k_out = torch.zeros((Hkv, bkv.total, d), dtype=torch.int16, device="cuda")
    v_out = torch.zeros_like(k_out)
    h_out = torch.zeros((bt.total, hidden), dtype=torch.int16, device="cuda")
    p_out = torch.zeros((bt.total,), dtype=torch.int32, device="cuda")
    B.fastkv_compact(shape, t(idx_kv), bkv, t(idx_tsp), bt, t(kbuf), t(vbuf), t(hbuf), t(pos), k_out, v_out, h_out,
                     p_out, ws)
    status, site = B.fastkv_device_status(ws)
    f = lambda x: x.cpu().numpy().view(np.uint16)
    return f(k_out), f(v_out), f(h_out), p_out.cpu().numpy(), status


@pytest.mark.parametrize("Hkv,d,hidden", [(8, 128, 4096), (2, 64, 520), (1, 64, 256), (4, 128, 8)])
def test_compact_is_row_indexing(Hkv, d, hidden):
    rng = np.random.default_rng(d + hidden)
    for lens, ks_kv, ks_tsp, ragged in [([3000], [700], [901], False), ([500, 64, 1200], [100, 64, 333], [77, 8, 1200], True),
                                        ([400, 400], [50, 50], [60, 60], False)]:
        kbuf, vbuf, hbuf, pos, idx_kv, idx_tsp = make_compact_case(rng, lens, ks_kv, ks_tsp, Hkv, d, hidden)
        k_out, v_out, h_out, p_out, status = run_compact(lens, ks_kv, ks_tsp, Hkv, d, hidden, kbuf, vbuf, hbuf, pos,
                                                         idx_kv, idx_tsp, ragged)
        assert status == 0
        cu = np.concatenate([[0], np.cumsum(lens)])
        cuk = np.concatenate([[0], np.cumsum(ks_kv)])
        cut = np.concatenate([[0], np.cumsum(ks_tsp)])
        K3, V3 = kbuf.reshape(-1, Hkv, d), vbuf.reshape(-1, Hkv, d)
        for b in range(len(lens)):
            for h in range(Hkv):
                rows = cu[b] + idx_kv[h, cuk[b]:cuk[b + 1]]
                np.testing.assert_array_equal(k_out[h, cuk[b]:cuk[b + 1]], oracle.gather_rows(K3[:, h, :], rows))
                np.testing.assert_array_equal(v_out[h, cuk[b]:cuk[b + 1]], V3[rows, h])
            rows = cu[b] + idx_tsp[cut[b]:cut[b + 1]]
            np.testing.assert_array_equal(h_out[cut[b]:cut[b + 1]], oracle.gather_rows(hbuf, rows))
            np.testing.assert_array_equal(p_out[cut[b]:cut[b + 1]], pos[rows])


def test_compact_strided_sources_and_bad_index():
    rng = np.random.default_rng(3)
    Hkv, d, hidden = 4, 128, 512
    lens, ks_kv, ks_tsp = [2000], [300], [400]
    stride, hstride = Hkv * d + 64, hidden + 8             # padded rows
    kbuf, vbuf, hbuf, pos, idx_kv, idx_tsp = make_compact_case(rng, lens, ks_kv, ks_tsp, Hkv, d, hidden, stride, hstride)
    k_out, v_out, h_out, p_out, status = run_compact(lens, ks_kv, ks_tsp, Hkv, d, hidden, kbuf, vbuf, hbuf, pos, idx_kv,
                                                     idx_tsp, False, stride, hstride)
    assert status == 0
    for h in range(Hkv):
        np.testing.assert_array_equal(k_out[h], kbuf[idx_kv[h], h * d:(h + 1) * d])
        np.testing.assert_array_equal(v_out[h], vbuf[idx_kv[h], h * d:(h + 1) * d])
    np.testing.assert_array_equal(h_out, hbuf[idx_tsp, :hidden])
    # an index outside the sequence is skipped (its output row keeps its old contents) and reported
    bad_kv, bad_tsp = idx_kv.copy(), idx_tsp.copy()
    bad_kv[1, 5], bad_tsp[7] = 2000, -1
    k_out, v_out, h_out, p_out, status = run_compact(lens, ks_kv, ks_tsp, Hkv, d, hidden, kbuf, vbuf, hbuf, pos, bad_kv,
                                                     bad_tsp, False, stride, hstride)
    assert status == B.ERR_DEVICE_INDEX
    assert not k_out[1, 5].any() and not h_out[7].any() and p_out[7] == 0
    np.testing.assert_array_equal(k_out[1, 6], kbuf[idx_kv[1, 6], d:2 * d])
    np.testing.assert_array_equal(h_out[8], hbuf[idx_tsp[8], :hidden])
