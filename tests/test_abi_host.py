"""Host-side checks that need no GPU: the library loads, exports everything the header declares,
and rejects bad arguments with the documented status codes before touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2502_01068_b200 import binding as B
from paper_2502_01068_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    build.build_library()


def header_functions():
    text = open(os.path.join(ROOT, "include", "fastkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fastkv_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(B.library_path())
    names = header_functions()
    assert {"fastkv_score", "fastkv_select_kv", "fastkv_select_tsp", "fastkv_compact"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(B.EXPORTS) == sorted(n for n in names if n in B.EXPORTS)
    for n in names:                                    # the binding mirrors the ABI names
        assert hasattr(B, n), n


def good_shape(**kw):
    args = dict(total_len=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, hidden_dim=4096)
    args.update(kw)
    return B.make_shape(**args)


def status_of(fn, *a):
    with pytest.raises(B.FastKVError) as e:
        fn(*a)
    return e.value.status


def test_workspace_bytes_and_shape_validation():
    n = B.fastkv_workspace_bytes(good_shape())
    assert n % 256 == 0 and n > 8 * 4096 * 4
    # the persistent kernels keep one fp32 row per KV head plus statistics, not the fp32 logits
    assert 8 * 131072 * 4 < B.fastkv_workspace_bytes(good_shape(total_len=131072)) < 6 * 2 ** 20
    B.fastkv_debug_set("score_path", 1)                 # the buffered path needs room for the logits
    try:
        assert B.fastkv_workspace_bytes(good_shape(total_len=131072)) > 8 * 32 * 131072 * 4
    finally:
        B.fastkv_debug_set("score_path", 0)
    assert status_of(B.fastkv_debug_set, "no_such_key", 1) == B.ERR_INVALID_ARG
    assert status_of(B.fastkv_debug_set, "score_path", 9) == B.ERR_INVALID_ARG
    assert status_of(B.fastkv_workspace_bytes, good_shape(head_dim=96)) == B.ERR_UNSUPPORTED
    assert status_of(B.fastkv_workspace_bytes, good_shape(window=32)) == B.ERR_UNSUPPORTED      # G*w = 128
    assert status_of(B.fastkv_workspace_bytes, good_shape(n_q_heads=30)) == B.ERR_INVALID_ARG
    assert status_of(B.fastkv_workspace_bytes, good_shape(pool_kernel=4)) == B.ERR_INVALID_ARG
    assert status_of(B.fastkv_workspace_bytes, good_shape(pool_kernel=0)) == B.ERR_INVALID_ARG
    assert status_of(B.fastkv_workspace_bytes, good_shape(pool_mode=5)) == B.ERR_INVALID_ARG
    assert status_of(B.fastkv_workspace_bytes, good_shape(window=0)) == B.ERR_INVALID_ARG
    assert status_of(B.fastkv_workspace_bytes, good_shape(total_len=4, window=8)) == B.ERR_INVALID_ARG
    assert status_of(B.fastkv_workspace_bytes, good_shape(batch=2)) == B.ERR_INVALID_ARG        # no cu_seqlens
    assert status_of(B.fastkv_workspace_bytes, good_shape(k_stride_tok=1028)) == B.ERR_UNSUPPORTED
    assert status_of(B.fastkv_workspace_bytes, good_shape(softmax_scale=float("nan"))) == B.ERR_INVALID_ARG
    assert "head_dim" in B.fastkv_last_error() or B.fastkv_last_error()


class FakeBuf:
    """Stands in for a device tensor: the calls below must fail before any pointer is used."""
    def __init__(self, nbytes, ptr=0x1000):
        self._n, self._p = nbytes, ptr

    def numel(self):
        return self._n

    def element_size(self):
        return 1

    def data_ptr(self):
        return self._p


def test_calls_reject_bad_arguments_without_a_device(monkeypatch):
    monkeypatch.setattr(B, "_p", lambda t: None if t is None else (t.data_ptr() if hasattr(t, "data_ptr") else t.ctypes.data))
    monkeypatch.setattr(B, "_stream", lambda s: None)
    s = good_shape()
    ws = FakeBuf(B.fastkv_workspace_bytes(s), 0x10000)
    buf = FakeBuf(1 << 20, 0x20000)
    assert status_of(B.fastkv_score, s, None, buf, buf, None, ws) == B.ERR_INVALID_ARG
    assert status_of(B.fastkv_score, s, buf, buf, buf, None, FakeBuf(1024, 0x10000)) == B.ERR_WORKSPACE
    assert status_of(B.fastkv_score, s, buf, buf, buf, None, FakeBuf(ws.numel(), 0x10010)) == B.ERR_WORKSPACE
    bad_k = B.make_budget(4)                         # k < window with the window forced in
    assert status_of(B.fastkv_select_kv, s, buf, bad_k, buf, ws) == B.ERR_INVALID_ARG
    assert status_of(B.fastkv_select_tsp, s, buf, B.make_budget(5000), buf, ws) == B.ERR_INVALID_ARG   # k > L
    assert status_of(B.fastkv_select_tsp, s, None, B.make_budget(64), buf, ws) == B.ERR_INVALID_ARG
    assert status_of(B.fastkv_select_tsp, s, buf, B.make_budget(64, total=65), buf, ws) == B.ERR_INVALID_ARG
    kv = B.make_budget(64)
    assert status_of(B.fastkv_compact, s, buf, kv, None, None, buf, None, None, None, None, None, None, None,
                     ws) == B.ERR_INVALID_ARG       # k without k_out
    assert status_of(B.fastkv_compact, s, None, kv, None, None, buf, None, None, None, buf, None, None, None,
                     ws) == B.ERR_INVALID_ARG       # k/k_out without idx_kv
    assert B.fastkv_status_string(B.ERR_DEVICE_TIMEOUT).startswith("a bounded")
    assert B.fastkv_status_string(0) == "ok"


def test_sweep_schedule_matches_the_papers_compute_rate():
    """Sec. 5.1: with the TSP layer at 15 of 32 and a 20 % TSP rate the prefill compute rate is 60 %:
    layers 0..15 see the full prompt, layers 16..31 the propagated tokens."""
    from paper_2502_01068_b200 import workloads as W
    wl = W.llama8b_32k_sweep()
    L, kt = wl.seq_lens[0], wl.k_tsp[0]
    lens = [L if l <= W.SWEEP_TSP_LAYER else kt for l in range(W.SWEEP_LAYERS)]
    assert abs(sum(lens) / (W.SWEEP_LAYERS * L) - 0.60) < 1e-3
    assert kt == 6553 and W.llama8b_8k().k_tsp[0] == 1638 and W.llama8b_128k().k_tsp[0] == 26214
    assert W.llama8b_128k().k_kv[0] == 13107


def test_workload_generator_is_seeded_and_thread_independent():
    from paper_2502_01068_b200 import workloads as W
    wl = W.tiny()
    a, b = W.make_layer(wl), W.make_layer(wl)
    np.testing.assert_array_equal(a.k, b.k)
    np.testing.assert_array_equal(a.q_win, b.q_win)
    assert a.planted[0].tolist()[:4] == [0, 1, 2, 3] and len(a.planted[0]) == 9
    lens = W.ragged_lengths()
    assert len(lens) == 8 and all(4096 <= n <= 65536 for n in lens) and lens == W.ragged_lengths()
    x = np.array([1.0, 1.00390625, 1.01171875, -3.3, 65504.0], dtype=np.float32)
    import torch
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(W.f32_to_bf16_bits(x), ref)
