"""fastkv_score_static is the scoring call for users who cannot hand the library a workspace (their
process may not call cudaMalloc, or the device allocator is not theirs to use).  It must give what
fastkv_score gives.  Both run the same kernels, so the comparison is exact; it is made on two calls
in a row because the built-in scratch array is shared and keeps the previous call's contents.
This file sorts last on purpose."""
import numpy as np
import pytest
import torch

from paper_2502_01068_b200 import binding as B
from paper_2502_01068_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _inputs(cfg, L, Hq=32, Hkv=8, d=128):
    wl = W.Workload(name="static", cfg=cfg, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, hidden_dim=64, window=8,
                    pool_kernel=7, pool_mode=W.POOL_AVG, seq_lens=[L], k_kv=[64], k_tsp=[64])
    x = W.make_layer(wl, with_v=False, with_hidden=False)
    shape = B.make_shape(total_len=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d)
    q = torch.from_numpy(x.q_win.view(np.int16)).cuda()
    k = torch.from_numpy(x.k.view(np.int16)).cuda()
    return shape, q, k


def _score(shape, q, k, static):
    L, Hkv = shape.total_len, shape.n_kv_heads
    s_kv = torch.full((Hkv, L), -1.0, dtype=torch.float32, device="cuda")
    s_tsp = torch.full((L,), -1.0, dtype=torch.float32, device="cuda")
    if static:
        B.fastkv_score_static(shape, q, k, s_kv, s_tsp)
        assert B.fastkv_score_static_status() == (0, 0)      # the status word inside the built-in array
    else:
        ws = torch.empty(B.fastkv_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
        B.fastkv_score(shape, q, k, s_kv, s_tsp, ws)
        assert B.fastkv_device_status(ws)[0] == 0
    torch.cuda.synchronize()
    return s_kv.cpu().numpy(), s_tsp.cpu().numpy()


def test_static_scratch_matches_workspace_path_on_two_calls_in_a_row():
    first = _inputs(901, 5000)
    second = _inputs(902, 3001, Hq=8, Hkv=2, d=64)          # a different shape reuses the same array
    third = _inputs(903, 40000)                             # 1.6 MB of scratch: well inside the array
    for shape, q, k in (first, second, first, third):
        ref_kv, ref_tsp = _score(shape, q, k, static=False)
        got_kv, got_tsp = _score(shape, q, k, static=True)
        assert np.isfinite(got_kv).all() and got_kv.min() >= 0.0
        np.testing.assert_allclose(got_kv, ref_kv, rtol=2e-3, atol=1e-12)
        np.testing.assert_allclose(got_tsp, ref_tsp, rtol=2e-3, atol=1e-12)
        np.testing.assert_array_equal(got_kv, ref_kv)       # same kernels, same order of operations


def test_static_scratch_rejects_shapes_beyond_its_size():
    shape = B.make_shape(total_len=600000, n_q_heads=32, n_kv_heads=8, head_dim=128)
    assert B.fastkv_workspace_bytes(shape) > (16 << 20)
    assert B.fastkv_workspace_bytes(B.make_shape(total_len=131072, n_q_heads=32, n_kv_heads=8, head_dim=128)) < (6 << 20)
    buf = torch.zeros(8, dtype=torch.int16, device="cuda")
    with pytest.raises(B.FastKVError) as e:
        B.fastkv_score_static(shape, buf, buf, buf, None)
    assert e.value.status == B.ERR_WORKSPACE
    assert "built-in array" in str(e.value)


def test_a_short_sequence_is_reported_through_the_static_status_reader():
    """A ragged batch with a sequence shorter than the observation window leaves FASTKV_ERR_INVALID_ARG in the
    status word of the built-in array; the next good call clears it."""
    lens = [300, 5, 700]
    wl = W.Workload(name="static_short", cfg=904, n_q_heads=8, n_kv_heads=2, head_dim=128, hidden_dim=64, window=8,
                    pool_kernel=7, pool_mode=W.POOL_AVG, seq_lens=lens, k_kv=[40, 8, 60], k_tsp=[50, 8, 90])
    x = W.make_layer(wl, with_v=False, with_hidden=False)
    cu = torch.from_numpy(x.cu_seqlens.astype(np.int32)).cuda()
    shape = B.make_shape(total_len=sum(lens), n_q_heads=8, n_kv_heads=2, head_dim=128, batch=3, max_len=700,
                         cu_seqlens=cu)
    q = torch.from_numpy(x.q_win.view(np.int16)).cuda()
    k = torch.from_numpy(x.k.view(np.int16)).cuda()
    s_kv = torch.zeros((2, sum(lens)), dtype=torch.float32, device="cuda")
    B.fastkv_score_static(shape, q, k, s_kv, None)
    status, site = B.fastkv_score_static_status()
    assert status == B.ERR_INVALID_ARG and site != 0
    shape1, q1, k1 = _inputs(901, 5000)
    _score(shape1, q1, k1, static=True)                     # asserts status (0, 0) again
