"""fastkv_score_static is the scoring call for users who cannot hand the library a workspace (their
process may not call cudaMalloc, or the device allocator is not theirs to use).  It must give what
fastkv_score gives.  Both run the same kernels, so the comparison is exact; it is made on two calls
in a row because the built-in scratch array is shared and keeps the previous call's contents.
This file sorts last on purpose: a run that stops at the first failure has then run everything else."""
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
    else:
        ws = torch.empty(B.fastkv_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
        B.fastkv_score(shape, q, k, s_kv, s_tsp, ws)
        assert B.fastkv_device_status(ws)[0] == 0
    torch.cuda.synchronize()
    return s_kv.cpu().numpy(), s_tsp.cpu().numpy()


def test_static_scratch_matches_workspace_path_on_two_calls_in_a_row():
    first = _inputs(901, 5000)
    second = _inputs(902, 3001, Hq=8, Hkv=2, d=64)          # a different shape reuses the same array
    for shape, q, k in (first, second, first):
        ref_kv, ref_tsp = _score(shape, q, k, static=False)
        got_kv, got_tsp = _score(shape, q, k, static=True)
        assert np.isfinite(got_kv).all() and got_kv.min() >= 0.0
        np.testing.assert_allclose(got_kv, ref_kv, rtol=2e-3, atol=1e-12)
        np.testing.assert_allclose(got_tsp, ref_tsp, rtol=2e-3, atol=1e-12)
        np.testing.assert_array_equal(got_kv, ref_kv)       # same kernels, same order of operations


def test_static_scratch_rejects_shapes_beyond_its_size():
    shape = B.make_shape(total_len=32768, n_q_heads=32, n_kv_heads=8, head_dim=128)
    assert B.fastkv_workspace_bytes(shape) > (16 << 20)
    buf = torch.zeros(8, dtype=torch.int16, device="cuda")
    with pytest.raises(B.FastKVError) as e:
        B.fastkv_score_static(shape, buf, buf, buf, None)
    assert e.value.status == B.ERR_WORKSPACE
    assert "built-in array" in str(e.value)
