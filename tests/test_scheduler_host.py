"""The multi-request scheduler on CPU: packing policy, and packed runs against per-request oracle runs
(the oracle's layer step stands in for the CUDA backend; the scheduler does no arithmetic of its own)."""
import numpy as np
import pytest

from oracle.layer import layer_step
from paper_2502_01068_b200 import workloads as W
from paper_2502_01068_b200.scheduler import BatchScheduler, LayerGeometry, LayerJob, pack, unpack


def geometry(with_tsp=True, Hq=4, Hkv=2, d=32, hidden=64):
    return LayerGeometry(n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, hidden_dim=hidden, window=8, pool_kernel=7,
                         pool_mode=W.POOL_AVG, with_tsp=with_tsp)


def job(rid, L, geo, k_kv, k_tsp=0):
    wl = W.Workload(name="rq", cfg=2000 + rid, n_q_heads=geo.n_q_heads, n_kv_heads=geo.n_kv_heads, head_dim=geo.head_dim,
                    hidden_dim=geo.hidden_dim, window=geo.window, pool_kernel=geo.pool_kernel, pool_mode=geo.pool_mode,
                    seq_lens=[L], k_kv=[k_kv], k_tsp=[k_tsp] if geo.with_tsp else None)
    x = W.make_layer(wl, with_hidden=geo.with_tsp)
    return LayerJob(rid, geo, x.q_win, x.k, x.v, x.hidden if geo.with_tsp else None, x.pos if geo.with_tsp else None,
                    k_kv, k_tsp)


class OracleBackend:
    """layer_step on the packed batch: what the CUDA backend computes, in fp64 on the CPU."""
    def __init__(self):
        self.calls = []

    def layer(self, batch):
        g = batch.geometry
        self.calls.append([j.request_id for j in batch.jobs])
        o = layer_step(batch.q_win, batch.k, batch.v, batch.hidden, batch.pos, batch.cu_seqlens, g.window, g.pool_kernel,
                       batch.k_kv, batch.k_tsp, pool_mode=g.pool_mode)
        return o


def per_request(j):
    g = j.geometry
    cu = np.array([0, j.length], dtype=np.int32)
    return layer_step(j.q_win, j.k, j.v, j.hidden, j.pos, cu, g.window, g.pool_kernel, [j.k_kv],
                      [j.k_tsp] if g.with_tsp else None, pool_mode=g.pool_mode)


def test_packed_batches_give_every_request_its_own_result():
    geo, geo_kv = geometry(True), geometry(False)
    jobs = [job(0, 300, geo, 40, 60), job(1, 64, geo, 16, 20), job(2, 513, geo_kv, 100), job(3, 129, geo, 30, 33),
            job(4, 200, geo_kv, 50), job(5, 700, geo, 70, 140)]
    sched = BatchScheduler(max_tokens=800, max_requests=8)
    for j in jobs:
        sched.submit(j)
    backend = OracleBackend()
    done = sched.run_all(backend)
    assert sorted(done) == [0, 1, 2, 3, 4, 5] and len(sched) == 0
    # FIFO with a token budget: 0 + 1 + 3 share the first call (493 tokens; 5 would exceed 800), the KV-only jobs
    # share one, the long job runs last
    assert backend.calls == [[0, 1, 3], [2, 4], [5]] and sched.batches_run == 3
    for j in jobs:
        ref, got = per_request(j), done[j.request_id]
        np.testing.assert_array_equal(got.idx_kv, ref["idx_kv"])
        np.testing.assert_array_equal(got.k_out, ref["k_out"])
        np.testing.assert_array_equal(got.v_out, ref["v_out"])
        if j.geometry.with_tsp:
            np.testing.assert_array_equal(got.idx_tsp, ref["idx_tsp"])
            np.testing.assert_array_equal(got.hidden_out, ref["hidden_out"])
            np.testing.assert_array_equal(got.pos_out, ref["pos_out"])
        else:
            assert got.idx_tsp is None


def test_packing_policy():
    geo = geometry(True)
    sched = BatchScheduler(max_tokens=256, max_requests=2)
    for rid, L in enumerate([100, 100, 40, 1000, 50]):
        sched.submit(job(rid, L, geo, 16, 16))
    order = []
    while len(sched):
        b = sched.next_batch()
        order.append([j.request_id for j in b.jobs])
        assert b.total_len <= 256 or len(b.jobs) == 1          # a job longer than the budget runs alone
        assert len(b.jobs) <= 2
        assert b.cu_seqlens.tolist() == np.concatenate([[0], np.cumsum([j.length for j in b.jobs])]).tolist()
    assert order == [[0, 1], [2, 4], [3]]                        # nothing waits behind more than one batch of later arrivals


def test_pack_rejects_what_the_library_would_reject():
    geo = geometry(True)
    with pytest.raises(ValueError):
        pack([job(0, 100, geo, 4, 16)])                          # k_kv smaller than the window
    with pytest.raises(ValueError):
        pack([job(0, 100, geo, 16, 200)])                        # k_tsp larger than the sequence
    with pytest.raises(ValueError):
        pack([job(0, 100, geo, 16, 16), job(1, 100, geometry(False), 16)])
    with pytest.raises(ValueError):
        pack([])
    b = pack([job(0, 100, geo, 16, 20), job(1, 50, geo, 10, 12)])
    out = {"idx_kv": np.zeros((2, 26), np.int32), "k_out": np.zeros((2, 26, 32), np.uint16), "v_out": np.zeros((2, 26, 32), np.uint16),
           "idx_tsp": np.arange(32, dtype=np.int32), "hidden_out": np.zeros((32, 64), np.uint16), "pos_out": np.zeros(32, np.int32)}
    r = unpack(b, out)
    assert r[0].idx_kv.shape == (2, 16) and r[1].idx_kv.shape == (2, 10)
    assert r[0].idx_tsp.tolist() == list(range(20)) and r[1].idx_tsp.tolist() == list(range(20, 32))
