"""The multi-request scheduler driving the CUDA library: several requests of different lengths packed into
ragged batches, every request's result checked against its own oracle run."""
import numpy as np
import pytest

from paper_2502_01068_b200 import workloads as W
from paper_2502_01068_b200.scheduler import BatchScheduler, CudaBatchBackend, LayerGeometry, LayerJob
from tests.parity import check_index_set, oracle_layer

pytestmark = pytest.mark.gpu


def test_requests_packed_into_ragged_batches_match_their_own_oracle_runs():
    geo = LayerGeometry(n_q_heads=8, n_kv_heads=2, head_dim=128, hidden_dim=256, window=8, pool_kernel=7,
                        pool_mode=W.POOL_AVG, with_tsp=True)
    specs = [(0, 3000, 300, 500), (1, 130, 20, 30), (2, 2049, 256, 400), (3, 700, 64, 140), (4, 5000, 512, 1000)]
    sched = BatchScheduler(max_tokens=6000, max_requests=4)
    work = {}
    for rid, L, k_kv, k_tsp in specs:
        wl = W.Workload(name="rq", cfg=2100 + rid, n_q_heads=8, n_kv_heads=2, head_dim=128, hidden_dim=256, window=8,
                        pool_kernel=7, pool_mode=W.POOL_AVG, seq_lens=[L], k_kv=[k_kv], k_tsp=[k_tsp])
        x = W.make_layer(wl)
        work[rid] = (wl, x)
        sched.submit(LayerJob(rid, geo, x.q_win, x.k, x.v, x.hidden, x.pos, k_kv, k_tsp))
    done = sched.run_all(CudaBatchBackend())
    assert sched.batches_run == 2 and sorted(done) == [0, 1, 2, 3, 4]
    for rid, (wl, x) in work.items():
        o, r = oracle_layer(wl, x), done[rid]
        L = wl.seq_lens[0]
        for h in range(2):
            check_index_set(r.idx_kv[h], o["idx_kv"][h], o["S_kv"][h], o["tau_kv"][0, h], L, 8, True, "request %d kv" % rid)
            np.testing.assert_array_equal(r.k_out[h], x.k[r.idx_kv[h], h])
            np.testing.assert_array_equal(r.v_out[h], x.v[r.idx_kv[h], h])
        check_index_set(r.idx_tsp, o["idx_tsp"], o["S_tsp"], o["tau_tsp"][0], L, 8, True, "request %d tsp" % rid)
        np.testing.assert_array_equal(r.hidden_out, x.hidden[r.idx_tsp])
        np.testing.assert_array_equal(r.pos_out, x.pos[r.idx_tsp])
