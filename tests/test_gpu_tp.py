"""Tensor-parallel layer step on the GPU: two ranks' shards run one after the other on one device (their
kernels never wait on each other, so this is a faithful emulation); the all-reduce of the layer-level score
is done by hand.  Checked against the unsharded oracle."""
import numpy as np
import pytest
import torch

from paper_2502_01068_b200 import workloads as W
from paper_2502_01068_b200.tp import CudaBackend, HeadShard, shard_heads, tp_layer_step
from tests.parity import check_index_set, check_scores, oracle_layer

pytestmark = pytest.mark.gpu


def test_two_emulated_ranks_match_the_oracle():
    wl = W.Workload(name="tp", cfg=56, n_q_heads=16, n_kv_heads=4, head_dim=128, hidden_dim=512, window=8,
                    pool_kernel=7, pool_mode=W.POOL_AVG, seq_lens=[6000], k_kv=[700], k_tsp=[1200])
    x = W.make_layer(wl)
    o = oracle_layer(wl, x)
    L, w, world = wl.seq_lens[0], wl.window, 2
    t = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).cuda()
    hidden, pos = t(x.hidden), t(x.pos)
    shards = [HeadShard(r, world, wl.n_q_heads, wl.n_kv_heads) for r in range(world)]
    backends = [CudaBackend(s, L, wl.head_dim, wl.hidden_dim) for s in shards]
    locals_ = [(shard_heads(t(x.q_win), s.q_range), shard_heads(t(x.k), s.kv_range), shard_heads(t(x.v), s.kv_range))
               for s in shards]
    # what the all-reduce delivers: the sum of the ranks' partial layer-level scores
    partials = [b.score(q, k)[1] for b, (q, k, v) in zip(backends, locals_)]
    s_tsp = partials[0] + partials[1]
    check_scores(s_tsp.cpu().numpy(), o["S_tsp"], "all-reduced S_tsp")
    idx_tsp_all = []
    for s, b, (q, k, v) in zip(shards, backends, locals_):
        idx_kv, idx_tsp, k_out, v_out, hid_out, pos_out = tp_layer_step(b, s, q, k, v, hidden, pos, 700, 1200,
                                                                         reduce_fn=lambda _: s_tsp.clone())
        torch.cuda.synchronize()
        idx_kv, idx_tsp = idx_kv.cpu().numpy(), idx_tsp.cpu().numpy()
        for j, g in enumerate(s.kv_range):
            check_index_set(idx_kv[j], o["idx_kv"][g], o["S_kv"][g], o["tau_kv"][0, g], L, w, True, "tp idx_kv[%d]" % g)
            np.testing.assert_array_equal(k_out[j].cpu().numpy().view(np.uint16), x.k[idx_kv[j], g])
            np.testing.assert_array_equal(v_out[j].cpu().numpy().view(np.uint16), x.v[idx_kv[j], g])
        check_index_set(idx_tsp, o["idx_tsp"], o["S_tsp"], o["tau_tsp"][0], L, w, True, "tp idx_tsp")
        np.testing.assert_array_equal(hid_out.cpu().numpy().view(np.uint16), x.hidden[idx_tsp])
        np.testing.assert_array_equal(pos_out.cpu().numpy(), x.pos[idx_tsp])
        idx_tsp_all.append(idx_tsp)
    np.testing.assert_array_equal(idx_tsp_all[0], idx_tsp_all[1])      # same numbers in, same set out
