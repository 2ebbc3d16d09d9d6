"""fastkv_layer_host (the whole step from HOST buffers: the end-to-end leg of the bench) against the
fp64 oracle: every output that comes back over PCIe goes through the same acceptance rules as the
device-buffer path."""
import numpy as np
import pytest

from paper_2502_01068_b200 import binding as B
from paper_2502_01068_b200 import workloads as W
from tests.parity import check_layer, gpu_layer, host_layer, oracle_layer

pytestmark = pytest.mark.gpu


def _wl(name, cfg, lens, k_kv, k_tsp, Hq=8, Hkv=2, d=128, hidden=256):
    return W.Workload(name=name, cfg=cfg, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, hidden_dim=hidden, window=8,
                      pool_kernel=7, pool_mode=W.POOL_AVG, seq_lens=list(lens), k_kv=[k_kv] * len(lens),
                      k_tsp=None if k_tsp is None else [k_tsp] * len(lens))


@pytest.mark.parametrize("pinned", [True, False])
def test_tiny_config_from_host_buffers(pinned):
    wl = W.tiny()
    x = W.make_layer(wl)
    g = host_layer(wl, x, pinned=pinned)
    o = oracle_layer(wl, x)
    check_layer(wl, x, g, o, what="tiny host")
    np.testing.assert_array_equal(g["idx_kv"][0], g["idx_tsp"])


def test_odd_length_from_host_buffers():
    wl = _wl("host_odd", 1200, [3001], 333, 517)
    x = W.make_layer(wl)
    g = host_layer(wl, x)
    o = oracle_layer(wl, x)
    check_layer(wl, x, g, o, what="odd host")
    d = gpu_layer(wl, x)                       # the device-buffer path gives the same bytes
    for key in ("idx_kv", "idx_tsp", "k_out", "v_out", "hidden_out", "pos_out"):
        np.testing.assert_array_equal(g[key], d[key])


def test_uniform_budget_batch_with_host_cu_seqlens():
    wl = _wl("host_batch", 1201, [700, 129, 2048, 300], 64, 100)
    x = W.make_layer(wl)
    g = host_layer(wl, x)
    o = oracle_layer(wl, x)
    check_layer(wl, x, g, o, what="batch host")


def test_layer_without_tsp_from_host_buffers():
    wl = _wl("host_kv_only", 1202, [1500], 200, None, Hq=4, Hkv=1, d=64)
    x = W.make_layer(wl, with_hidden=False)
    g = host_layer(wl, x)
    o = oracle_layer(wl, x)
    check_layer(wl, x, g, o, what="kv-only host")
