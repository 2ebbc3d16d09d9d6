"""A bounded device-side wait that runs out: the scoring kernel's second pass is told (test hook) to wait
for one more publication of softmax statistics than there are CTAs, with the poll limit cut to about two
milliseconds.  Nothing faults and nothing hangs: the wait gives up, the CTA runs through the rest of its
loops without work, the call's status word reads FASTKV_ERR_DEVICE_TIMEOUT with the site of the wait, and
the next ordinary call on the same workspace is correct."""
import numpy as np
import pytest
import torch

from paper_2502_01068_b200 import binding as B
from paper_2502_01068_b200 import workloads as W
from tests.parity import check_layer, dev, gpu_layer, oracle_layer

pytestmark = pytest.mark.gpu

SITE_PASS2_PUBLICATION_WAIT = 14


@pytest.mark.parametrize("path", [3, 2])
def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_correct(debug_hooks, path):
    wl = W.tiny()
    x = W.make_layer(wl)
    L = wl.seq_lens[0]
    shape = B.make_shape(total_len=L, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim)
    debug_hooks("score_path", path)
    ws = torch.empty(B.fastkv_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    s_kv = torch.zeros((wl.n_kv_heads, L), dtype=torch.float32, device="cuda")
    q, k = dev(x.q_win), dev(x.k)

    debug_hooks("wait_limit_cycles", 1 << 22)
    debug_hooks("extra_publications", 1)
    B.fastkv_score(shape, q, k, s_kv, None, ws)
    status, site = B.fastkv_device_status(ws)
    assert status == B.ERR_DEVICE_TIMEOUT
    assert site == SITE_PASS2_PUBLICATION_WAIT

    debug_hooks("wait_limit_cycles", 0)
    debug_hooks("extra_publications", 0)
    B.fastkv_score(shape, q, k, s_kv, None, ws)              # same workspace: the call clears the status word
    assert B.fastkv_device_status(ws) == (0, 0)
    g = gpu_layer(wl, x)
    o = oracle_layer(wl, x)
    check_layer(wl, x, g, o, what="after the timeout")
    np.testing.assert_allclose(s_kv.cpu().numpy(), o["S_kv"], rtol=2e-3, atol=1e-12)
