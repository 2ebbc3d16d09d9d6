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


SITE_ATTN_S_READY_WAIT = 33          # the softmax warps' wait for "S of this key tile is in tensor memory"
SITE_ATTN_P_READY_WAIT = 31          # the issuer's wait for the P the stalled softmax warps never hand over
SITE_ATTN_TURN_WAIT = 32             # the other query tile's issuer's wait for its turn, which the stalled one never passes on
SITE_ATTN_RING_WAIT = 26             # the producer's wait for a K / V stage the stalled issuer never releases


def test_prefill_attention_wait_that_runs_out(debug_hooks):
    """The prefill attention's softmax warps wait (bounded) for the tensor core to have left S of the key tile in
    tensor memory; the test hook withholds that signal for one key tile of every CTA's first query tile.  The wait
    gives up after about two milliseconds,
    every role of the CTA runs out of its loops, copies and contractions in flight are waited for, the status word
    says where -- and the next call on the same workspace is correct."""
    import oracle
    wl = W.Workload(name="prefill_timeout", cfg=980, n_q_heads=4, n_kv_heads=2, head_dim=64, hidden_dim=64, window=8,
                    pool_kernel=7, pool_mode=W.POOL_AVG, seq_lens=[900], k_kv=[8], k_tsp=[8])
    x = W.make_layer(wl)
    q_full = W.full_q(wl, x)
    L = wl.total_len
    shape = B.make_shape(total_len=L, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                         window=wl.window, pool_kernel=wl.pool_kernel, q_layout=B.Q_FULL)
    ws = torch.empty(B.fastkv_prefill_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    out = torch.zeros((L, wl.n_q_heads, wl.head_dim), dtype=torch.int16, device="cuda")
    s_kv = torch.zeros((wl.n_kv_heads, L), dtype=torch.float32, device="cuda")
    debug_hooks("wait_limit_cycles", 1 << 22)
    debug_hooks("prefill_skip_commit", 2)                      # key tile 1: every CTA whose first query tile has two or more key tiles stalls
    B.fastkv_prefill_attention(shape, dev(q_full), dev(x.k), dev(x.v), out, s_kv, None, ws)
    status, site = B.fastkv_device_status(ws)
    assert status == B.ERR_DEVICE_TIMEOUT
    assert site in (SITE_ATTN_S_READY_WAIT, SITE_ATTN_P_READY_WAIT, SITE_ATTN_TURN_WAIT, SITE_ATTN_RING_WAIT)   # whichever gives up first

    debug_hooks("wait_limit_cycles", 0)
    debug_hooks("prefill_skip_commit", 0)
    B.fastkv_prefill_attention(shape, dev(q_full), dev(x.k), dev(x.v), out, s_kv, None, ws)
    assert B.fastkv_device_status(ws) == (0, 0)
    got = W.bf16_bits_to_f32(out.cpu().numpy().view(np.uint16)).astype(np.float64)
    ref = oracle.prefill_attention(q_full, x.k, x.v)
    assert np.all(np.abs(got - ref) <= 1e-2 * np.abs(ref) + 1e-2)
    o = oracle_layer(wl, x, do_compact=False)
    np.testing.assert_allclose(s_kv.cpu().numpy(), o["S_kv"], rtol=2e-3, atol=1e-12)
