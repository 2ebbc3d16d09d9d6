"""The N > 1 path of the bench shards independent layers over ranks with no data-path collective; what the
ranks do exchange is the timing (max over ranks) -- covered here with two gloo ranks on CPU -- and each rank's
inputs must be its own layer, drawn from its own seed."""
import os
import socket
import subprocess
import sys
import textwrap

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    from paper_2502_01068_b200 import workloads as W
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)            # rank 1 is the slow one
    x = W.make_layer(W.tiny(), layer=rank, with_v=False, with_hidden=False)
    dist.barrier()
    print(json.dumps({"rank": rank, "ms": ms, "value": bench.whole_job_throughput(512, world, ms),
                      "k_sum": int(x.k.astype("int64").sum())}))
    dist.destroy_process_group()
""" % ROOT)


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_agree_on_the_slowest_time_and_draw_their_own_layers():
    import json
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    assert [o["ms"] for o in outs] == [15.0, 15.0]                  # max over ranks on every rank
    np.testing.assert_allclose([o["value"] for o in outs], 2 * 512 / 15e-3)
    assert outs[0]["k_sum"] != outs[1]["k_sum"]                     # independent layers per rank


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.whole_job_throughput(1000, 1, 2.0) == 500000.0
    ab = bench.algorithmic_bytes(bench.pick_workload("llama8b_128k_tsp_layer"))
    assert ab["step_rw"] == 816059168 and ab["compact"] == 537596712


TP_WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import numpy as np, torch, torch.distributed as dist
    import oracle
    from paper_2502_01068_b200 import workloads as W
    from paper_2502_01068_b200.tp import HeadShard, tp_layer_step, shard_heads

    class OracleBackend:                      # the three steps on this rank's heads, in fp64 on the CPU
        def __init__(self, w, p): self.w, self.p = w, p
        def score(self, q, k):
            L = k.shape[0]
            s_kv, s_tsp, _ = oracle.scores(q.numpy().view(np.uint16), L - self.w, k.numpy().view(np.uint16), self.w, self.p)
            return torch.from_numpy(s_kv), torch.from_numpy(s_tsp)
        def select(self, s_kv, k_kv, s_tsp, k_tsp):
            idx_kv = np.stack([oracle.select(s_kv[g].numpy(), k_kv, self.w)[0] for g in range(s_kv.shape[0])])
            return torch.from_numpy(idx_kv), torch.from_numpy(oracle.select(s_tsp.numpy(), k_tsp, self.w)[0])
        def compact(self, idx_kv, idx_tsp, k, v, hidden, pos):
            k_out = torch.stack([k[idx_kv[g], g] for g in range(idx_kv.shape[0])])
            v_out = torch.stack([v[idx_kv[g], g] for g in range(idx_kv.shape[0])])
            return k_out, v_out, hidden[idx_tsp], pos[idx_tsp]

    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = W.Workload(name="tp", cfg=55, n_q_heads=8, n_kv_heads=4, head_dim=32, hidden_dim=64, window=8, pool_kernel=7,
                    pool_mode=W.POOL_AVG, seq_lens=[700], k_kv=[90], k_tsp=[150])
    x = W.make_layer(wl)                                    # every rank draws the same layer, keeps its heads
    shard = HeadShard(rank, world, wl.n_q_heads, wl.n_kv_heads)
    t = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a)
    q, k, v = (shard_heads(t(a), r) for a, r in ((x.q_win, shard.q_range), (x.k, shard.kv_range), (x.v, shard.kv_range)))
    out = tp_layer_step(OracleBackend(wl.window, wl.pool_kernel), shard, q, k, v, t(x.hidden), t(x.pos), 90, 150)
    idx_kv, idx_tsp, k_out, v_out, hidden_out, pos_out = out
    # the unsharded oracle, for comparison
    from oracle.layer import layer_step
    ref = layer_step(x.q_win, x.k, x.v, x.hidden, x.pos, x.cu_seqlens, wl.window, wl.pool_kernel, wl.k_kv, wl.k_tsp)
    ok = {
        "idx_kv": bool(np.array_equal(idx_kv.numpy(), ref["idx_kv"][shard.kv_range.start:shard.kv_range.stop])),
        "idx_tsp": bool(np.array_equal(idx_tsp.numpy(), ref["idx_tsp"])),
        "k_out": bool(np.array_equal(k_out.numpy().view(np.uint16), ref["k_out"][shard.kv_range.start:shard.kv_range.stop])),
        "hidden_out": bool(np.array_equal(hidden_out.numpy().view(np.uint16), ref["hidden_out"])),
        "pos_out": bool(np.array_equal(pos_out.numpy(), ref["pos_out"])),
    }
    gathered = [torch.zeros_like(idx_tsp) for _ in range(world)]
    dist.all_gather(gathered, idx_tsp)
    ok["same_idx_tsp_on_all_ranks"] = all(bool(torch.equal(g, idx_tsp)) for g in gathered)
    print(json.dumps({"rank": rank, **ok}))
    dist.destroy_process_group()
""" % ROOT)


def test_tensor_parallel_step_on_two_gloo_ranks_matches_the_unsharded_oracle():
    """KV heads sharded over two ranks, the layer-level score all-reduced: each rank's KV selection and
    rows are the unsharded ones for its heads, and every rank gets the same TSP index set."""
    import json
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", TP_WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-3000:]
        res = json.loads(out.strip().splitlines()[-1])
        assert all(v for k, v in res.items() if k != "rank"), res


def test_head_shard_arithmetic():
    sys.path.insert(0, ROOT)
    from paper_2502_01068_b200.tp import HeadShard
    import pytest
    s = HeadShard(rank=1, world=4, n_q_heads=32, n_kv_heads=8)
    assert list(s.kv_range) == [2, 3] and list(s.q_range) == list(range(8, 16)) and s.group == 4
    with pytest.raises(ValueError):
        HeadShard(0, 3, 32, 8)


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`bench.py --gpus N` without WORLD_SIZE re-executes itself under the torch launcher with N ranks on
    127.0.0.1.  Checked here on CPU with the oracle arm on the tiny workload: rank 0 prints the one JSON line,
    the other rank exits 0 without work."""
    import json
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.spawn_command(2, ["--impl", "reference", "--workload", "tiny", "--steps", "1", "--warmup", "0", "--gpus", "2"],
                              free_port())
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "127.0.0.1" in cmd and "2" in cmd
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-3000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2
    assert lines[0]["config"] == bench.config_of("tiny", bench.pick_workload("tiny"))
