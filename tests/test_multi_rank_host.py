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
