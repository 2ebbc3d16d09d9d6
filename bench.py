#!/usr/bin/env python
"""Benchmark of the FastKV score -> select -> compact layer step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference] [--tp]

One "step" is one pass of the whole hot path (fastkv_score, fastkv_select = select_kv + select_tsp in
one launch, fastkv_compact) over one layer of synthetic, seeded input.  The default workload is the
Llama-3.1-8B-shaped layer at L = 131072 with Token-Selective Propagation (KV retention 10 %, TSP
rate 20 %).  With N > 1 every rank (one per GPU; started here when the launcher has not started
them) runs its own layer of the same shape -- the path partitions over independent layers /
requests, so there is no collective on the data path -- and the reported value is all ranks' tokens
over the slowest rank's time.  `--tp` adds the tensor-parallel form of the same layer (KV heads
sharded over the ranks, one all-reduce of the layer-level score).

Prints one JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2502_01068_b200 import workloads as W  # noqa: E402

METRIC = "context tokens/sec for score+select+compact, per layer"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126 * 2 ** 20
KERNELS = {0: "score", 1: "pool", 2: "select", 3: "compact"}
KERNEL_SYMBOLS = {"score": "score_parked_kernel / score_fused_kernel", "pool": "pool_rows_kernel",
                  "select": "select_topk_kernel", "compact": "compact_rows_kernel"}


def pick_workload(name: str) -> W.Workload:
    table = {
        "llama8b_128k_tsp_layer": W.llama8b_128k,
        "llama8b_8k": W.llama8b_8k,
        "llama8b_32k_tsp_layer": W.llama8b_32k_sweep,
        "llama8b_ragged": W.llama8b_ragged,
        "tiny": W.tiny,
    }
    return table[name]()


def config_of(name: str, wl: W.Workload) -> dict:
    """What both arms print as `config`."""
    return {"workload": name, "seq_lens": wl.seq_lens, "k_kv": wl.k_kv, "k_tsp": wl.k_tsp,
            "n_q_heads": wl.n_q_heads, "n_kv_heads": wl.n_kv_heads, "head_dim": wl.head_dim,
            "hidden_dim": wl.hidden_dim, "window": wl.window, "pool_kernel": wl.pool_kernel}


def algorithmic_bytes(wl: W.Workload) -> dict:
    """Bytes the step must move (each tensor read or written once): K streamed by the scoring, the
    window queries, scores written and read, indices written and read, kept rows read and written."""
    Hkv, d, hid = wl.n_kv_heads, wl.head_dim, wl.hidden_dim
    total = wl.total_len
    kkv = sum(wl.k_kv)
    kt = sum(wl.k_tsp) if wl.k_tsp else 0
    k_read = total * Hkv * d * 2
    q_read = wl.batch * wl.window * wl.n_q_heads * d * 2
    unpooled = 4 * Hkv * total
    scores = 4 * (Hkv * total + (total if kt else 0))
    idx = 4 * (Hkv * kkv + kt)
    kv_rows = 2 * Hkv * kkv * d * 2
    hid_rows = kt * (hid * 2 + 4)
    return {
        "score": k_read + q_read + scores,                 # the fastkv_score call: both of its kernels
        "score_kernel": k_read + q_read + unpooled,        # K streamed once, one un-pooled fp32 row per KV head written
        "pool_kernel": unpooled + scores,
        "select": scores + idx,
        "compact": idx + 2 * kv_rows + 2 * hid_rows,
        "step_rw": k_read + q_read + 2 * scores + 2 * idx + 2 * kv_rows + 2 * hid_rows,
        "step_min": k_read + q_read + 2 * scores + 2 * idx + kv_rows + hid_rows,
    }


def measured_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d.get("bf16_tflops", 1590.0)),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", 1400.0)),
                "source": "measured (MEASURED_PEAKS.json)"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback (earlier measurement on this pool)"}


def profiled_traffic(kernel: str, workload: str):
    """DRAM bytes per launch of `kernel` from the committed ncu summary of this workload, or None."""
    tag = {"llama8b_128k_tsp_layer": "llama8b_128k"}.get(workload)
    if tag is None:
        return None
    for name in {"score": ("score_parked_kernel",), "compact": ("compact_rows_kernel",),
                 "select": ("select_topk_kernel",), "pool": ("pool_rows_kernel",)}.get(kernel, ()):
        path = os.path.join(ROOT, "profiles", "%s_%s.txt" % (name, tag))
        try:
            with open(path) as f:
                for line in f:
                    if line.startswith("dram_bytes_per_launch:"):
                        return int(line.split(":")[1])
        except OSError:
            pass
    return None


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if bit and (mask & bit):
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self) -> dict:
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2.0)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(value: float, world: int, device=None) -> float:
    """The slowest rank's time: every multi-GPU number is the max over ranks (device-timed per rank)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Weak scaling over independent layers: all ranks' tokens over the slowest rank's step time."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def spawn_command(n: int, argv, port: int):
    """The launcher line that starts `n` ranks of this script on one node (what the scaling run uses)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n: int, argv) -> int:
    """`--gpus N` without a launcher: start the N ranks here and hand their output through."""
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "WARN")
    return subprocess.call(spawn_command(n, argv, free_port()), env=env)


def oracle_layer_timed(wl: W.Workload, x: W.LayerInputs) -> dict:
    """One whole layer through the oracle's routines in the order of Algorithm 1, each step timed."""
    import oracle
    w, t = wl.window, {"scores": 0.0, "select": 0.0, "compact": 0.0}
    for b in range(wl.batch):
        lo, hi = int(x.cu_seqlens[b]), int(x.cu_seqlens[b + 1])
        t0 = time.perf_counter()
        s_kv, s_tsp, _ = oracle.scores(x.q_win[b * w:(b + 1) * w], hi - lo - w, x.k[lo:hi], w, wl.pool_kernel, wl.pool_mode)
        t1 = time.perf_counter()
        idx_kv = [oracle.select(s_kv[g], int(wl.k_kv[b]), w)[0] for g in range(wl.n_kv_heads)]
        idx_tsp = oracle.select(s_tsp, int(wl.k_tsp[b]), w)[0] if wl.k_tsp else None
        t2 = time.perf_counter()
        for g in range(wl.n_kv_heads):
            oracle.gather_rows(x.k[:, g, :], lo + idx_kv[g])
            if x.v is not None:
                oracle.gather_rows(x.v[:, g, :], lo + idx_kv[g])
        if idx_tsp is not None and x.hidden is not None:
            oracle.gather_rows(x.hidden, lo + idx_tsp)
            oracle.gather_rows(x.pos, lo + idx_tsp)
        t3 = time.perf_counter()
        t["scores"] += t1 - t0
        t["select"] += t2 - t1
        t["compact"] += t3 - t2
    t["layer"] = t["scores"] + t["select"] + t["compact"]
    return t


ONE_THREAD_CHILD = r"""
import json, sys, time
sys.path.insert(0, %r)
import bench
from paper_2502_01068_b200 import workloads as W
wl = bench.pick_workload(%r)
x = W.make_layer(wl)
import oracle
oracle.build()
t = bench.oracle_layer_timed(wl, x)
print(json.dumps({"threads": oracle.num_threads(), "seconds": t}))
"""


def oracle_baseline(name: str, wl: W.Workload, x: W.LayerInputs, budget_s: float = 12.0, max_reps: int = 8) -> dict:
    """Times the fp64 oracle, as it stands, on this machine's host cores on the same layer: with all cores
    (mean of a few whole layers, per step), and once with a single thread (a child process with
    OMP_NUM_THREADS=1; skipped when one run would not fit the budget)."""
    import oracle
    oracle.build()
    reps, runs = 0, []
    t_all = time.perf_counter()
    while reps < max_reps and (time.perf_counter() - t_all) < budget_s:
        runs.append(oracle_layer_timed(wl, x))
        reps += 1
    t = statistics.mean(r["layer"] for r in runs)
    steps = {k: statistics.mean(r[k] for r in runs) for k in ("scores", "select", "compact")}
    out = {"value": wl.total_len / t, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
           "sample": "the whole layer (%d tokens), mean of %d run(s), %.2f s each" % (wl.total_len, reps, t),
           "seconds_per_step": steps}
    est_one = t * oracle.num_threads()
    if est_one <= 45.0:
        try:
            env = dict(os.environ, OMP_NUM_THREADS="1")
            r = subprocess.run([sys.executable, "-c", ONE_THREAD_CHILD % (ROOT, name)], env=env, capture_output=True,
                               text=True, timeout=240)
            d = json.loads(r.stdout.strip().splitlines()[-1])
            out["one_thread"] = {"value": wl.total_len / d["seconds"]["layer"], "unit": UNIT, "cores": d["threads"],
                                 "seconds_per_step": {k: d["seconds"][k] for k in ("scores", "select", "compact")}}
        except Exception as e:   # the all-core figure stands on its own
            out["one_thread"] = {"skipped": "%s" % (e,)}
    else:
        out["one_thread"] = {"skipped": "one single-threaded layer would take about %.0f s" % est_one}
    return out


LAYER_SEQUENCES = {
    # config 3: layers 0..14 on the full prompt (KV selection only), Token-Selective Propagation at layer 15,
    # layers 16..31 on the propagated tokens with the KV budget of the original prompt
    "llama8b_32k_sweep": lambda: [("layers 0-14 (L = 32768, KV only)", 15, W.llama8b_32k_sweep(), False, None),
                                  ("layer 15 (L = 32768, TSP)", 1, W.llama8b_32k_sweep(), True, None),
                                  ("layers 16-31 (L = 6553, KV only)", 16, W.llama8b_32k_sweep(), False, 6553)],
    # config 4: the layer after the TSP layer runs on the 26214 propagated tokens and keeps 13107 of them
    "llama8b_128k_post_tsp_layer": lambda: [("post-TSP layer (L = 26214, KV only)", 1, W.llama8b_128k(), False, 26214)],
}


def run_layer_sequence(args) -> None:
    """A sequence of layers of different kinds (the 32-layer sweep of config 3, the post-TSP layer of config 4):
    every kind is timed by itself like the default workload's step -- CUDA events on the launching stream,
    the L2 overwritten before every step because these inputs fit in it, the L2-warm figure beside it,
    per-kernel times from the library's hook -- and `ms_per_step` is the sum over the sequence."""
    import dataclasses
    import torch
    from paper_2502_01068_b200 import binding as B
    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream()
    warmup, steps = max(3, args.warmup), max(1, min(args.steps, 50))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    tdev = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).cuda()
    peaks = measured_peaks()
    sampler = ClockSampler(0)
    sampler.start()
    n0 = B.fastkv_kernel_launches()
    kinds, total_ms, total_warm, total_tokens, total_bytes = [], 0.0, 0.0, 0, 0
    kernel_tot = {}
    for label, count, wl, with_tsp, length in LAYER_SEQUENCES[args.workload]():
        if length is not None:
            wl = dataclasses.replace(wl, seq_lens=[length])
        if not with_tsp:
            wl = dataclasses.replace(wl, k_tsp=None)
        wl = dataclasses.replace(wl, k_kv=[min(wl.k_kv[0], wl.seq_lens[0])])
        x = W.make_layer(wl, with_hidden=with_tsp)
        L = wl.total_len
        shape = B.make_shape(total_len=L, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                             hidden_dim=wl.hidden_dim, window=wl.window, pool_kernel=wl.pool_kernel, pool_mode=wl.pool_mode)
        q, k, v = tdev(x.q_win), tdev(x.k), tdev(x.v)
        b_kv = B.make_budget(int(wl.k_kv[0]))
        ws = torch.empty(B.fastkv_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
        s_kv = torch.empty((wl.n_kv_heads, L), dtype=torch.float32, device="cuda")
        idx_kv = torch.empty((wl.n_kv_heads, b_kv.total), dtype=torch.int32, device="cuda")
        k_out = torch.empty((wl.n_kv_heads, b_kv.total, wl.head_dim), dtype=torch.int16, device="cuda")
        v_out = torch.empty_like(k_out)
        if with_tsp:
            hid, pos = tdev(x.hidden), tdev(x.pos)
            b_tsp = B.make_budget(int(wl.k_tsp[0]))
            s_tsp = torch.empty((L,), dtype=torch.float32, device="cuda")
            idx_tsp = torch.empty((b_tsp.total,), dtype=torch.int32, device="cuda")
            hid_out = torch.empty((b_tsp.total, wl.hidden_dim), dtype=torch.int16, device="cuda")
            pos_out = torch.empty((b_tsp.total,), dtype=torch.int32, device="cuda")

            def step():
                B.fastkv_score(shape, q, k, s_kv, s_tsp, ws, stream)
                B.fastkv_select(shape, s_kv, b_kv, idx_kv, s_tsp, b_tsp, idx_tsp, ws, stream)
                B.fastkv_compact(shape, idx_kv, b_kv, idx_tsp, b_tsp, k, v, hid, pos, k_out, v_out, hid_out, pos_out, ws, stream)
        else:
            def step():
                B.fastkv_score(shape, q, k, s_kv, None, ws, stream)
                B.fastkv_select_kv(shape, s_kv, b_kv, idx_kv, ws, stream)
                B.fastkv_compact(shape, idx_kv, b_kv, None, None, k, v, None, None, k_out, v_out, None, None, ws, stream)

        for _ in range(warmup):
            step()
        torch.cuda.synchronize()
        status, site = B.fastkv_device_status(ws)
        if status != 0:
            raise SystemExit("device status %d at site %d (%s)" % (status, site, label))

        def timed(with_flush: bool) -> float:
            ts = []
            for _ in range(steps):
                if with_flush:
                    flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                step()
                e1.record(stream)
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1))
            return statistics.median(ts)

        ms, ms_warm = timed(True), timed(False)
        B.fastkv_debug_set("time_kernels", 1)
        for _ in range(steps):
            flush.zero_()
            step()
        torch.cuda.synchronize()
        B.fastkv_debug_set("time_kernels", 0)
        kernel_ms = {}
        for kid, kname in KERNELS.items():
            _name, kms, cnt = B.fastkv_debug_kernel_time(kid)
            if cnt:
                kernel_ms[kname] = kms / cnt
                kernel_tot[kname] = kernel_tot.get(kname, 0.0) + count * kms / cnt
        ab = algorithmic_bytes(wl)
        kinds.append({"layers": label, "count": count, "tokens": L, "k_kv": int(wl.k_kv[0]),
                      "k_tsp": int(wl.k_tsp[0]) if with_tsp else None, "ms": ms, "ms_l2_warm": ms_warm,
                      "kernels_ms": kernel_ms, "bytes_rw": ab["step_rw"],
                      "frac_of_measured": ab["step_rw"] / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]})
        total_ms += count * ms
        total_warm += count * ms_warm
        total_tokens += count * L
        total_bytes += count * ab["step_rw"]
    launches = B.fastkv_kernel_launches() - n0
    clocks = sampler.stop()
    dominant = max(kernel_tot, key=kernel_tot.get)
    gbs = total_bytes / (total_ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": METRIC, "value": total_tokens / (total_ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": steps,
        "warmup": warmup, "ms_per_step": total_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "step": "every layer of the sequence once (sum of count x median time of its kind)",
                   "n_q_heads": 32, "n_kv_heads": 8, "head_dim": 128, "hidden_dim": 4096, "window": 8, "pool_kernel": 7,
                   "l2": "L2 overwritten (256 MB write) before every step, not timed: these inputs fit in L2"},
        "clocks": clocks, "gpu_launches": int(launches), "e2e": None,
        "roofline": {"bound": "hbm", "kernel": KERNEL_SYMBOLS[dominant], "achieved": gbs, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "peak_source": peaks["source"],
                     "algorithmic_bytes": total_bytes, "traffic": None,
                     "note": "whole sequence on its read + write bytes: below 64K tokens the step is bound by kernel "
                             "launch and dependency latencies, not by one kernel; the dominant kernel by time is named"},
        "l2_warm": {"ms_per_step": total_warm, "value": total_tokens / (total_warm * 1e-3)},
        "kernels_ms": kernel_tot, "layers": kinds}))


def run_reference(args) -> None:
    """--impl reference: the oracle is the reference arm (no reference implementation exists)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from oracle.layer import layer_step
    oracle.build()
    wl = pick_workload(args.workload)
    x = W.make_layer(wl)

    def one():
        layer_step(x.q_win, x.k, x.v, x.hidden, x.pos, x.cu_seqlens, wl.window, wl.pool_kernel, wl.k_kv, wl.k_tsp,
                   pool_mode=wl.pool_mode)

    # each step is the whole layer; steps are capped so that the run ends within a few minutes
    t0 = time.perf_counter()
    one()
    first = time.perf_counter() - t0
    warm = max(0, min(args.warmup, int(20.0 / max(first, 1e-3)) - 1))
    steps = max(1, min(args.steps, int(90.0 / max(first, 1e-3))))
    for _ in range(warm):
        one()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    dt = (time.perf_counter() - t0) / steps
    value = wl.total_len / dt
    sample = "the whole layer per step; %d timed step(s) of %.2f s (requested %d)" % (steps, dt, args.steps)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(args.workload, wl),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="llama8b_128k_tsp_layer")
    ap.add_argument("--impl", default="fastkv", choices=["fastkv", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--min-region-s", type=float, default=0.5,
                    help="the K-step timed region is repeated until this much device time has been measured")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tp", action="store_true",
                    help="with N > 1: also time the tensor-parallel form (KV heads sharded, one all-reduce of S_tsp)")
    ap.add_argument("--no-decode", action="store_true",
                    help="skip the decode-time attention over the compact cache the step produced")
    ap.add_argument("--no-prefill", action="store_true",
                    help="skip the prefill attention that hands out the same scores as a by-product")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.workload in LAYER_SEQUENCES:
        run_layer_sequence(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))      # one rank per GPU; rank 0 prints the line

    import torch
    from paper_2502_01068_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    warmup = max(3, args.warmup)
    steps = max(1, args.steps)

    wl = pick_workload(args.workload)
    x = W.make_layer(wl, layer=rank)                      # each rank owns an independent layer
    lens, Bn, total = wl.seq_lens, wl.batch, wl.total_len
    tdev = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).cuda()
    d_cu = tdev(x.cu_seqlens) if Bn > 1 else None
    shape = B.make_shape(total_len=total, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                         hidden_dim=wl.hidden_dim, window=wl.window, pool_kernel=wl.pool_kernel,
                         pool_mode=wl.pool_mode, batch=Bn, max_len=max(lens), cu_seqlens=d_cu)
    q, k, v, hid, pos = tdev(x.q_win), tdev(x.k), tdev(x.v), tdev(x.hidden), tdev(x.pos)

    def budget(ks):
        if len(set(ks)) == 1:
            return B.make_budget(int(ks[0]), batch=Bn), None
        cu_k = tdev(np.concatenate([[0], np.cumsum(ks)]).astype(np.int32))
        return B.make_budget(0, cu_k=cu_k, total=int(sum(ks))), cu_k

    b_kv, _keep1 = budget(wl.k_kv)
    b_tsp, _keep2 = budget(wl.k_tsp)
    ws = torch.empty(B.fastkv_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    s_kv = torch.empty((wl.n_kv_heads, total), dtype=torch.float32, device="cuda")
    s_tsp = torch.empty((total,), dtype=torch.float32, device="cuda")
    idx_kv = torch.empty((wl.n_kv_heads, b_kv.total), dtype=torch.int32, device="cuda")
    idx_tsp = torch.empty((b_tsp.total,), dtype=torch.int32, device="cuda")
    k_out = torch.empty((wl.n_kv_heads, b_kv.total, wl.head_dim), dtype=torch.int16, device="cuda")
    v_out = torch.empty_like(k_out)
    hid_out = torch.empty((b_tsp.total, wl.hidden_dim), dtype=torch.int16, device="cuda")
    pos_out = torch.empty((b_tsp.total,), dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()
    input_bytes = x.k.nbytes + x.v.nbytes + x.hidden.nbytes
    fits_l2 = x.k.nbytes + x.q_win.nbytes <= L2_BYTES       # then "HBM GB/s" needs an L2 flush between steps
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if fits_l2 else None

    def step():
        B.fastkv_score(shape, q, k, s_kv, s_tsp, ws, stream)
        B.fastkv_select(shape, s_kv, b_kv, idx_kv, s_tsp, b_tsp, idx_tsp, ws, stream)   # select_kv + select_tsp
        B.fastkv_compact(shape, idx_kv, b_kv, idx_tsp, b_tsp, k, v, hid, pos, k_out, v_out, hid_out, pos_out, ws,
                         stream)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    status, site = B.fastkv_device_status(ws)
    if status != 0:
        raise SystemExit("device status %d at site %d after warm-up" % (status, site))

    def timed_region() -> float:
        """Exactly K steps, device-timed from the first launch to the last kernel's end, in ms.  Workloads whose
        inputs fit in L2 get the L2 overwritten before every step (not timed) and are timed step by step."""
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        torch.cuda.synchronize()
        if flush is None:
            t0.record(stream)
            for _ in range(steps):
                step()
            t1.record(stream)
            torch.cuda.synchronize()
            ms = t0.elapsed_time(t1)
        else:
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
            for a, b in ev:
                flush.zero_()
                a.record(stream)
                step()
                b.record(stream)
            torch.cuda.synchronize()
            ms = sum(a.elapsed_time(b) for a, b in ev)
        barrier()
        return ms

    # ---- timed region: K steps, repeated until enough device time has been measured; the median repeat is reported -----
    sampler = ClockSampler(local_rank)
    launches0 = B.fastkv_kernel_launches()
    sampler.start()
    region_ms = [timed_region()]
    launches = B.fastkv_kernel_launches() - launches0
    n_rep = int(min(400, max(1, np.ceil(args.min_region_s * 1e3 / max(region_ms[0], 1e-3)))))
    n_rep = int(max_over_ranks(n_rep, world, "cuda"))
    for _ in range(n_rep - 1):
        region_ms.append(timed_region())
    region_ms = [max_over_ranks(t, world, "cuda") for t in region_ms]
    total_ms = statistics.median(region_ms)
    ms_per_step = total_ms / steps
    value = whole_job_throughput(total, world, ms_per_step)

    # ---- L2-warm variant for the workloads that fit in L2 (same K steps back to back, no flush) -------------------------
    warm_ms = None
    if flush is not None:
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0.record(stream)
        for _ in range(steps):
            step()
        t1.record(stream)
        torch.cuda.synchronize()
        warm_ms = max_over_ranks(t0.elapsed_time(t1), world, "cuda") / steps

    # ---- the same K steps with a pair of events around every kernel (the library's own hook): per-kernel durations.
    # An event between two kernels keeps the second from starting under the first one's tail (programmatic dependent
    # launch), so these add up to a little more than a step of the timed region.
    B.fastkv_debug_set("time_kernels", 1)
    for _ in range(steps):
        if flush is not None:
            flush.zero_()
        step()
    torch.cuda.synchronize()
    B.fastkv_debug_set("time_kernels", 0)
    clocks = sampler.stop()
    kernel_ms = {}
    for kid, kname in KERNELS.items():
        _, ms, n = B.fastkv_debug_kernel_time(kid)
        if n:
            kernel_ms[kname] = ms / n

    # ---- end to end through the host-buffer entry point (pinned host memory, copies timed) -------------
    e2e = None
    uniform = len(set(wl.k_kv)) == 1 and len(set(wl.k_tsp)) == 1
    if uniform and args.e2e_steps > 0:
        pin = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
        hq, hk, hv, hh, hp = pin(x.q_win), pin(x.k), pin(x.v), pin(x.hidden), pin(x.pos)
        kk, kt = int(wl.k_kv[0]), int(wl.k_tsp[0])
        o_idx_kv = torch.empty((wl.n_kv_heads, Bn * kk), dtype=torch.int32).pin_memory()
        o_idx_tsp = torch.empty((Bn * kt,), dtype=torch.int32).pin_memory()
        o_k = torch.empty((wl.n_kv_heads, Bn * kk, wl.head_dim), dtype=torch.int16).pin_memory()
        o_v = torch.empty_like(o_k).pin_memory()
        o_h = torch.empty((Bn * kt, wl.hidden_dim), dtype=torch.int16).pin_memory()
        o_p = torch.empty((Bn * kt,), dtype=torch.int32).pin_memory()
        hshape = B.make_shape(total_len=total, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
                              head_dim=wl.head_dim, hidden_dim=wl.hidden_dim, window=wl.window,
                              pool_kernel=wl.pool_kernel, pool_mode=wl.pool_mode, batch=Bn, max_len=max(lens),
                              cu_seqlens=x.cu_seqlens if Bn > 1 else None)
        arena = torch.empty(B.fastkv_layer_host_arena_bytes(hshape, kk, kt), dtype=torch.uint8, device="cuda")

        def host_step():
            B.fastkv_layer_host(hshape, kk, kt, hq, hk, hv, hh, hp, o_idx_kv, o_idx_tsp, o_k, o_v, o_h, o_p, arena,
                                stream)

        host_step()
        barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            host_step()                                   # synchronises: outputs are on the host
        e2e_s = (time.perf_counter() - t0) / args.e2e_steps
        e2e_s = max_over_ranks(e2e_s, world, "cuda")
        h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv, hh, hp))
        d2h = sum(t.numel() * t.element_size() for t in (o_idx_kv, o_idx_tsp, o_k, o_v, o_h, o_p))
        e2e = {"value": world * total / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "ms_per_step": e2e_s * 1e3, "steps": args.e2e_steps}
        same = (np.array_equal(o_idx_tsp.numpy(), idx_tsp.cpu().numpy()) and
                np.array_equal(o_idx_kv.numpy(), idx_kv.cpu().numpy()) and
                np.array_equal(o_k.numpy(), k_out.cpu().numpy()) and np.array_equal(o_h.numpy(), hid_out.cpu().numpy()))
        if not same:
            raise SystemExit("host-buffer path and device path disagree")

    # ---- optional: tensor-parallel form of the same layer (KV heads sharded, one all-reduce of S_tsp) -------------------
    tp = None
    if args.tp and world > 1 and Bn == 1 and wl.n_kv_heads % world == 0:
        from paper_2502_01068_b200.tp import CudaBackend, HeadShard, shard_heads, tp_layer_step
        x0 = W.make_layer(wl, layer=0)                     # every rank draws the same layer and keeps its heads
        shard = HeadShard(rank, world, wl.n_q_heads, wl.n_kv_heads)
        backend = CudaBackend(shard, total, wl.head_dim, wl.hidden_dim, wl.window, wl.pool_kernel, wl.pool_mode)
        tq, tk, tv = (shard_heads(tdev(a), r) for a, r in ((x0.q_win, shard.q_range), (x0.k, shard.kv_range),
                                                            (x0.v, shard.kv_range)))
        th, tpos = tdev(x0.hidden), tdev(x0.pos)
        kk, kt = int(wl.k_kv[0]), int(wl.k_tsp[0])
        for _ in range(3):
            out = tp_layer_step(backend, shard, tq, tk, tv, th, tpos, kk, kt)
        barrier()
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(steps):
            out = tp_layer_step(backend, shard, tq, tk, tv, th, tpos, kk, kt)
        t1.record(stream)
        torch.cuda.synchronize()
        tp_ms = max_over_ranks(t0.elapsed_time(t1), world, "cuda") / steps
        gathered = [torch.zeros_like(out[1]) for _ in range(world)]
        import torch.distributed as dist
        dist.all_gather(gathered, out[1])
        tp = {"ms_per_step": tp_ms, "value": total / (tp_ms * 1e-3), "unit": UNIT, "scaling": "strong",
              "kv_heads_per_rank": shard.local_kv_heads, "all_reduce_bytes": 4 * total,
              "same_idx_tsp_on_all_ranks": all(bool(torch.equal(g, out[1])) for g in gathered)}

    # ---- optional: decode-time attention of one new token over the compacted cache of this layer ------------------
    decode = None
    if not args.no_decode and len(set(wl.k_kv)) == 1:
        qd = torch.randn((Bn, wl.n_q_heads, wl.head_dim), device="cuda").to(torch.bfloat16).view(torch.int16)
        dws = torch.empty(B.fastkv_decode_attn_workspace_bytes(shape), dtype=torch.uint8, device="cuda")
        dout = torch.empty((Bn, wl.n_q_heads, wl.head_dim), dtype=torch.float32, device="cuda")
        dflush = flush if flush is not None else torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        times = []
        for i in range(13):
            dflush.zero_()                                # the cache alone would fit in L2
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            B.fastkv_decode_attn(shape, qd, k_out, v_out, b_kv, dout, None, dws, stream)
            e1.record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                times.append(e0.elapsed_time(e1))
        dms = statistics.median(times)
        dbytes = 2 * wl.n_kv_heads * b_kv.total * wl.head_dim * 2
        decode = {"ms": dms, "algorithmic_bytes": dbytes, "achieved_gbs": dbytes / (dms * 1e-3) / 1e9,
                  "frac_of_measured": dbytes / (dms * 1e-3) / 1e9 / measured_peaks()["hbm_gbs"],
                  "l2": "flushed between iterations (256 MB write)", "kept_per_head": int(wl.k_kv[0])}
    # ---- optional: the layer's own causal attention, which hands out the same scores as a by-product -----------------
    prefill = None
    if not args.no_prefill and rank == 0 and Bn == 1:
        L, Hq, Hkv, d = total, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
        q_full = torch.randn((L, Hq, d), device="cuda").to(torch.bfloat16).view(torch.int16)
        q_full[L - wl.window:] = q                          # the window rows are the layer's window queries
        pshape = B.make_shape(total_len=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, hidden_dim=wl.hidden_dim,
                              window=wl.window, pool_kernel=wl.pool_kernel, pool_mode=wl.pool_mode, q_layout=B.Q_FULL)
        pws = torch.empty(B.fastkv_prefill_workspace_bytes(pshape), dtype=torch.uint8, device="cuda")
        att_out = torch.empty((L, Hq, d), dtype=torch.int16, device="cuda")
        p_kv, p_tsp = torch.empty_like(s_kv), torch.empty_like(s_tsp)

        def timed(with_scores: bool) -> float:
            reps = 3 if L > 40000 else 10
            ts = []
            for i in range(reps + 1):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                B.fastkv_prefill_attention(pshape, q_full, k, v, att_out, p_kv if with_scores else None,
                                           p_tsp if with_scores else None, pws, stream)
                e1.record(stream)
                torch.cuda.synchronize()
                if i >= 1:
                    ts.append(e0.elapsed_time(e1))
            return statistics.median(ts)

        ms_with, ms_without = timed(True), timed(False)
        pstatus, psite = B.fastkv_device_status(pws)
        if pstatus != 0:
            raise SystemExit("prefill attention: device status %d at site %d" % (pstatus, psite))
        step()                                              # s_kv / s_tsp of the scoring path, same inputs
        torch.cuda.synchronize()
        rel = ((p_kv - s_kv).abs() / s_kv.abs().clamp_min(1e-30)).max().item()
        flops = 4.0 * d * Hq * (L * (L + 1) / 2.0)          # two contractions over the causal half
        peaks_ = measured_peaks()
        peak = peaks_["bf16_tflops_sustained"] if ms_with > 20.0 else peaks_["bf16_tflops"]
        prefill = {"kernel": "prefill_attn_kernel", "bound": "tensor", "ms": ms_with, "ms_attention_only": ms_without,
                   "byproduct_overhead_ms": ms_with - ms_without, "flops": flops,
                   "achieved": flops / (ms_with * 1e-3) / 1e12, "unit": "TFLOP/s", "peak": peak,
                   "peak_source": peaks_["source"] + (", sustained bf16 figure: the call runs for tens of milliseconds"
                                                      if ms_with > 20.0 else ", burst bf16 figure"),
                   "frac": flops / (ms_with * 1e-3) / 1e12 / peak,
                   "scores_kv_max_rel_diff_vs_scoring_path": rel}
        del q_full, att_out, pws
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    if rank != 0:
        return
    ab = algorithmic_bytes(wl)
    peaks = measured_peaks()
    kbytes = {"score": ab["score_kernel"], "pool": ab["pool_kernel"], "select": ab["select"], "compact": ab["compact"]}

    def roof(kname: str) -> dict:
        gbs = kbytes[kname] / (kernel_ms[kname] * 1e-3) / 1e9
        return {"bound": "hbm", "kernel": KERNEL_SYMBOLS[kname], "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": gbs / peaks["hbm_gbs"], "peak_source": peaks["source"], "algorithmic_bytes": kbytes[kname],
                "traffic": profiled_traffic(kname, args.workload), "ms": kernel_ms[kname],
                "share_of_kernel_time": kernel_ms[kname] / sum(kernel_ms.values())}

    dominant = max(kernel_ms, key=kernel_ms.get)
    step_gbs = ab["step_rw"] / (ms_per_step * 1e-3) / 1e9
    config = config_of(args.workload, wl)
    config["l2"] = ("L2 overwritten (256 MB write) before every step, not timed: the inputs (%.0f MB of K) fit in L2"
                    % (x.k.nbytes / 1e6)) if flush is not None else (
        "inputs larger than L2 (K %.0f MB, hidden %.0f MB per step)" % (x.k.nbytes / 1e6, x.hidden.nbytes / 1e6))
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": config,
        "repeats": {"n": len(region_ms), "ms_per_step_median": ms_per_step, "ms_per_step_min": min(region_ms) / steps,
                    "ms_per_step_max": max(region_ms) / steps,
                    "ms_times_sm_mhz": ms_per_step * clocks["sm_mhz"] if clocks.get("sm_mhz") else None},
        "clocks": clocks,
        "gpu_launches": int(launches),
        "e2e": e2e,
        "roofline": roof(dominant),
        "roofline_compact": roof("compact") if "compact" in kernel_ms else None,
        "step_roofline": {"bytes_rw": ab["step_rw"], "bytes_rows_once": ab["step_min"], "achieved_gbs": step_gbs,
                          "frac_of_measured": step_gbs / peaks["hbm_gbs"],
                          "frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS,
                          "rows_once_gbs": ab["step_min"] / (ms_per_step * 1e-3) / 1e9},
        "kernels_ms": kernel_ms,
    }
    if warm_ms is not None:
        line["l2_warm"] = {"ms_per_step": warm_ms, "value": whole_job_throughput(total, world, warm_ms)}
    if tp is not None:
        line["tensor_parallel"] = tp
    if decode is not None:
        line["decode_attn"] = decode
    if prefill is not None:
        line["prefill_attn"] = prefill
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = oracle_baseline(args.workload, wl, x)
    print(json.dumps(line))


if __name__ == "__main__":
    main()
