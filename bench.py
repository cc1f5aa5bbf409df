#!/usr/bin/env python
"""Benchmark of the similarity-join hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

One "step" is one pass of the whole hot path (norm pre-pass where the kind needs
it, tile streaming, tile products, fused threshold + compaction, counter read-back)
over one synthetic workload through ``simjoin_run`` of the C-ABI library.  The
default workload is the throughput-headline configuration (inner-product join,
n = m = 1 048 576, d = 128, int8 +-1, t = 100).  Rank 0 prints ONE JSON line.

Metric: pair-TOPS = 2*n*m*d / time.  With N > 1 ranks (torchrun) every rank joins
its own row block of P against a replicated Q (weak scaling, no data-path
collective); the value is the ops of all ranks over the slowest rank's time.

``--impl reference`` times the CPU oracle (as it stands) on a bounded row slab of
the same workload on the host cores.

Two side modes time the widened entry points on synthetic data and say so in their line (they are not the
headline metric): ``--lsh L,k[,L_low]`` the LSH-bucketed join (``simjoin_run_lsh``, ``--lsh-family``) of the
configuration, ``--jl n,d,k`` the JL transform (``simjoin_jl_transform``) with an HBM roofline.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2006_12608_b200 import workloads as W  # noqa: E402

METRIC = "join pair-TOPS (2*n*m*d/s)"
UNIT = "TOPS"
NOMINAL_TOPS = {"i8": 4500.0, "bf16": 2250.0}          # dense, per GPU (context only)
# DRAM bytes per join-kernel launch (dram__bytes_read.sum + dram__bytes_write.sum), from a one-pass ncu
# capture of the full-size launch (profiles/join_kernel_dram_traffic_cfg4_full.md).
NCU_TRAFFIC_BYTES = {4: 690.11e6 + 5.89e6}
# the same for all levels of one JL transform call, keyed by (n, d, k) (profiles/jl_transform_*.md)
# captured at n = 262144 (1.2956e9 read + 0.6277e9 written); the 1 048 576-point entry is that x 4 (every level's
# traffic is proportional to n)
NCU_JL_TRAFFIC_BYTES = {(262144, 1024, 64): 1923.3e6, (1048576, 1024, 64): 4 * 1923.3e6}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p["bf16_tflops_sustained"]), "source": "measured"}
    except (OSError, KeyError, ValueError):
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        import torch
        self.gpu_id = str(device_index)
        try:
            self.gpu_id = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
        except Exception:
            pass
        self.proc = None
        self.lines = []
        self.first = 0
        self.thread = None

    def start(self, wait_first: float = 3.0):
        """Start sampling every 50 ms and wait (at most `wait_first` seconds) for the first sample, so that a short
        timed region is not over before nvidia-smi has come up; samples taken before mark() are dropped."""
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()
        t0 = time.perf_counter()
        while not self.lines and time.perf_counter() - t0 < wait_first:
            time.sleep(0.01)
        self.mark()

    def mark(self):
        """The timed region starts now: forget what was sampled before."""
        self.first = len(self.lines)

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        if self.thread:
            self.thread.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines[self.first:]:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[2:6]):
                if v == "Active":
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_slab(w, rows: int):
    """Time the CPU oracle on the first `rows` rows of P against all of Q. Returns (seconds, count, threads)."""
    from oracle import simjoin_oracle as O
    t0 = time.perf_counter()
    _pairs, cnt = O.join(w.P[:rows], w.Q, w.kind, w.threshold, w.dtype)
    return time.perf_counter() - t0, cnt, O.max_threads()


def slab_rows_for(w, seconds: float) -> int:
    """Rows of P whose oracle join takes roughly `seconds` (rates measured on 8 cores: ~25 GMAC/s
    int8, ~3.3 GMAC/s bf16/fp64; scaled by the core count)."""
    cores = os.cpu_count() or 1
    rate = (25e9 if w.dtype == "i8" else 3.3e9) * cores / 8.0
    rows = int(seconds * rate / (w.m * w.d))
    return max(1, min(w.n, rows))


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import simjoin_oracle as O
    O.build()
    rows = slab_rows_for(w, 4.0)
    times = []
    for it in range(args.warmup + args.steps):
        dt, _cnt, threads = oracle_slab(w, rows)
        if it >= args.warmup:
            times.append(dt)
    total = sum(times)
    ops_per_step = 2.0 * rows * w.m * w.d
    value = ops_per_step * len(times) / total / 1e12
    sample = f"first {rows} rows of P x all {w.m} rows of Q per step (the oracle's cost is linear in rows)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int64" if w.dtype == "i8" else "f64", "data": "synthetic",
            "config": {"workload": w.name, "n": w.n, "m": w.m, "d": w.d, "kind": w.kind, "threshold": w.threshold,
                       "sample_rows": rows},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def jl_level_dims(d: int, k: int):
    """Coordinates per point before level 1 and after every level of the JL transform (zeta = 2)."""
    levels = int(round(np.log2(d // k)))
    dims = [d]
    for i in range(1, levels + 1):
        dims.append((1 << (levels - i)) * (i * k if i < levels else k))
    return dims


def run_jl(args):
    """--jl n,d,k: the JL transform of Section 3 (simjoin_jl_transform) on n synthetic bf16 points; HBM-bound.
    Algorithmic bytes per call: every level reads its input once and writes its output once."""
    import torch
    from paper_2006_12608_b200 import binding as B
    from paper_2006_12608_b200 import build
    n, d, k = args.jl
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the transform has no CPU path")
    if not os.path.exists(B.LIB_PATH):
        build.build()
    torch.cuda.set_device(0)
    gen = torch.Generator(device="cuda").manual_seed(2006)
    X = torch.randn((n, d), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    out = torch.empty((n, k), dtype=torch.bfloat16, device="cuda")
    ctx = B.Simjoin("bf16", 0)

    def step():
        st = ctx.simjoin_jl_transform(X, n, d, k, 2006, out)
        if st != B.SIMJOIN_OK:
            raise RuntimeError(f"simjoin_jl_transform: {B.strerror(st)}")

    for _ in range(args.warmup):
        step()
    ratio = float((out.float().norm(dim=1) / X.float().norm(dim=1)).mean())       # JL: close to 1
    sampler = ClockSampler(0)
    torch.cuda.synchronize()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    kernel_ms = []
    e0.record()
    for _ in range(args.steps):
        step()
        kernel_ms.append(ctx.simjoin_last_kernel_ms()[2])
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms_per_step = e0.elapsed_time(e1) / args.steps
    dims = jl_level_dims(d, k)
    byts = sum(2.0 * n * (a + b) for a, b in zip(dims, dims[1:]))
    peaks = measured_peaks()
    km = statistics.mean(kernel_ms)
    achieved = byts / (km * 1e-3) / 1e9
    line = {"metric": "JL transform algorithmic GB/s (level inputs + outputs, bf16)", "value": byts / (ms_per_step * 1e-3) / 1e9,
            "unit": "GB/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"jl_bf16_{n}x{d}_to_{k}", "n": n, "d": d, "k": k, "levels": len(dims) - 1,
                       "level_dims": dims, "mean_norm_ratio": ratio, "l2": "input larger than L2; no flush",
                       "note": "not the headline metric: the dimensionality reduction of Section 3"},
            "clocks": clocks, "e2e": None, "gpu_launches": 2 * (len(dims) - 1) * args.steps,
            "roofline": {"bound": "hbm", "kernel": "join_kernel (store epilogue), all levels", "achieved": achieved,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                         "traffic": NCU_JL_TRAFFIC_BYTES.get((n, d, k)), "peak_source": f"{peaks['source']}: copy bandwidth",
                         "kernel_ms": km, "algorithmic_bytes": byts}}
    print(json.dumps(line), flush=True)


def run_jl_join(args):
    """--jl-join n,d,k[,slack]: the Euclidean join behind a JL pre-reduction (simjoin_run_jl_l2) on the config-2 recipe
    at dimension d (unit rows, 5000 planted near pairs, r = 0.45), timed beside the direct join of the same points."""
    import torch
    from paper_2006_12608_b200 import binding as B
    from paper_2006_12608_b200 import build
    n, d, k = (int(x) for x in args.jl_join[:3])
    slack = float(args.jl_join[3]) if len(args.jl_join) > 3 else 0.3
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the join has no CPU path")
    if not os.path.exists(B.LIB_PATH):
        build.build()
    torch.cuda.set_device(0)
    w = W.make_workload(2, n=n, m=n, d=d, planted=5000)
    r = 0.45
    ctx = B.Simjoin("bf16", 0)
    dP, dQ = B.to_device(w.P), B.to_device(w.Q)
    cap = 1 << 22
    out = torch.empty((cap, 2), dtype=torch.int32, device="cuda:0")

    def timed(fn):
        ts = []
        for it in range(args.warmup + args.steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            st, cnt = fn()
            e1.record()
            torch.cuda.synchronize()
            if st != B.SIMJOIN_OK:
                raise RuntimeError(B.strerror(st))
            if it >= args.warmup:
                ts.append(e0.elapsed_time(e1))
        got = out[:cnt].cpu().numpy().astype(np.int64)
        return statistics.mean(ts), (got[:, 0] << 32) | got[:, 1]

    direct_ms, exact = timed(lambda: ctx.simjoin_run(dP, n, dQ, n, d, "l2", r, out, cap))
    sampler = ClockSampler(0)
    sampler.start()
    ms, got = timed(lambda: ctx.simjoin_run_jl_l2(dP, n, dQ, n, d, r, k, 2006, slack, out, cap))
    clocks = sampler.stop()
    _st, jl_ms, rest_ms = ctx.simjoin_last_kernel_ms()
    ctx.close()
    ops = 2.0 * n * n * d
    line = {"metric": METRIC, "value": ops / (ms * 1e-3) / 1e12, "unit": UNIT, "n_gpus": 1, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"cfg2 recipe at d={d}, {n} x {n}, l2 r={r}", "n": n, "m": n, "d": d, "kind": "l2",
                       "threshold": r, "pairs_found": int(len(got))},
            "clocks": clocks, "e2e": None, "gpu_launches": None, "roofline": None,
            "algorithm": {"name": "JL pre-reduction + join + candidate filter (simjoin_run_jl_l2)", "k": k, "slack": slack,
                          "jl_ms": jl_ms, "reduced_join_and_filter_ms": rest_ms, "direct_join_ms": direct_ms,
                          "speedup_over_direct_join": direct_ms / ms,
                          "recall_of_the_direct_join": float(np.isin(exact, got).mean()) if len(exact) else None,
                          "false_pairs": int((~np.isin(got, exact)).sum()),
                          "note": "value = 2*n*m*d of the ORIGINAL dimension over the pipeline's time: the brute-force-"
                                  "equivalent rate of an approximate join, not the headline metric"}}
    print(json.dumps(line), flush=True)


def size_kw(args):
    kw = {}
    if args.n is not None:
        kw["n"] = args.n
    if args.m is not None:
        kw["m"] = args.m
    if args.planted is not None and args.config != 5:
        kw["planted"] = args.planted
    if args.d is not None:
        kw["d"] = args.d
    if args.threshold is not None:
        kw["threshold"] = args.threshold
    return kw


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=4, help="1..5, the benchmark configuration (default 4: the headline)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-per-config", action="store_true",
                    help="skip the per_config block (configurations 1, 2, 3, 5 at full size) and the int8 library peak")
    ap.add_argument("--per-config-seconds", type=float, default=0.6, help="length of each per_config timed region")
    ap.add_argument("--n", type=int, default=None, help="override the row count of P (profiling / experiments)")
    ap.add_argument("--m", type=int, default=None, help="override the row count of Q")
    ap.add_argument("--planted", type=int, default=None)
    ap.add_argument("--d", type=int, default=None, help="override the dimension (profiling other row lengths; give --threshold too)")
    ap.add_argument("--threshold", type=float, default=None)
    ap.add_argument("--kind", default=None, choices=["ip", "cos", "l2"],
                    help="join kind to run on the configuration's points instead of its own (give --threshold too)")
    ap.add_argument("--sigma-reading", default="radial")
    ap.add_argument("--seed", type=int, default=0, help="seed of the synthetic inputs (rank r of a sharded run draws its P block with seed + r)")
    ap.add_argument("--lsh", default=None, metavar="L,k[,L_low]",
                    help="time the LSH-bucketed join of the configuration instead of the brute-force join: "
                         "L tables of k bits (+ L_low of k-1); not the headline metric, the line says so")
    ap.add_argument("--lsh-family", default="bits", choices=["bits", "hyperplanes"],
                    help="hash family of --lsh: sampled coordinates, or random hyperplanes (keys computed on the tensor cores)")
    ap.add_argument("--jl", default=None, metavar="n,d,k",
                    help="time the JL transform (simjoin_jl_transform) of n bf16 points from d to k coordinates instead "
                         "of the join; HBM-bound, reported in algorithmic GB/s; not the headline metric")
    ap.add_argument("--jl-join", default=None, metavar="n,d,k[,slack]",
                    help="time the Euclidean join behind a JL pre-reduction (simjoin_run_jl_l2) beside the direct join; "
                         "reports speedup and recall; not the headline metric")
    args = ap.parse_args()
    if args.jl_join:
        args.jl_join = args.jl_join.split(",")
        if args.warmup < 3:
            args.warmup = 3
        if int(os.environ.get("RANK", "0")) == 0:
            run_jl_join(args)
        return
    if args.jl:
        args.jl = tuple(int(x) for x in args.jl.split(","))
        if args.warmup < 3:
            args.warmup = 3
        if int(os.environ.get("RANK", "0")) == 0:
            run_jl(args)
        return
    args.lsh = tuple(int(x) for x in args.lsh.split(",")) if args.lsh else None
    if args.lsh and args.impl == "reference":
        raise SystemExit("--lsh times the CUDA path only")
    if args.warmup < 3:
        args.warmup = 3

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        w = W.make_workload(args.config, seed=args.seed, sigma_reading=args.sigma_reading, **size_kw(args)) if rank == 0 else None
        if w is not None and args.kind:
            w.kind = args.kind
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2006_12608_b200 import binding as B
    from paper_2006_12608_b200 import build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the join has no CPU path")
    if rank == 0 and not os.path.exists(B.LIB_PATH):
        build.build()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    B.load()

    # Each rank owns one row block of a (world * n)-row P and a full copy of Q.
    w = W.make_workload(args.config, seed=args.seed + rank, sigma_reading=args.sigma_reading, **size_kw(args))
    if args.kind:
        w.kind = args.kind
    if world > 1:
        w.Q = W.make_workload(args.config, seed=args.seed, sigma_reading=args.sigma_reading, **size_kw(args)).Q if rank else w.Q
        w.planted = w.planted if rank == 0 else np.zeros((0, 2), np.int64)
    dev = torch.device("cuda", local_rank)
    dP, dQ = B.to_device(w.P, dev), B.to_device(w.Q, dev)
    same_cluster = None
    if w.cfg_id == 5 and args.sigma_reading == "radial":
        ncl = int(max(w.labels_p.max(), w.labels_q.max())) + 1
        same_cluster = int(np.sum(np.bincount(w.labels_p, minlength=ncl).astype(np.int64)
                                  * np.bincount(w.labels_q, minlength=ncl).astype(np.int64)))
    capacity = int(same_cluster * 1.05) if same_cluster else max(4 * len(w.planted), 1 << 20)
    out = torch.empty((capacity, 2), dtype=torch.int32, device=dev)
    ctx = B.Simjoin(w.dtype, local_rank)
    ctx.simjoin_set_offsets(rank * w.n, 0)


    def step():
        if args.lsh:
            L, k = args.lsh[0], args.lsh[1]
            st, cnt = ctx.simjoin_run_lsh(dP, w.n, dQ, w.m, w.d, w.threshold, L, k, 2006, out, capacity,
                                          L_low=args.lsh[2] if len(args.lsh) > 2 else 0, family=args.lsh_family, kind=w.kind)
        else:
            st, cnt = ctx.simjoin_run(dP, w.n, dQ, w.m, w.d, w.kind, w.threshold, out, capacity)
        if st != B.SIMJOIN_OK:
            raise RuntimeError(f"simjoin_run: {B.strerror(st)}")
        return cnt

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    cnt = 0
    for _ in range(args.warmup):
        cnt = step()
    # result sanity (not timed): every planted pair is in the output, nothing is duplicated
    got = out[:cnt].cpu().numpy().astype(np.int64)
    keys = (got[:, 0] << 32) | got[:, 1]
    if cnt <= (1 << 24):
        assert len(np.unique(keys)) == cnt, "duplicate pairs in the join output"
    if w.labels_p is not None and cnt:
        assert np.all(w.labels_p[got[:, 0] - rank * w.n] == w.labels_q[got[:, 1]]), "pair across clusters"
    args.recall = None
    if len(w.planted):
        pk = ((w.planted[:, 0] + rank * w.n) << 32) | w.planted[:, 1]
        if args.lsh:
            args.recall = float(np.isin(pk, keys).mean())       # the LSH join is approximate by design
        else:
            assert np.isin(pk, keys).all(), "a planted pair is missing from the join output"
    if same_cluster is not None and not args.lsh:
        assert cnt == same_cluster, (cnt, same_cluster)
    if same_cluster is not None and args.lsh:
        args.recall = cnt / same_cluster                          # every reported pair is a same-cluster pair (checked above)

    sampler = ClockSampler(local_rank)
    sync_all()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    join_ms, pre_ms = [], []
    e0.record()
    for _ in range(args.steps):
        step()
        _st, a, b = ctx.simjoin_last_kernel_ms()
        pre_ms.append(a)
        join_ms.append(b)
    e1.record()
    sync_all()
    clocks = sampler.stop()
    elapsed_ms = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([elapsed_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms = float(t.item())
    ms_per_step = elapsed_ms / args.steps
    value = world * w.ops / (ms_per_step * 1e-3) / 1e12

    e2e = None
    if not args.no_e2e and not args.lsh:
        e2e = measure_e2e(args, ctx, w, capacity, cnt, world, dev, sync_all)

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return
    finish(args, ctx, w, world, cnt, value, ms_per_step, join_ms, pre_ms, clocks, e2e)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def measure_e2e(args, ctx, w, capacity, cnt, world, dev, sync_all):
    """End to end: host buffers in, host pairs out, copies inside the timed region."""
    import torch
    import torch.distributed as dist
    from paper_2006_12608_b200 import binding as B
    hP = torch.from_numpy(w.P.view(np.int16) if w.P.dtype == np.uint16 else w.P).pin_memory()
    hQ = torch.from_numpy(w.Q.view(np.int16) if w.Q.dtype == np.uint16 else w.Q).pin_memory()
    hout = torch.empty((capacity, 2), dtype=torch.int32).pin_memory()
    e2e_steps = getattr(args, "e2e_steps", None) or max(1, min(args.steps, 5))

    def e2e_step():
        st, c = ctx.simjoin_run_host(hP, w.n, hQ, w.m, w.d, w.kind, w.threshold, hout, capacity)
        if st != B.SIMJOIN_OK:
            raise RuntimeError(f"simjoin_run_host: {B.strerror(st)}")
        return c

    e2e_step()
    sync_all()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        c2 = e2e_step()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    if world > 1:
        t = torch.tensor([e2e_s], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e_value = world * w.ops * e2e_steps / e2e_s / 1e12
    assert c2 == cnt
    return {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(w.P.nbytes + w.Q.nbytes),
            "d2h_bytes_per_step": int(cnt * 8 + 16), "steps": e2e_steps}


def roofline_of(w, kernel_ms, region_ms, clocks, peaks, int8_peak=None):
    """Roofline entry of the join kernel for workload w.  `frac` follows the measured-peak rule: the measured cuBLAS
    bf16 rate (sustained for a timed region of a quarter second and more, which runs at the power cap; burst below),
    times the nominal 2:1 ratio for int8.  That denominator is a library's rate, not the chip's ceiling, so three
    other readings go beside it: the share of the nominal dense peak, of the ceiling at the SM clock actually sampled
    (148 SMs x 8192 int8 (4096 bf16) multiply-adds per clock), and of an int8 library GEMM measured in this run."""
    achieved = w.ops / (kernel_ms * 1e-3) / 1e12
    ratio = 2.0 if w.dtype == "i8" else 1.0
    sustained = region_ms >= 250.0
    peak_key = "bf16_tflops_sustained" if sustained else "bf16_tflops"
    peak = peaks[peak_key] * ratio
    r = {"bound": "tensor", "kernel": "join_kernel", "achieved": achieved, "peak": peak, "unit": "TOP/s",
         "frac": achieved / peak, "traffic": NCU_TRAFFIC_BYTES.get(w.cfg_id) if (w.n, w.m) == (W.CONFIGS[w.cfg_id]["n"], W.CONFIGS[w.cfg_id]["m"]) else None,
         "peak_source": f"{peaks['source']}: cuBLAS bf16 {'sustained' if sustained else 'burst'} {peaks[peak_key]} TFLOP/s"
                        + (" x 2 (nominal int8:bf16 ratio)" if ratio == 2.0 else ""),
         "frac_of_nominal": achieved / NOMINAL_TOPS[w.dtype], "kernel_ms": kernel_ms}
    r["traffic_source"] = ("one-pass ncu capture of the full-size launch, profiles/join_kernel_dram_traffic_cfg4_full.md "
                           "(a constant of this file, not observed by this run)") if r["traffic"] else None
    if clocks.get("sm_mhz"):
        per_clk = 148 * (8192 if w.dtype == "i8" else 4096) * 2
        r["frac_of_clock_ceiling"] = achieved / (per_clk * clocks["sm_mhz"] * 1e6 / 1e12)
    if int8_peak and "burst_tops" in int8_peak and w.dtype == "i8":
        r["frac_of_int8_library_peak"] = achieved / int8_peak["sustained_tops" if sustained else "burst_tops"]
    return r


def measure_int8_library_peak(seconds: float = 4.0):
    """An int8 library GEMM on this GPU, measured the way the bf16 peaks were: torch._int_mm on 8192^3 ternary data,
    best of 10 single calls (burst) and back-to-back calls for `seconds` (sustained, at the power cap)."""
    import torch
    try:
        N = 8192
        gen = torch.Generator(device="cuda").manual_seed(7)
        a = torch.randint(-1, 2, (N, N), generator=gen, device="cuda", dtype=torch.int8)
        b = torch.randint(-1, 2, (N, N), generator=gen, device="cuda", dtype=torch.int8)
        ops = 2.0 * N * N * N
        for _ in range(3):
            torch._int_mm(a, b)
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch._int_mm(a, b)
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        reps = max(10, int(seconds * 1e3 / best))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            torch._int_mm(a, b)
        e1.record()
        torch.cuda.synchronize()
        return {"burst_tops": ops / (best * 1e-3) / 1e12, "sustained_tops": ops * reps / (e0.elapsed_time(e1) * 1e-3) / 1e12,
                "how": f"torch._int_mm {N}^3, ternary int8 data: best of 10 calls; {reps} calls back to back"}
    except Exception as exc:                       # the library call is context, never a reason to lose the line
        return {"unavailable": f"{type(exc).__name__}: {exc}"}


def measure_side_config(cfg_id, args, peaks, int8_peak, min_seconds):
    """One of the other configurations at full size, measured like the headline one: warm-up, a result check, a timed
    region of at least `min_seconds` (so that the clock sampler sees it), the kernel's own CUDA-event time, and a short
    end-to-end leg through simjoin_run_host."""
    import torch
    from paper_2006_12608_b200 import binding as B
    w = W.make_workload(cfg_id, sigma_reading=args.sigma_reading)
    dev = torch.device("cuda", 0)
    dP, dQ = B.to_device(w.P, dev), B.to_device(w.Q, dev)
    same_cluster = None
    if w.cfg_id == 5 and args.sigma_reading == "radial":
        ncl = int(max(w.labels_p.max(), w.labels_q.max())) + 1
        same_cluster = int(np.sum(np.bincount(w.labels_p, minlength=ncl).astype(np.int64)
                                  * np.bincount(w.labels_q, minlength=ncl).astype(np.int64)))
    capacity = int(same_cluster * 1.05) if same_cluster else max(4 * len(w.planted), 1 << 20)
    out = torch.empty((capacity, 2), dtype=torch.int32, device=dev)
    ctx = B.Simjoin(w.dtype, 0)

    def step():
        st, c = ctx.simjoin_run(dP, w.n, dQ, w.m, w.d, w.kind, w.threshold, out, capacity)
        if st != B.SIMJOIN_OK:
            raise RuntimeError(f"simjoin_run (config {cfg_id}): {B.strerror(st)}")
        return c

    cnt = 0
    for _ in range(3):
        cnt = step()
    # step time after the warm-up (first calls allocate and set kernel attributes), for sizing the timed region
    reps, t0 = 0, time.perf_counter()
    while reps < 2 or (time.perf_counter() - t0 < 0.02 and reps < 2000):
        step()
        reps += 1
    est = (time.perf_counter() - t0) / reps
    got = out[:cnt].cpu().numpy().astype(np.int64)
    keys = (got[:, 0] << 32) | got[:, 1]
    if cnt <= (1 << 24):
        assert len(np.unique(keys)) == cnt, "duplicate pairs in the join output"
    if len(w.planted):
        assert np.isin((w.planted[:, 0] << 32) | w.planted[:, 1], keys).all(), "a planted pair is missing"
    if same_cluster is not None:
        assert cnt == same_cluster and np.all(w.labels_p[got[:, 0]] == w.labels_q[got[:, 1]])
    del got, keys
    steps = max(5, int(np.ceil(min_seconds / max(est, 1e-6))))
    sampler = ClockSampler(0)
    torch.cuda.synchronize()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    join_ms, pre_ms = 0.0, 0.0
    e0.record()
    for _ in range(steps):
        step()
        _st, a, b = ctx.simjoin_last_kernel_ms()
        pre_ms += a
        join_ms += b
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    region_ms = e0.elapsed_time(e1)
    ms_per_step = region_ms / steps
    args_e2e = argparse.Namespace(steps=3, e2e_steps=int(min(2000, max(3, np.ceil(0.2 / max(est, 1e-6))))))
    e2e = measure_e2e(args_e2e, ctx, w, capacity, cnt, 1, dev, torch.cuda.synchronize)
    ctx.close()
    entry = {"workload": w.name, "n": w.n, "m": w.m, "d": w.d, "kind": w.kind, "in_dtype": w.dtype, "threshold": w.threshold,
             "steps": steps, "ms_per_step": ms_per_step, "kernel_ms": join_ms / steps, "prepass_ms": pre_ms / steps,
             "value": w.ops / (ms_per_step * 1e-3) / 1e12, "unit": UNIT, "pairs_found": int(cnt), "e2e": e2e, "clocks": clocks,
             "l2": ("inputs (P+Q) larger than L2; no flush" if w.P.nbytes + w.Q.nbytes > 126e6
                    else "inputs (P+Q) fit in L2 and are not flushed between steps")}
    if cfg_id == 1:
        entry["note"] = "latency-bound: one partial wave of tiles; its time is the figure, not a fraction of a peak"
    else:
        r = roofline_of(w, join_ms / steps, region_ms, clocks, peaks, int8_peak)
        entry.update({k: r[k] for k in ("frac", "frac_of_nominal", "peak", "peak_source") if k in r})
        for k in ("frac_of_clock_ceiling", "frac_of_int8_library_peak"):
            if k in r:
                entry[k] = r[k]
    del dP, dQ, out
    torch.cuda.empty_cache()
    return entry


def finish(args, ctx, w, world, cnt, value, ms_per_step, join_ms, pre_ms, clocks, e2e):
    peaks = measured_peaks()
    jm = statistics.mean(join_ms)
    side = world == 1 and not args.lsh and not args.no_per_config
    int8_peak = measure_int8_library_peak() if side else None
    roofline = roofline_of(w, jm, ms_per_step * args.steps, clocks, peaks, int8_peak)
    roofline["prepass_ms"] = statistics.mean(pre_ms)
    # the join (int8 and bf16 Euclidean: both variants are launched, one returns at once), the norm pre-pass, max|x|
    launches_per_step = (2 if (w.dtype == "i8" or w.kind == "l2") else 1) + (2 if w.kind != "ip" else 0) + (1 if w.dtype == "i8" else 0)
    # dense bf16 joins of short rows run on transformed copies of both point sets: two more launches
    blocks = -(-w.n // 32) * -(-w.m // 128)
    if w.dtype == "bf16" and (w.d + 8) * 2 <= 256 and cnt / blocks >= 1.0:
        launches_per_step += 2
    if args.lsh:
        # max|x| x2, sampled coordinates, keys x2, then per table: 2 histograms, offsets + work list, 2 scatters, 2 row
        # gathers, the join
        tables = args.lsh[0] + (args.lsh[2] if len(args.lsh) > 2 else 0)
        launches_per_step = 5 + 8 * tables
        roofline = None
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int32" if w.dtype == "i8" else "f32", "data": "synthetic",
            "config": {"workload": w.name, "n": w.n, "m": w.m, "d": w.d, "kind": w.kind, "in_dtype": w.dtype,
                       "threshold": w.threshold, "pairs_found": int(cnt), "seed": args.seed,
                       "l2": ("inputs (P+Q) larger than L2; no flush" if w.P.nbytes + w.Q.nbytes > 126e6
                              else "inputs (P+Q) fit in L2 and are not flushed between steps: not a headline number"),
                       "inputs_sha256": {"P": hashlib.sha256(w.P).hexdigest(), "Q": hashlib.sha256(w.Q).hexdigest()},
                       "sharding": f"P row blocks x{world}, Q replicated" if world > 1 else "single GPU",
                       "note": w.note},
            "clocks": clocks,
            "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline}
    if args.lsh:
        line["algorithm"] = {"name": "lsh-bucketed join (simjoin_run_lsh)", "family": args.lsh_family, "L": args.lsh[0], "k": args.lsh[1],
                             "L_low": args.lsh[2] if len(args.lsh) > 2 else 0, "recall_on_planted_pairs": args.recall,
                             "hash_ms": statistics.mean(pre_ms), "tables_ms": jm,
                             "note": "value = 2*n*m*d over the step time: the brute-force-equivalent rate of an approximate "
                                     "join, not the headline metric; precision is 1, recall as given"}
    if int8_peak is not None:
        line["int8_library_peak"] = int8_peak
    if side and args.config == 4 and not size_kw(args) and not args.kind:
        # the other four configurations at full size, each with its own clock record (the headline stays config 4)
        line["per_config"] = {str(c): measure_side_config(c, args, peaks, int8_peak, args.per_config_seconds) for c in (1, 2, 3, 5)}
    if not args.no_cpu_baseline and world == 1 and not args.lsh:
        rows = slab_rows_for(w, 12.0)
        dt, _c, threads = oracle_slab(w, rows)
        line["cpu_baseline"] = {"value": 2.0 * rows * w.m * w.d / dt / 1e12, "unit": UNIT, "cores": threads,
                                "kind": "oracle",
                                "sample": f"first {rows} rows of P x all {w.m} rows of Q, {dt:.1f} s "
                                          "(the oracle's cost is linear in rows)"}
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
