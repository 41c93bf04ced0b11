#!/usr/bin/env python
"""Benchmark of the SketchedAMSGrad step: `python bench.py --gpus N --steps K --warmup W`.

A step is one pass of the whole hot path (second moments on I_{t-1}, moments + Count Sketch of n workers,
sum of sketches, unsketch + top-k, apply + error feedback) over one batch of synthetic gradients that is
already resident in HBM.  The path does not shard (all n workers live on one GPU), so N > 1 runs N
independent replicas, one process per GPU, and reports the aggregate (weak scaling).

Prints ONE JSON line on rank 0.  `--impl reference` times the CPU oracle on the same workload instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "sketched_amsgrad_step_throughput"
UNIT = "Gcoord/s"
DEFAULT_WORKLOAD = "C3"      # d = 25.6M: the size the headline metric is quoted on

# DRAM traffic of the dominant kernel (moments + sketch) from an ncu capture, in bytes per worker-coordinate, valid
# only for the kernel source it was taken on (sha256 of the file); otherwise reported as null.  The traffic grows in
# proportion to n*d, so the capture (C3 at half size, see profiles/) is scaled to the timed launch.
NCU_TRAFFIC = {
    # shared-memory ownership kernel (windowed hash family, the default path)
    # capture: 1.2653 GB read + 0.8005 GB written for 1.024e8 worker-coordinates (profiles/c3_half_moment_sketch_own_ncu_full.md)
    "k_moment_sketch_own": {"file": "sk_sketch_own.cu", "sha256": "943a8f79d4234ea88447d157741e7beb5e9bf7c32ab37ea428bc7c65e07cc04c",
                            "bytes_per_worker_coord": 20.17},
    # L2-reduction kernel (plain hash family): 1.2540 GB read + 0.7948 GB written for 1.024e8 worker-coordinates
    "k_moment_sketch_v4": {"file": "sk_sketch.cu", "sha256": "22a40f26423a95e6b6fa606c5e4a3e3e111270585219b1883d76157e2977a1c0",
                           "bytes_per_worker_coord": 20.01},
}


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc = gpu_index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.gpu)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    @staticmethod
    def _stamp(text: str):
        import datetime
        try:
            return datetime.datetime.strptime(text, "%Y/%m/%d %H:%M:%S.%f").timestamp()
        except ValueError:
            return None

    def stop(self, windows=()):
        """windows: (t0, t1) wall-clock intervals (time.time()) of the timed repetitions; returns the summary over the
        samples inside them (all samples if none fall inside) and the median SM clock of every window."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out = self.proc.communicate(timeout=5)[0]
        except Exception:
            self.proc.kill()
            out = ""
        rows, mx = [], []
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                rows.append((self._stamp(f[0]), float(f[1]), [v.lower().startswith("active") for v in f[5:9]]))
                mx.append(float(f[2]))
            except ValueError:
                continue
        inside = [r for r in rows if r[0] is not None and any(a <= r[0] <= b for a, b in windows)]
        use = inside if inside else rows
        reasons = set()
        for _, _, flags in use:
            for name, on in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), flags):
                if on:
                    reasons.add(name)
        per_rep = []
        for a, b in windows:
            v = [r[1] for r in rows if r[0] is not None and a <= r[0] <= b]
            per_rep.append(statistics.median(v) if v else None)
        return {"sm_mhz": statistics.median([r[1] for r in use]) if use else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(rows), "samples_in_timed_region": len(inside),
                "sm_mhz_per_repetition": per_rep if len(per_rep) <= 20 else self._spread(per_rep)}

    @staticmethod
    def _spread(per_rep):
        seen = [v for v in per_rep if v is not None]
        return {"repetitions_with_samples": len(seen), "min": min(seen) if seen else None,
                "median": statistics.median(seen) if seen else None, "max": max(seen) if seen else None}


def _dist():
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return world, rank, local


def reduce_max(value: float, world: int, device) -> float:
    """Max over ranks (one number per rank); identity without a process group."""
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def reduce_sum(value: float, world: int, device) -> float:
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def default_family(c: int):
    """The library's default hash family for a row of c buckets: groups of 32 in windows of 8 lines when a row holds a
    window, else the plain family with the largest group that fits (restated here for the oracle's arguments)."""
    lg = 5
    while (1 << lg) > c:
        lg -= 1
    return lg, (8 if lg == 5 and c >= 256 else 0)


def cpu_oracle_rate(w, scale: int, steps: int, threads: int, variant: str = "ga", P: int = 1, family=None):
    """Times the CPU oracle, as it stands, on `steps` steps of the workload scaled down by `scale`.
    family: (log2g, window_lines) of the hash family (default: the library's default for the scaled row length)."""
    import oracle
    from paper_2210_07454_b200 import synthetic
    ws = synthetic.scaled(w, scale) if scale > 1 else w
    src = synthetic.GradientSource(ws, device="cpu", cfg_id=int(w.name[1]) if w.name[1:2].isdigit() else 9)
    lg, wl = family if family is not None else default_family(ws.c)
    if scale > 1 and (wl * 32 > ws.c or (1 << lg) > ws.c):
        lg, wl = default_family(ws.c)
    o = oracle.Oracle(ws.d, ws.n, ws.r, ws.c, ws.k, seed=ws.seed, log2g=lg, lr=ws.lr, beta1=ws.beta1, beta2=ws.beta2,
                      eps=ws.eps, threads=threads, variant=variant, P=P, window_lines=wl)
    x = src.x0().numpy()
    grads = [src.grads(t).numpy() for t in range(1, min(steps, 2) + 1)]
    times = []
    for t in range(steps):
        t0 = time.perf_counter()
        o.step(grads[t % len(grads)], x)
        times.append(time.perf_counter() - t0)
    o.close()
    size = "at full size" if scale == 1 else f"scaled 1/{scale}"
    sample = (f"{steps} step(s) of {w.name} {size} (d={ws.d}, n={ws.n}, r={ws.r}, c={ws.c}, k={ws.k}), "
              f"gcc -O2 OpenMP oracle, {threads} thread(s)")
    return ws, times, sample


def cpu_model() -> str:
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def run_reference(args, w):
    """The reference arm: there is no reference code, so it is the CPU oracle itself on all host cores.  Each step is
    one oracle step of the workload; at full size when the whole run then stays within a few minutes (probed on a
    1/16-size step first), else at the smallest power-of-two reduction that does."""
    world, rank, _ = _dist()
    if rank != 0:
        return
    threads = os.cpu_count() or 1
    total = args.steps + args.warmup
    scale = args.ref_scale
    if scale <= 0:                                    # automatic: full size if (steps + warmup) oracle steps fit the budget
        _, probe, _ = cpu_oracle_rate(w, 16, 2, threads, args.variant, args.P)
        full_step = 16.0 * probe[-1]
        scale = 1
        while total * full_step / scale > 200.0 and scale < 64:
            scale *= 2
    ws, times, sample = cpu_oracle_rate(w, scale, total, threads, args.variant, args.P)
    timed = times[args.warmup:]
    ms = 1e3 * sum(timed) / len(timed)
    value = ws.n * ws.d / (ms * 1e-3) / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "d": w.d, "n": w.n, "r": w.r, "c": w.c, "k": w.k,
                       "sampled_as": "each step is one oracle step at full size" if scale == 1
                       else f"each step is one oracle step at 1/{scale} size", "same_config": scale == 1,
                       "cpu": cpu_model()},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def quick_step_roofline(name: str, dev, peak: float, steps: int = 5, reps: int = 3):
    """A short run of another workload with the default options: step time (median of `reps` loops of `steps` steps
    after 3 warm-up steps, two rotating gradient sets, both far larger than L2) and its fraction of the roofline."""
    import torch
    from paper_2210_07454_b200 import binding, synthetic
    w = synthetic.WORKLOADS[name]
    src = synthetic.GradientSource(w, device=dev, cfg_id=int(w.name[1]))
    opt = binding.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=w.seed, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps)
    gsets = [src.grads(1), src.grads(2)]
    x = src.x0()
    for t in range(3):
        opt.step(gsets[t % 2], x)
    opt.sync()
    ms = []
    for _ in range(reps):
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for t in range(steps):
            opt.step(gsets[t % 2], x)
        ev1.record()
        torch.cuda.synchronize()
        ms.append(ev0.elapsed_time(ev1) / steps)
    opt.sync()
    ms_step = statistics.median(ms)
    b_alg = opt.algorithmic_bytes()
    out = {"d": w.d, "n": w.n, "r": w.r, "c": w.c, "k": w.k, "ms_per_step": ms_step, "steps": steps, "repetitions": reps,
           "value": w.n * w.d / (ms_step * 1e-3) / 1e9, "unit": UNIT, "algorithmic_bytes": b_alg,
           "achieved_gbs": b_alg / (ms_step * 1e-3) / 1e9, "frac": b_alg / (ms_step * 1e-3) / 1e9 / peak}
    del opt, gsets, x, src
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--log2g", type=int, default=None)
    ap.add_argument("--P", type=int, default=1,
                    help="candidate multiplier of the second selection round (Section III-A); 1 = no second round")
    ap.add_argument("--variant", default="ga", choices=["ga", "pa"],
                    help="ga = gradient averaging (Algorithm 2, the headline path); pa = parameter averaging (Algorithm 1)")
    ap.add_argument("--window-lines", type=int, default=None, help="windowed hash family: lines per window (0 = plain)")
    ap.add_argument("--window-workers", type=int, default=0, help="workers per launch of the windowed sketch kernel")
    ap.add_argument("--chained-launches", type=int, default=-1,
                    help="0: launch the step's kernels without programmatic dependent launch (the default is chained)")
    ap.add_argument("--worker-sum", type=int, default=-1, help="1: the sketch kernel leaves the worker sum of a_t for the update of x")
    ap.add_argument("--worker-chunk", type=int, default=0)
    ap.add_argument("--sketch-ctas", type=int, default=0, help="CTAs per SM of the sketch kernel (0 = default)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--ref-scale", type=int, default=0, help="reference arm: 1/SCALE size per step (0 = full size if it fits the time budget)")
    ap.add_argument("--reps", type=int, default=0,
                    help="repetitions of the --steps long timed loop, the median is reported; 0 = as many as fill about "
                         "half a second (at least 10, at most 400), so that the clock sampler sees the timed region")
    ap.add_argument("--no-other-workloads", action="store_true", help="skip the short C4 and C5 runs reported beside the headline")
    ap.add_argument("--scale", type=int, default=1, help="run the workload at 1/SCALE size (profiling captures)")
    ap.add_argument("--grad-sets", type=int, default=0, help="rotating gradient sets (0 = as many as fit, 2..4)")
    ap.add_argument("--partition-workers", action="store_true",
                    help="split the workload's n workers over the processes (one step = three phases with two "
                         "all-reduces between them) instead of running one full replica per process")
    ap.add_argument("--sum-sketch", action="store_true",
                    help="NOT the headline path: one sketch of the worker sum instead of n sketches and their sum")
    ap.add_argument("--grads-bf16", action="store_true", help="pass the gradients as bf16 (18 B per worker-coordinate)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-stage-timing", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2210_07454_b200 import synthetic
    w = synthetic.WORKLOADS[args.workload]
    cfg_id = int(w.name[1])
    if args.scale > 1:
        w = synthetic.scaled(w, args.scale)
    if args.impl == "reference":
        return run_reference(args, w)

    import torch
    from paper_2210_07454_b200 import binding
    world, rank, local = _dist()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        if args.partition_workers:                   # the communicator's set-up lines (ranks, transports) go to stderr
            os.environ.setdefault("NCCL_DEBUG", "INFO")
            os.environ.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
        dist.init_process_group("nccl", device_id=dev)

    n_all = w.n
    if args.partition_workers:                       # this process holds n / world of the workers; x is replicated
        assert w.n % world == 0, f"--partition-workers needs the workers ({w.n}) to divide by the processes ({world})"
        w = synthetic.Workload(**{**w.__dict__, "n": w.n // world})
    src = synthetic.GradientSource(w, device=dev, cfg_id=cfg_id + (100 * rank if args.partition_workers else 0))
    opt = binding.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=w.seed, lr=w.lr, beta1=w.beta1, beta2=w.beta2,
                                  eps=w.eps, log2g=args.log2g, window_lines=args.window_lines, variant=args.variant,
                                  P=args.P, workers_total=n_all if args.partition_workers else None)
    if args.sum_sketch:
        opt.set_option("sum_sketch", 1)
    if args.grads_bf16:
        opt.set_option("grads_bf16", 1)
    gbytes = 2 if args.grads_bf16 else 4
    step = opt.step
    if args.partition_workers:
        from paper_2210_07454_b200.partitioned import PartitionedStep
        step = PartitionedStep(opt, dev).step
    opt.set_option("worker_chunk", args.worker_chunk)
    if args.window_workers:
        opt.set_option("window_workers", args.window_workers)
    if args.sketch_ctas:
        opt.set_option("sketch_ctas_per_sm", args.sketch_ctas)
    if args.worker_sum >= 0:
        opt.set_option("worker_sum", args.worker_sum)
    if args.chained_launches >= 0:
        opt.set_option("chained_launches", args.chained_launches)
    # gradient buffers rotate so that no step finds its inputs in L2 (each set is far larger than L2 anyway)
    free_b, _ = torch.cuda.mem_get_info()
    set_bytes = gbytes * w.n * w.d
    nsets = args.grad_sets if args.grad_sets > 0 else int(max(2, min(4, (free_b * 0.5) // set_bytes)))
    gsets = [src.grads(t + 1) for t in range(nsets)]
    if args.grads_bf16:
        gsets = [g.to(torch.bfloat16) for g in gsets]
    x = src.x0()
    torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()                              # started early: nvidia-smi takes a while to deliver samples
    for t in range(args.warmup):
        step(gsets[t % nsets], x)
    opt.sync()
    opt.timing()                                     # clear launch counters
    opt.set_option("timing", 0)                      # the headline loop runs without per-stage events (they cost ~3 %)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()
    # the --steps long loop is timed `reps` times (CUDA events on the launching stream, barrier and synchronize on both
    # sides of every repetition, max over ranks); the median repetition is the reported step time
    rep_ms, windows = [], []
    reps = args.reps if args.reps > 0 else 10
    rep = 0
    while rep < reps:
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        ev0.record()
        for t in range(args.steps):
            step(gsets[(args.warmup + t) % nsets], x)
        ev1.record()
        torch.cuda.synchronize()
        windows.append((t0, time.time()))
        if world > 1:
            dist.barrier()
        rep_ms.append(reduce_max(ev0.elapsed_time(ev1), world, dev))
        rep += 1
        if args.reps <= 0 and rep == 1:              # every rank derives the same count from the reduced time
            reps = int(min(400, max(10, math.ceil(500.0 / max(rep_ms[0], 1e-3)))))
    clocks = sampler.stop(windows) if rank == 0 else None
    opt.sync()
    ms_total = statistics.median(rep_ms)
    _, _, stage_launches = opt.timing()              # launch counts of all timed repetitions
    launches = reduce_sum(float(sum(stage_launches)), world, dev)
    # per-stage times: the same steps once more with CUDA events around every stage (inside the library, on its stream)
    nsteps, stage_ms = 0, [0.0] * binding.NUM_STAGES
    if not args.no_stage_timing:
        opt.set_option("timing", 1)
        for t in range(args.steps):
            step(gsets[(args.warmup + t) % nsets], x)
        opt.sync()
        nsteps, stage_ms, stage_launches = opt.timing()
        opt.set_option("timing", 0)

    ms_step = ms_total / args.steps
    units = n_all * w.d if args.partition_workers else world * w.n * w.d     # worker-coordinates per step, whole job
    value = units / (ms_step * 1e-3) / 1e9
    peak, peak_kind = _peaks()
    b_alg = opt.algorithmic_bytes()

    # dominant kernel: moments + sketch.  Algorithmic bytes per launch: 20 B per worker-coordinate streamed
    # (read g, m, e; write m, e) plus the worker tables it fills (4 B per bucket).
    k1_launches = max(1, stage_launches[2])
    k1_bytes_step = ((20 if args.variant == "ga" else 36) - (4 - gbytes)) * w.n * w.d \
        + 4 * (1 if args.sum_sketch else w.n) * w.r * w.c
    roofline = None
    if not args.no_stage_timing and stage_ms[2] > 0:
        k1_ms = stage_ms[2] / k1_launches
        k1_bytes = k1_bytes_step * args.steps / k1_launches
        achieved = k1_bytes / (k1_ms * 1e-3) / 1e9
        windowed = bool(opt.get_option("window_lines")) and args.variant == "ga" and not args.sum_sketch
        kernel = "k_moment_sketch_pa_v4" if args.variant != "ga" else ("k_moment_sketch_own" if windowed else "k_moment_sketch_v4")
        traffic = None
        rec = NCU_TRAFFIC.get(kernel)
        if rec and rec["sha256"] and rec["bytes_per_worker_coord"] and not args.grads_bf16 and not args.sum_sketch \
                and args.P == 1 and args.worker_sum <= 0:
            path = os.path.join(ROOT, "paper_2210_07454_b200", "csrc", rec["file"])
            if hashlib.sha256(open(path, "rb").read()).hexdigest() == rec["sha256"]:
                traffic = rec["bytes_per_worker_coord"] * w.n * w.d * args.steps / k1_launches
        roofline = {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak,
                    "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak, "traffic": traffic,
                    "ms_per_launch": k1_ms, "launches_per_step": k1_launches / args.steps,
                    "algorithmic_bytes_per_launch": k1_bytes}

    # end to end through the host entry point: pinned host gradients in, x back out, every step
    e2e = None
    if args.e2e_steps > 0:
        hg = torch.empty((w.n, w.d), dtype=gsets[0].dtype, pin_memory=True)
        hg.copy_(gsets[0])
        hx = torch.empty(w.d, dtype=torch.float32, pin_memory=True)
        hx.copy_(x)
        if args.partition_workers:                    # the phases take device buffers: stage through torch copies
            gdev = gsets[0]

            def step_host(hgrads, hxx):
                gdev.copy_(hgrads, non_blocking=True)
                x.copy_(hxx, non_blocking=True)
                step(gdev, x)
                hxx.copy_(x)
        else:
            step_host = opt.step_host
        step_host(hg, hx)                             # warm-up (allocates the staging buffers)
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            step_host(hg, hx)
        torch.cuda.synchronize()
        dt = reduce_max(time.perf_counter() - t0, world, dev)
        e2e = {"value": units * args.e2e_steps / dt / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": gbytes * w.n * w.d + 4 * w.d, "d2h_bytes_per_step": 4 * w.d,
               "ms_per_step": 1e3 * dt / args.e2e_steps, "steps": args.e2e_steps}

    # the same through the sparse-return host step (Section III-B's pattern: parameters stay on the device, host
    # gradients in, k indices and values back); reported beside e2e, not instead of it
    e2e_sparse = None
    if args.e2e_steps > 0 and not args.partition_workers:
        import numpy as np
        idx = np.empty(w.k, np.uint32)
        val = np.empty(w.k, np.float32)
        opt.set("x", x)
        opt.step_host_sparse(hg, idx, val)
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            opt.step_host_sparse(hg, idx, val)
        torch.cuda.synchronize()
        dt = reduce_max(time.perf_counter() - t0, world, dev)
        e2e_sparse = {"value": units * args.e2e_steps / dt / 1e9, "unit": UNIT,
                      "h2d_bytes_per_step": gbytes * w.n * w.d, "d2h_bytes_per_step": 8 * w.k,
                      "ms_per_step": 1e3 * dt / args.e2e_steps, "steps": args.e2e_steps,
                      "api": "sk_step_host_sparse: parameters resident on the device, sparse update returned"}

    fam = (opt.get_option("log2g"), opt.get_option("window_lines"))
    hash_group, worker_chunk = 1 << fam[0], opt.get_option("worker_chunk")
    # the other configurations of d >= 25.6M the roofline target covers, in short runs with the default options
    others = None
    if world == 1 and not args.no_other_workloads and args.workload == DEFAULT_WORKLOAD and args.scale == 1:
        del opt, gsets, x
        torch.cuda.empty_cache()
        others = {name: quick_step_roofline(name, dev, peak) for name in ("C4", "C5")}

    if rank != 0:
        return
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        # the oracle as it stands, at the benchmark's own size: two steps on all host cores (the second is reported:
        # from it on I_{t-1} is not empty), and one step on a single thread
        threads = os.cpu_count() or 1
        ws, times, sample = cpu_oracle_rate(w, 1, 2, threads, args.variant, args.P, family=fam)
        _, times1, sample1 = cpu_oracle_rate(w, 1, 1, 1, args.variant, args.P, family=fam)
        cpu = {"value": ws.n * ws.d / times[-1] / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
               "seconds_per_step": times[-1], "cpu": cpu_model(),
               "single_thread": {"value": ws.n * ws.d / times1[-1] / 1e9, "unit": UNIT, "cores": 1,
                                 "seconds_per_step": times1[-1], "sample": sample1}}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "strong" if args.partition_workers else "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"sketches": "one, of the worker sum (linearity; not the headline path)" if args.sum_sketch
                       else "one per worker, then summed", "gradient_storage": "bf16" if args.grads_bf16 else "f32",
                       "workload": w.name, "d": w.d, "n": n_all, "r": w.r, "c": w.c, "k": w.k,
                       "recipe": w.recipe, "variant": args.variant, "P": args.P, "hash_group": hash_group,
                       "window_lines": fam[1], "worker_chunk": worker_chunk,
                       "replicas": 1 if args.partition_workers else world,
                       "workers_per_process": w.n, "partitioned": bool(args.partition_workers),
                       "stage_times": "a second pass of the same steps with CUDA events around every stage; "
                                      "ms_per_step is from the pass without them",
                       "l2": f"inputs larger than L2: {nsets} rotating gradient sets of {set_bytes / 1e9:.2f} GB",
                       "repetitions": len(rep_ms),
                       "timing": "ms_per_step is the median over the repetitions of (time of --steps steps) / steps",
                       "ms_per_step_min": min(rep_ms) / args.steps, "ms_per_step_max": max(rep_ms) / args.steps},
            "steps_per_s": 1e3 / ms_step,
            "step_roofline": {"algorithmic_bytes": b_alg, "achieved_gbs": b_alg / (ms_step * 1e-3) / 1e9,
                              "peak_gbs": peak, "peak_kind": f"of {peak_kind}",
                              "frac": b_alg / (ms_step * 1e-3) / 1e9 / peak},
            "roofline": roofline,
            "stage_ms_per_step": {nm: stage_ms[q] / max(1, nsteps) for q, nm in enumerate(binding.STAGE_NAMES)},
            "cpu_baseline": cpu, "e2e": e2e, "e2e_sparse_return": e2e_sparse, "gpu_launches": int(launches),
            "gpu_launches_per_step": launches / (world * args.steps * len(rep_ms)), "clocks": clocks,
            "other_workloads": others}
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
