#!/usr/bin/env python
"""Benchmark of the stencil sweep on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference]

One "step" is one ``stencil_apply`` of the workload (all of its time steps)
on a grid resident in HBM.  Rank 0 prints ONE JSON line.  With N > 1 (under
torchrun) every rank runs its own replica of the workload: the sweep has no
exchange step on one GPU, so there is no data-path collective; the timing is
the max over ranks and the value is the sum of all ranks' points.

``--impl reference`` times the CPU oracle (the plain definition, as it
stands) on a bounded slab of the same workload instead.
"""
from __future__ import annotations

import argparse
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

from paper_2608_21157_b200 import workloads as wl  # noqa: E402

METRIC = "stencil_gpoints_per_s"
UNIT = "GPoints/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes per launch of the dominant kernel (dram__bytes_read.sum +
# dram__bytes_write.sum from an ncu capture; see profiles/).  None = not captured.
NCU_TRAFFIC_BYTES = {
    "cfg2": 978.1e6,    # stream kernel, star R=1: 2 x (268.5 MB read + 220.5 MB written) on the half grid
    "cfg3": 1004.6e6,   # stream kernel, box R=1
    "cfg4": 995.7e6,    # stream kernel, star R=4
    "cfg5": 99.9e6,     # one fused pass (2 time steps of 256^3): 77.7 MB read + 22.2 MB written
    "cfg5L": 1035.1e6,  # one fused pass (2 time steps of 512^3): 545.4 MB read + 489.7 MB written
    "heat2d": 756.3e6,  # one fused pass (4 time steps of 10240^2): 2.5 x (180.6 + 121.9 MB) captured on 4096 x 10240
}


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi for SM clock and throttle reasons while running."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str, period_ms: int = 50):
        self.gpu_id, self.period_ms = gpu_id, period_ms
        self.rows, self.proc, self.thread = [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", str(self.period_ms)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        def pump():
            for line in self.proc.stdout:
                self.rows.append((time.time(), line.strip()))
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()          # the exact process started above
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=2)

    def summary(self, t0: float, t1: float):
        sm, mx, power, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for t, line in self.rows:
            if t < t0 or t > t1 + 0.05:
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, flag in zip(names, parts[3:7]):
                if flag.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


# ---------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------
def time_workload(torch, b, wk, steps, warmup, knobs, variant=None, per_launch_events=True):
    """Times `steps` applies of workload `wk` with inputs resident in HBM.
    Returns dict with batch ms/step, per-apply event ms, launches, plan info."""
    dev = torch.device("cuda", torch.cuda.current_device())
    a = wk.input()
    src = torch.from_numpy(a).to(dev)
    dst = torch.empty_like(src)
    stream = torch.cuda.current_stream()
    plan = b.Plan.for_workload(wk, variant=variant, **knobs)
    for _ in range(max(warmup, 0)):
        plan.apply(src, dst, wk.steps, stream.cuda_stream)
    torch.cuda.synchronize()
    l0 = plan.launches
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    evs[0].record(stream)
    for i in range(steps):
        plan.apply(src, dst, wk.steps, stream.cuda_stream)
        evs[i + 1].record(stream)
    torch.cuda.synchronize()
    total_ms = evs[0].elapsed_time(evs[-1])
    per = [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]
    launches = plan.launches - l0
    status = plan.query_status()
    info = {"variant": plan.variant, "tile_y": plan.get(b.KEY_TILE_Y),
            "rows_per_thread": plan.get(b.KEY_ROWS_PER_THREAD),
            "fuse_steps": plan.get(b.KEY_FUSE_STEPS) if wk.steps > 1 else 1}
    graph_ms = None
    if wk.point_updates < (1 << 22):
        # a launch-latency-bound workload: the host loop above cannot issue launches as fast
        # as the GPU retires them, so also time a CUDA graph that replays `steps` applies
        try:
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for _ in range(steps):
                    plan.apply(src, dst, wk.steps, torch.cuda.current_stream().cuda_stream)
            graph.replay()
            torch.cuda.synchronize()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record()
            graph.replay()
            g1.record()
            torch.cuda.synchronize()
            graph_ms = g0.elapsed_time(g1) / steps
            del graph
        except Exception:
            graph_ms = None
    return {"total_ms": total_ms, "per_apply_ms": per, "launches": launches, "status": status,
            "plan": plan, "src": src, "dst": dst, "info": info, "input": a, "graph_ms_per_apply": graph_ms}


def config_summary(wk, total_ms, steps, peak):
    pts = wk.point_updates * steps
    sec = total_ms / 1e3
    gp = pts / sec / 1e9
    gbs = 2.0 * wk.itemsize * pts / sec / 1e9      # one read + one write of the grid's element type
    return {"gpoints_per_s": round(gp, 2), "effective_gbs": round(gbs, 1),
            "frac_of_measured_hbm": round(gbs / peak, 4), "frac_of_nominal_8tbs": round(gbs / NOMINAL_HBM_GBS, 4),
            "ms_per_apply": round(total_ms / steps, 5), "time_steps_per_apply": wk.steps,
            "ms_per_time_step": round(total_ms / steps / max(wk.steps, 1), 5),
            "taps": wk.taps(), "dtype": "f64" if wk.itemsize == 8 else "f32"}


def max_over_ranks(value, dist, device):
    """Largest `value` over all ranks (timings of a multi-rank run are the slowest rank's)."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gpoints(world, point_updates_per_apply, applies, total_ms):
    """Replicas only: every rank sweeps its own full grid, so the job's point count is
    world x one rank's, over the slowest rank's time."""
    return world * point_updates_per_apply * applies / (total_ms / 1e3) / 1e9


def pick_workload(args):
    wk = wl.get(args.workload)
    if args.dims:
        wk = wk.scaled(tuple(int(v) for v in args.dims.split(",")), name=wk.name)
    return wk


def run_gpu(args):
    import torch
    from paper_2608_21157_b200 import binding as b
    from paper_2608_21157_b200 import build as build_mod

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback; use --impl reference for the oracle)")
    torch.cuda.set_device(local % torch.cuda.device_count())
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", torch.cuda.current_device()))
    if rank == 0:
        build_mod.build()
    if dist is not None:
        dist.barrier()
    b.load()

    peak, peak_kind = measured_hbm_peak()
    wk = pick_workload(args)
    knobs = dict(tile_y=args.tile_y, chunk_z=args.chunk_z, stages=args.stages,
                 rows_per_thread=args.rows_per_thread, streaming_store=args.streaming_store,
                 fuse_steps=args.fuse_steps)
    variant = {"auto": None, "generic": b.VARIANT_GENERIC, "stream": b.VARIANT_STREAM,
               "fused": b.VARIANT_FUSED}[args.variant]

    props = torch.cuda.get_device_properties(torch.cuda.current_device())
    gpu_id = f"GPU-{props.uuid}" if hasattr(props, "uuid") else str(torch.cuda.current_device())
    sampler = ClockSampler(gpu_id)
    sampler.start()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: K applies, events on the launching stream -------------
    dev = torch.device("cuda", torch.cuda.current_device())
    a_host = wk.input()
    src = torch.from_numpy(a_host).to(dev)
    dst = torch.empty_like(src)
    stream = torch.cuda.current_stream()
    plan = b.Plan.for_workload(wk, variant=variant, **knobs)
    for _ in range(args.warmup):
        plan.apply(src, dst, wk.steps, stream.cuda_stream)
    barrier()
    l0 = plan.launches
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    t_wall0 = time.time()
    evs[0].record(stream)
    for i in range(args.steps):
        plan.apply(src, dst, wk.steps, stream.cuda_stream)
        evs[i + 1].record(stream)
    barrier()
    t_wall1 = time.time()
    total_ms = evs[0].elapsed_time(evs[-1])
    per_apply = [evs[i].elapsed_time(evs[i + 1]) for i in range(args.steps)]
    launches = plan.launches - l0
    if plan.query_status() != b.OK:
        raise SystemExit("device status word reports a timeout; results are invalid")

    # keep the same kernel running long enough for nvidia-smi to see clocks under load
    t_load0 = time.time()
    while time.time() - t_load0 < args.clock_seconds:
        for _ in range(20):
            plan.apply(src, dst, wk.steps, stream.cuda_stream)
        torch.cuda.synchronize()
    t_load1 = time.time()

    total_ms_max = max_over_ranks(total_ms, dist, dev)

    # ---- end to end: host buffers through the C ABI, copies inside the timing --
    e2e = None
    if not args.no_e2e:
        hsrc = torch.from_numpy(a_host).pin_memory()
        hdst = torch.empty_like(hsrc).pin_memory()
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        for _ in range(2):
            plan.apply_host(hsrc, hdst, wk.steps, stream.cuda_stream)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            plan.apply_host(hsrc, hdst, wk.steps, stream.cuda_stream)
        e1.record(stream)
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1), dist, dev)
        e2e = {"value": round(whole_job_gpoints(world, wk.point_updates, e2e_steps, e2e_ms), 4),
               "unit": UNIT, "h2d_bytes_per_step": int(a_host.nbytes), "d2h_bytes_per_step": int(a_host.nbytes),
               "steps": e2e_steps, "ms_per_step": round(e2e_ms / e2e_steps, 4),
               "api": "stencil_apply_host (pinned host buffers)"}
        del hsrc, hdst

    # ---- roofline of the dominant kernel --------------------------------------
    launches_per_apply = max(launches // max(args.steps, 1), 1)
    kernel_ms = statistics.mean(per_apply) / launches_per_apply
    # algorithmic bytes: 8 B (one fp32 read + one write) per point per time step; a launch
    # advances N points by (time steps per apply / launches per apply) steps
    steps_per_launch = max(wk.steps, 1) / launches_per_apply
    algo_bytes = 2.0 * wk.itemsize * wk.npoints * steps_per_launch
    achieved = algo_bytes / (kernel_ms / 1e3) / 1e9
    fuse = plan.get(b.KEY_FUSE_STEPS) if wk.steps > 1 else 1
    f64 = wk.itemsize == 8
    if plan.variant == "generic":
        kernel_name = "stencil_generic_kernel"
    elif fuse > 1:
        kernel_name = "stencil_rows2d_fused_kernel" if len(wk.dims) == 2 else "stencil_fused_kernel"
    elif len(wk.dims) == 2:
        kernel_name = "stencil_rows2d_f64_kernel" if f64 else "stencil_rows2d_kernel"
    else:
        kernel_name = "stencil_stream_f64_kernel" if f64 else "stencil_stream_kernel"
    roofline = {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                "frac": round(achieved / peak, 4), "traffic": NCU_TRAFFIC_BYTES.get(wk.name),
                "peak_kind": f"of {peak_kind} (copy bandwidth)", "kernel": kernel_name,
                "kernel_ms": round(kernel_ms, 5), "algorithmic_bytes_per_launch": int(algo_bytes),
                "time_steps_per_launch": steps_per_launch,
                "frac_of_nominal_8tbs": round(achieved / NOMINAL_HBM_GBS, 4)}
    # The sweeps with many taps are bound by plain FMA arithmetic, not by memory: report
    # against whichever limit the kernel is closer to.  ALU peak = 148 SMs x 128 fp32 (64 FP64)
    # FMA lanes x 2 flop x the maximum SM clock (1965 MHz).
    taps = int(np.count_nonzero(wk.weights()))
    alu_peak = 148 * (64 if f64 else 128) * 2 * 1.965e9 / 1e12
    alu_achieved = 2.0 * taps * wk.npoints * steps_per_launch / (kernel_ms / 1e3) / 1e12
    if alu_achieved / alu_peak > achieved / peak:
        roofline.update({"bound": "alu", "achieved": round(alu_achieved, 2), "peak": round(alu_peak, 1),
                         "unit": "TFLOP/s", "frac": round(alu_achieved / alu_peak, 4),
                         "peak_kind": "148 SMs x %d FMA lanes x 2 flop x 1965 MHz (no measured peak for plain "
                                      "FMA; the part runs 1.5-1.8 GHz under its power cap)" % (64 if f64 else 128),
                         "hbm_frac_of_measured": round(achieved / peak, 4), "taps": taps})
    info = {"variant": plan.variant, "tile_y": plan.get(b.KEY_TILE_Y),
            "rows_per_thread": plan.get(b.KEY_ROWS_PER_THREAD), "fuse_steps": fuse}
    plan.destroy()
    del src, dst

    # ---- the other configs, short runs, rank 0 only ----------------------------
    all_cfg = {}
    if rank == 0 and not args.no_all_configs:
        for name in args.also.split(","):
            if not name or name == wk.name:
                continue
            w2 = wl.get(name)
            n2 = args.also_steps
            r = time_workload(torch, b, w2, n2, 3, {}, None)
            s = config_summary(w2, r["total_ms"], n2, peak)
            s.update(r["info"])
            if r.get("graph_ms_per_apply"):
                s["ms_per_apply_cuda_graph"] = round(r["graph_ms_per_apply"], 5)
                s["gpoints_per_s_cuda_graph"] = round(w2.point_updates / r["graph_ms_per_apply"] / 1e6, 2)
                s["note"] = "launch-latency-bound: the graph replay figure is the device-side rate"
            s["launches_per_apply"] = r["launches"] // n2
            all_cfg[name] = s
            r["plan"].destroy()
            del r
            torch.cuda.empty_cache()
    all_cfg[wk.name] = dict(config_summary(wk, total_ms_max, args.steps, peak), **info)

    # ---- cuDNN reference point (fp32 conv via PyTorch), rank 0 only ------------
    cudnn = None
    if rank == 0 and args.cudnn:
        cudnn = cudnn_reference(torch, wk, a_host)

    sampler.stop()
    clocks = sampler.summary(t_wall0, t_load1)
    clocks["sampled_over"] = "timed region plus %.1f s of the same kernel" % (t_load1 - t_load0)

    # ---- CPU baseline: the oracle, on this machine's cores, rank 0 at N=1 only ------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(wk, a_host, budget_s=args.cpu_seconds)

    if rank == 0:
        pts = world * wk.point_updates * args.steps
        value = whole_job_gpoints(world, wk.point_updates, args.steps, total_ms_max)
        line = {
            "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(total_ms_max / args.steps, 5),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64" if wk.itemsize == 8 else "f32",
            "data": "synthetic (seeded numpy default_rng fields; see config.workload)",
            "config": {"workload": f"{wk.name}: {wk.description}", "dims": list(wk.dims), "radius": wk.radius,
                       "taps": wk.taps(), "time_steps_per_apply": wk.steps,
                       "l2": "grid in + out = %.0f MiB, larger than the 126 MB L2; no flush" % (2 * a_host.nbytes / 2**20)
                             if 2 * a_host.nbytes > 126e6 else "working set fits L2; warm-L2 figure",
                       "parallelism": "replicas only (one full grid per GPU, no exchange)" if world > 1 else "1 GPU",
                       **info},
            "effective_gbs": round(2.0 * wk.itemsize * pts / (total_ms_max / 1e3) / 1e9 / world, 1),
            "gpu_launches": int(launches),
            "clocks": clocks,
            "e2e": e2e,
            "roofline": roofline,
            "cpu_baseline": cpu,
            "all_configs": all_cfg,
            "cudnn_reference": cudnn,
            "paper_context": "paper: 1.53x over cuDNN on A100-PCIE-40GB, FP64, 2D box R=3 10240^2 (4.71 ms/step); other hardware and precision",
        }
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def cudnn_reference(torch, wk, a_host, iters=5):
    """fp32 conv2d/conv3d (TF32 off) on the same GPU: a reference point only."""
    try:
        import torch.nn.functional as F
        if wk.boundary != wl.ZERO:
            return {"unavailable": "periodic boundary has no conv padding mode here"}
        torch.backends.cudnn.allow_tf32 = False
        torch.backends.cuda.matmul.allow_tf32 = False
        torch.backends.cudnn.benchmark = True
        x = torch.from_numpy(a_host).cuda()[None, None]
        w = torch.from_numpy(wk.weights()).cuda()[None, None]
        conv = F.conv2d if wk.ndim == 2 else F.conv3d
        def run():
            y = x
            for _ in range(max(wk.steps, 1)):
                y = conv(y, w, padding=wk.radius)
            return y
        for _ in range(2):
            run()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            run()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / iters
        return {"ms_per_apply": round(ms, 4), "gpoints_per_s": round(wk.point_updates / (ms / 1e3) / 1e9, 2),
                "what": "torch.nn.functional.conv%dd fp32, TF32 off, dense (2R+1)^d kernel" % wk.ndim}
    except Exception as e:  # a reference point must never sink the benchmark
        return {"unavailable": f"{type(e).__name__}: {str(e)[:120]}"}


# ---------------------------------------------------------------------------
# CPU oracle arms
# ---------------------------------------------------------------------------
def _slab(wk, a_host, planes):
    """First `planes` entries along the slowest axis: same operator, same data."""
    planes = max(1, min(int(planes), wk.dims[0]))
    return np.ascontiguousarray(a_host[:planes]), planes


def cpu_baseline(wk, a_host, budget_s=12.0):
    """The oracle as it stands on this machine's host cores, for about `budget_s` seconds:
    a slab of the workload sized from a probe, swept repeatedly."""
    import oracle
    w = wk.weights()
    cores = oracle.num_threads()
    probe, pp = _slab(wk, a_host, max(4 * wk.radius + 2, wk.dims[0] // 16))
    t0 = time.perf_counter()
    oracle.apply(probe, w, wk.boundary, 1)
    t_probe = time.perf_counter() - t0
    rate = probe.size / max(t_probe, 1e-9)                 # point-updates per second
    steps = max(1, min(wk.steps, 4))
    plane_pts = a_host.size / wk.dims[0]
    planes = int(min(wk.dims[0], max(pp, rate * budget_s / steps / plane_pts)))
    sample, planes = _slab(wk, a_host, planes)
    reps, done, t0 = 0, 0.0, time.perf_counter()
    while True:
        oracle.apply(sample, w, wk.boundary, steps)
        reps += 1
        done = time.perf_counter() - t0
        if done >= budget_s or reps >= 200:
            break
    return {"value": round(sample.size * steps * reps / done / 1e9, 4), "unit": UNIT, "cores": cores,
            "kind": "oracle",
            "sample": f"first {planes} of {wk.dims[0]} slices along the slowest axis, {steps} time step(s), "
                      f"repeated {reps} times, {done:.1f} s wall", "seconds": round(done, 2)}


def run_reference(args):
    """The oracle as the reference arm: K steps, each one sweep of a bounded slab."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    wk = pick_workload(args)
    a_host = wk.input()
    w = wk.weights()
    cores = oracle.num_threads()
    probe, pp = _slab(wk, a_host, max(4 * wk.radius + 2, wk.dims[0] // 32))
    t0 = time.perf_counter()
    oracle.apply(probe, w, wk.boundary, 1)
    rate = probe.size / max(time.perf_counter() - t0, 1e-9)
    per_step_budget = args.reference_seconds / max(args.steps + args.warmup, 1)
    tsteps = max(1, min(wk.steps, 2))
    plane_pts = a_host.size / wk.dims[0]
    planes = int(min(wk.dims[0], max(2 * wk.radius + 2, rate * per_step_budget / tsteps / plane_pts)))
    sample, planes = _slab(wk, a_host, planes)
    for _ in range(args.warmup):
        oracle.apply(sample, w, wk.boundary, tsteps)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.apply(sample, w, wk.boundary, tsteps)
    dt = time.perf_counter() - t0
    value = sample.size * tsteps * args.steps / dt / 1e9
    sample_desc = (f"each step = {tsteps} sweep(s) of the first {planes} of {wk.dims[0]} slices along the "
                   f"slowest axis of the workload")
    line = {
        "impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(dt / args.steps * 1e3, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64 accumulate, f32 store", "data": "synthetic (same seeded fields)",
        "config": {"workload": f"{wk.name}: {wk.description}", "dims": list(wk.dims), "radius": wk.radius,
                   "taps": wk.taps(), "sample": sample_desc},
        "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample_desc},
        "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--dims", default=None, help="override the grid, e.g. 256,512,512 (profiling on smaller cases)")
    ap.add_argument("--variant", default="auto", choices=["auto", "generic", "stream", "fused"])
    ap.add_argument("--tile-y", dest="tile_y", type=int, default=None)
    ap.add_argument("--rows-per-thread", dest="rows_per_thread", type=int, default=None)
    ap.add_argument("--chunk-z", dest="chunk_z", type=int, default=None)
    ap.add_argument("--stages", type=int, default=None)
    ap.add_argument("--fuse-steps", dest="fuse_steps", type=int, default=None)
    ap.add_argument("--streaming-store", dest="streaming_store", type=int, default=None)
    ap.add_argument("--also", default="cfg1,cfg3,cfg4,cfg5,cfg5L,cfg5L_periodic,paper2d,paper2d_f64,heat2d", help="other workloads summarised in all_configs")
    ap.add_argument("--also-steps", dest="also_steps", type=int, default=20)
    ap.add_argument("--no-all-configs", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-steps", dest="e2e_steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", dest="cpu_seconds", type=float, default=12.0)
    ap.add_argument("--reference-seconds", dest="reference_seconds", type=float, default=90.0)
    ap.add_argument("--clock-seconds", dest="clock_seconds", type=float, default=1.5)
    ap.add_argument("--cudnn", type=int, default=1)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
