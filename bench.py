#!/usr/bin/env python
"""Benchmark of the stencil sweep on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference] [--sharded]

One "step" is one ``stencil_apply`` of the workload (all of its time steps)
on a grid resident in HBM.  Rank 0 prints ONE JSON line.

With N > 1 (under torchrun) the default is replicas: every rank runs its own
copy of the workload, there is no data-path collective, the time is the
slowest rank's and the value the sum of all ranks' points ("weak").  With
``--sharded`` the ranks instead share ONE grid, cut into slabs along the
slowest axis (``paper_2608_21157_b200.sharded``): the boundary planes travel
between neighbours by NCCL point-to-point sends, the value is the whole
grid's point-updates over the slowest rank's time ("strong").

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
SM_COUNT, SM_MAX_MHZ = 148, 1965.0

# DRAM bytes per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum of
# one launch at the workload's full size, from the ncu captures summarised under profiles/).
# None = not captured.
NCU_TRAFFIC_BYTES = {
    "cfg2": 1026.4e6,       # stream kernel, star R=1, 512^3: 536.9 MB read + 489.5 MB written
    "cfg3": 1055.0e6,       # stream kernel, box R=1, 512^3: 564.3 + 490.7
    "cfg4": 1049.1e6,       # stream kernel, star R=4, 512^3: 557.4 + 491.7
    "cfg5": 99.2e6,         # one fused pass (2 time steps of 256^3): 77.4 + 21.8 (both grids largely stay in L2)
    "cfg5L": 1044.7e6,      # one fused pass (2 time steps of 512^3): 554.7 + 490.0
    "cfg5L_f64": 2121.4e6,  # one fused pass (2 time steps of 512^3 in FP64): 1093.7 + 1027.7
    "heat2d": 805.9e6,      # one fused pass (4 time steps of 10240^2): 432.9 + 373.0
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

    def __init__(self, gpu_id: str, period_ms: int = 100):
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
# helpers of the GPU arm
# ---------------------------------------------------------------------------
def is_tiny(wk) -> bool:
    """Launch-latency-bound: the host cannot issue applies as fast as the GPU retires them, so an
    event after every apply would be what the loop measures."""
    return wk.point_updates < (1 << 22)


def host_warmup(torch, plan, src, dst, wk, stream, seconds=0.2):
    """A launch-latency-bound workload measures the host's launch path, which takes some ten
    thousand calls to reach its steady rate (7 us per apply at first, 4.1 us after): issue applies
    for `seconds` before such a workload is timed."""
    sp, dp, handle, t0 = src.data_ptr(), dst.data_ptr(), stream.cuda_stream, time.time()
    while time.time() - t0 < seconds:
        for _ in range(1000):
            plan.apply(sp, dp, wk.steps, handle)
    torch.cuda.synchronize()


def time_applies(torch, plan, src, dst, wk, steps, stream, per_apply=True):
    """`steps` applies, CUDA events on the launching stream.  Returns (total ms, per-apply ms or None)."""
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1 if per_apply else 2)]
    sp, dp, handle, tsteps = src.data_ptr(), dst.data_ptr(), stream.cuda_stream, wk.steps
    evs[0].record(stream)
    for i in range(steps):
        plan.apply(sp, dp, tsteps, handle)
        if per_apply:
            evs[i + 1].record(stream)
    if not per_apply:
        evs[1].record(stream)
    torch.cuda.synchronize()
    total_ms = evs[0].elapsed_time(evs[-1])
    per = [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)] if per_apply else None
    return total_ms, per


def graph_replay_ms(torch, plan, src, dst, wk, steps, stream):
    """ms per apply of a CUDA graph that replays `steps` applies (the device-side rate of a
    launch-latency-bound workload); None if capture fails."""
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
        ms = g0.elapsed_time(g1) / steps
        del graph
        return ms
    except Exception:
        return None


def plan_info(b, plan, wk):
    return {"variant": plan.variant, "tile_y": plan.get(b.KEY_TILE_Y),
            "rows_per_thread": plan.get(b.KEY_ROWS_PER_THREAD),
            "fuse_steps": plan.get(b.KEY_FUSE_STEPS) if wk.steps > 1 else 1}


def kernel_name(wk, info):
    f64, fuse = wk.itemsize == 8, info["fuse_steps"]
    if info["variant"] == "generic":
        return "stencil_generic_kernel"
    if fuse > 1:
        if len(wk.dims) == 2:
            return "stencil_rows2d_fused_f64_kernel" if f64 else "stencil_rows2d_fused_kernel"
        return "stencil_fused_kernel"
    if len(wk.dims) == 2:
        return "stencil_rows2d_f64_kernel" if f64 else "stencil_rows2d_kernel"
    if wk.boundary == wl.PERIODIC:
        return "stencil_stream_f64_wrap_kernel" if f64 else "stencil_stream_wrap_kernel"
    return "stencil_stream_f64_kernel" if f64 else "stencil_stream_kernel"


def roofline_block(wk, info, ms_per_apply, launches_per_apply, peak, peak_kind, sm_mhz=None):
    """Roofline of the dominant kernel: algorithmic bytes (one read + one write of the grid's
    element type per point per time step) per launch over the launch's average duration, against
    the measured copy bandwidth; sweeps with many taps are bound by plain FMA arithmetic instead
    and report against 148 SMs x 128 fp32 (64 FP64) FMA lanes x 2 flop x the maximum SM clock."""
    launches_per_apply = max(int(launches_per_apply), 1)
    kernel_ms = ms_per_apply / launches_per_apply
    steps_per_launch = max(wk.steps, 1) / launches_per_apply
    algo_bytes = 2.0 * wk.itemsize * wk.npoints * steps_per_launch
    achieved = algo_bytes / (kernel_ms / 1e3) / 1e9
    f64 = wk.itemsize == 8
    if is_tiny(wk):
        return {"bound": "launch latency", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                "frac": round(achieved / peak, 4), "traffic": None, "kernel": kernel_name(wk, info),
                "kernel_ms": round(kernel_ms, 5),
                "note": "the grid fits L2 and one launch is shorter than its own latency: the fraction is not meaningful"}
    r = {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
         "frac": round(achieved / peak, 4), "traffic": NCU_TRAFFIC_BYTES.get(wk.name),
         "peak_kind": f"of {peak_kind} (copy bandwidth)", "kernel": kernel_name(wk, info),
         "kernel_ms": round(kernel_ms, 5), "algorithmic_bytes_per_launch": int(algo_bytes),
         "time_steps_per_launch": steps_per_launch,
         "frac_of_nominal_8tbs": round(achieved / NOMINAL_HBM_GBS, 4)}
    lanes = 64 if f64 else 128
    taps = int(np.count_nonzero(wk.weights()))
    alu_peak = SM_COUNT * lanes * 2 * SM_MAX_MHZ * 1e6 / 1e12
    alu_achieved = 2.0 * taps * wk.npoints * steps_per_launch / (kernel_ms / 1e3) / 1e12
    if alu_achieved / alu_peak > achieved / peak:
        r.update({"bound": "alu", "achieved": round(alu_achieved, 2), "peak": round(alu_peak, 1),
                  "unit": "TFLOP/s", "frac": round(alu_achieved / alu_peak, 4),
                  "peak_kind": "148 SMs x %d FMA lanes x 2 flop x 1965 MHz (no measured peak for plain "
                               "FMA; the part runs 1.5-1.8 GHz under its power cap)" % lanes,
                  "hbm_frac_of_measured": round(achieved / peak, 4), "taps": taps})
        if sm_mhz:
            # the same fraction at the clock the part actually held while the kernel ran
            r["frac_at_sampled_clock"] = round(alu_achieved / (alu_peak * sm_mhz / SM_MAX_MHZ), 4)
            r["sampled_sm_mhz"] = sm_mhz
    return r


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


def sharded_job_summary(dims, radius, time_steps, halo_steps, applies, total_ms, world, itemsize):
    """Sharded run: the ranks share ONE grid, so the job's point count is the grid's, whatever the
    number of ranks, over the slowest rank's time.  Also the bytes a rank sends per time step: to
    each neighbour `halo_steps * radius` planes once every `halo_steps` steps."""
    npoints = 1
    for d in dims:
        npoints *= int(d)
    plane_bytes = itemsize * npoints // int(dims[0])
    neighbours = 0 if world == 1 else 2          # an inner rank's; the two end ranks of a chain have one
    rounds = -(-int(time_steps) // int(halo_steps))
    return {"value": npoints * int(time_steps) * applies / (total_ms / 1e3) / 1e9,
            "exchange_bytes_per_rank_per_apply": neighbours * halo_steps * radius * plane_bytes * rounds,
            "exchange_bytes_per_rank_per_time_step":
                neighbours * halo_steps * radius * plane_bytes * rounds / max(int(time_steps), 1),
            "messages_per_rank_per_apply": neighbours * rounds}


def pick_workload(args):
    wk = wl.get(args.workload)
    if args.dims:
        wk = wk.scaled(tuple(int(v) for v in args.dims.split(",")), name=wk.name)
    return wk


def init_ranks(torch, sharded=False):
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
    return rank, world, dist


# ---------------------------------------------------------------------------
# GPU arm: one grid per rank
# ---------------------------------------------------------------------------
def run_gpu(args):
    import torch
    from paper_2608_21157_b200 import binding as b
    from paper_2608_21157_b200 import build as build_mod

    rank, world, dist = init_ranks(torch)
    if rank == 0:
        build_mod.build()
    if dist is not None:
        dist.barrier()
    b.load()

    peak, peak_kind = measured_hbm_peak()
    wk = pick_workload(args)
    knobs = dict(tile_y=args.tile_y, chunk_z=args.chunk_z, stages=args.stages,
                 rows_per_thread=args.rows_per_thread, streaming_store=args.streaming_store,
                 fuse_steps=args.fuse_steps, tile_x=args.tile_x)
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
    if is_tiny(wk):
        host_warmup(torch, plan, src, dst, wk, stream)
    barrier()
    l0 = plan.launches
    t_wall0 = time.time()
    total_ms, per_apply = time_applies(torch, plan, src, dst, wk, args.steps, stream, per_apply=not is_tiny(wk))
    barrier()
    t_wall1 = time.time()
    launches = plan.launches - l0
    if plan.query_status() != b.OK:
        raise SystemExit("device status word reports a timeout; results are invalid")
    total_ms_max = max_over_ranks(total_ms, dist, dev)

    # ---- sustained: the same applies back to back for >= clock_seconds, timed as one region; the
    # clock samples of exactly this window go with it -----------------------------------------
    sustained = None
    t_load0 = t_load1 = time.time()
    if args.clock_seconds > 0:
        per = max(total_ms / max(args.steps, 1), 1e-3)
        batch = max(1, min(2000, int(100.0 / per)))            # ~0.1 s of applies between host syncs
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_sus = 0
        torch.cuda.synchronize()
        t_load0 = time.time()
        s0.record(stream)
        while time.time() - t_load0 < args.clock_seconds:
            for _ in range(batch):
                plan.apply(src, dst, wk.steps, stream.cuda_stream)
            n_sus += batch
            torch.cuda.synchronize()
        s1.record(stream)
        torch.cuda.synchronize()
        t_load1 = time.time()
        sus_ms = s0.elapsed_time(s1)
        sus_clocks = sampler.summary(t_load0, t_load1)
        sustained = {"value": round(wk.point_updates * n_sus / (sus_ms / 1e3) / 1e9, 3), "unit": UNIT,
                     "applies": n_sus, "seconds": round(sus_ms / 1e3, 3),
                     "sm_mhz": sus_clocks.get("sm_mhz"), "reasons": sus_clocks.get("reasons"),
                     "power_w_max": sus_clocks.get("power_w_max"),
                     "what": "the same applies back to back, CUDA events around the whole window "
                             "(host syncs every ~0.1 s included); this rank"}

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

    clocks = sampler.summary(t_wall0, t_load1)
    clocks["sampled_over"] = "timed region plus the %.1f s sustained window of the same applies" % (t_load1 - t_load0)

    # ---- roofline of the dominant kernel --------------------------------------
    info = plan_info(b, plan, wk)
    launches_per_apply = max(launches // max(args.steps, 1), 1)
    mean_apply_ms = statistics.mean(per_apply) if per_apply else total_ms / args.steps
    roofline = roofline_block(wk, info, mean_apply_ms, launches_per_apply, peak, peak_kind, clocks.get("sm_mhz"))
    plan.destroy()
    del src, dst
    torch.cuda.empty_cache()

    # ---- the other configs, short runs, rank 0 only ----------------------------
    all_cfg = {}
    headline = dict(config_summary(wk, total_ms_max, args.steps, peak), **info)
    headline["launches_per_apply"] = launches_per_apply
    headline["roofline"] = roofline
    headline["input_sha256"] = wl.sha256(a_host)
    if rank == 0 and args.cudnn:
        headline["cudnn_reference"] = cudnn_reference(torch, wk, a_host)
    if rank == 0 and not args.no_all_configs:
        for name in args.also.split(","):
            if not name or name == wk.name:
                continue
            all_cfg[name] = one_config(torch, b, wl.get(name), args, peak, peak_kind, sampler)
    all_cfg[wk.name] = headline

    sampler.stop()

    # ---- CPU baseline: the oracle, on this machine's cores, rank 0 at N=1 only ------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(wk, a_host, budget_s=args.cpu_seconds)
        all_cfg[wk.name]["cpu_baseline"] = cpu

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
                       "input_sha256": headline["input_sha256"], "numpy": np.__version__,
                       **info},
            "effective_gbs": round(2.0 * wk.itemsize * pts / (total_ms_max / 1e3) / 1e9 / world, 1),
            "gpu_launches": int(launches),
            "sustained": sustained,
            "clocks": clocks,
            "e2e": e2e,
            "roofline": roofline,
            "cpu_baseline": cpu,
            "all_configs": all_cfg,
            "cudnn_reference": headline.get("cudnn_reference"),
            "paper_context": "paper: 1.53x over cuDNN on A100-PCIE-40GB, FP64, 2D box R=3 10240^2 (4.71 ms/step); other hardware and precision",
        }
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def one_config(torch, b, wk, args, peak, peak_kind, sampler):
    """A short run of one more workload with its own roofline block, cuDNN reference point, a
    bounded oracle baseline and the hash of its input."""
    n = args.also_steps
    dev = torch.device("cuda", torch.cuda.current_device())
    a = wk.input()
    src = torch.from_numpy(a).to(dev)
    dst = torch.empty_like(src)
    stream = torch.cuda.current_stream()
    plan = b.Plan.for_workload(wk)
    for _ in range(3):
        plan.apply(src, dst, wk.steps, stream.cuda_stream)
    if is_tiny(wk):
        host_warmup(torch, plan, src, dst, wk, stream)
        n = max(n, 2000)                                 # ... and time enough calls to average over
    torch.cuda.synchronize()
    l0 = plan.launches
    t0 = time.time()
    total_ms, _ = time_applies(torch, plan, src, dst, wk, n, stream, per_apply=False)
    t1 = time.time()
    launches = plan.launches - l0
    info = plan_info(b, plan, wk)
    s = config_summary(wk, total_ms, n, peak)
    s.update(info)
    s["launches_per_apply"] = launches // n
    s["status"] = plan.query_status()
    clk = None
    if not is_tiny(wk) and args.also_clock_seconds > 0:
        # the same applies for a little longer, so that the clock sampler sees the part under this load
        per = max(total_ms / n, 1e-3)
        batch = max(1, min(500, int(50.0 / per)))
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        m = 0
        torch.cuda.synchronize()
        c0 = time.time()
        s0.record(stream)
        while time.time() - c0 < args.also_clock_seconds:
            for _ in range(batch):
                plan.apply(src, dst, wk.steps, stream.cuda_stream)
            m += batch
            torch.cuda.synchronize()
        s1.record(stream)
        torch.cuda.synchronize()
        c1 = time.time()
        window = sampler.summary(c0, c1)
        clk = window.get("sm_mhz")
        s["sustained"] = {"gpoints_per_s": round(wk.point_updates * m / (s0.elapsed_time(s1) / 1e3) / 1e9, 2),
                          "seconds": round(s0.elapsed_time(s1) / 1e3, 3), "sm_mhz": clk,
                          "reasons": window.get("reasons")}
    s["roofline"] = roofline_block(wk, info, total_ms / n, s["launches_per_apply"], peak, peak_kind, clk)
    if is_tiny(wk):
        g = graph_replay_ms(torch, plan, src, dst, wk, min(n, 200), stream)
        if g:
            s["ms_per_apply_cuda_graph"] = round(g, 5)
            s["gpoints_per_s_cuda_graph"] = round(wk.point_updates / g / 1e6, 2)
            s["note"] = ("launch-latency-bound: gpoints_per_s is the host-driven rate (one C-ABI call per "
                         "apply), the graph replay figure the device-side rate")
    plan.destroy()
    del src, dst
    torch.cuda.empty_cache()
    s["input_sha256"] = wl.sha256(a)
    if args.cudnn:
        s["cudnn_reference"] = cudnn_reference(torch, wk, a)
        torch.cuda.empty_cache()
    if not args.no_cpu_baseline and args.also_cpu_seconds > 0:
        s["cpu_baseline"] = cpu_baseline(wk, a, budget_s=args.also_cpu_seconds)
    return s


def cudnn_reference(torch, wk, a_host, iters=5):
    """conv2d/conv3d of PyTorch (cuDNN; TF32 off) with the dense (2R+1)^d kernel on the same GPU, in
    the workload's own dtype, iterated workloads as chained calls: a reference point only."""
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
                "what": "torch.nn.functional.conv%dd %s, TF32 off, dense (2R+1)^d kernel of %d entries, %d chained call(s)"
                        % (wk.ndim, "fp64" if wk.itemsize == 8 else "fp32", (2 * wk.radius + 1) ** wk.ndim,
                           max(wk.steps, 1))}
    except Exception as e:  # a reference point must never sink the benchmark
        return {"unavailable": f"{type(e).__name__}: {str(e)[:120]}"}


# ---------------------------------------------------------------------------
# GPU arm: one grid shared by all ranks (slab decomposition, halo exchange over NCCL)
# ---------------------------------------------------------------------------
def run_sharded(args):
    import torch
    from paper_2608_21157_b200 import binding as b
    from paper_2608_21157_b200 import build as build_mod
    from paper_2608_21157_b200.sharded import ShardedSweep

    # the communicator log stays on (it shows the transport each pair of ranks uses), on stderr so that stdout
    # keeps the one JSON line
    os.environ.setdefault("NCCL_DEBUG", "INFO")
    os.environ.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
    rank, world, dist = init_ranks(torch, sharded=True)
    if rank == 0:
        build_mod.build()
    if dist is not None:
        dist.barrier()
    b.load()
    wk = pick_workload(args)
    if wk.itemsize == 8 and wk.dims[-1] % 2 or wk.itemsize == 4 and wk.dims[-1] % 4:
        raise SystemExit("--sharded needs rows that are a multiple of 16 bytes")
    dev = torch.device("cuda", torch.cuda.current_device())
    stream = torch.cuda.current_stream()
    G = max(1, int(args.halo_steps))
    sw = ShardedSweep(wk.dims, wk.radius, wk.shape, wk.weights(), wk.boundary, rank=rank, world=world, dist=dist,
                      halo_steps=G, overlap=not args.no_overlap)
    a_host = wk.input()                                  # every rank draws the same seeded field and keeps its slab
    ext = torch.zeros(sw.local_dims, dtype=torch.from_numpy(a_host[:1]).dtype, device=dev)
    sw.interior(ext).copy_(torch.from_numpy(a_host[sw.z0:sw.z1]))
    start = ext.clone()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    props = torch.cuda.get_device_properties(torch.cuda.current_device())
    sampler = ClockSampler(f"GPU-{props.uuid}" if hasattr(props, "uuid") else str(torch.cuda.current_device()))
    sampler.start()
    for _ in range(args.warmup):
        ext.copy_(start)
        sw.apply(ext, wk.steps)
    barrier()
    launches0 = sw._plan.launches
    total = 0.0
    t_wall0 = time.time()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(args.steps):                          # the restore of the start field stays outside the timing
        ext.copy_(start)
        barrier()
        e0.record(stream)
        sw.apply(ext, wk.steps)
        e1.record(stream)
        barrier()
        total += max_over_ranks(e0.elapsed_time(e1), dist, dev)
    t_wall1 = time.time()
    sampler.stop()
    clocks = sampler.summary(t_wall0, t_wall1)
    clocks["sampled_over"] = "the timed applies of rank 0 (restores of the start field and barriers included)"
    launches = sw._plan.launches - launches0
    status = sw._plan.query_status()
    info = {"variant": sw._plan.variant, "fuse_steps": sw._plan.get(b.KEY_FUSE_STEPS) if wk.steps > 1 else 1}
    sw.close()
    if rank == 0:
        if status != b.OK:
            raise SystemExit("device status word reports a timeout; results are invalid")
        s = sharded_job_summary(wk.dims, wk.radius, wk.steps, G, args.steps, total, world, wk.itemsize)
        peak, peak_kind = measured_hbm_peak()
        line = {
            "metric": METRIC, "value": round(s["value"], 3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(total / args.steps, 5), "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "f64" if wk.itemsize == 8 else "f32",
            "data": "synthetic (seeded numpy default_rng fields; see config.workload)",
            "config": {"workload": f"{wk.name}: {wk.description}", "dims": list(wk.dims), "radius": wk.radius,
                       "taps": wk.taps(), "time_steps_per_apply": wk.steps,
                       "parallelism": "one grid in %d slab(s) along the slowest axis, %d plane(s) per rank; halo "
                                      "exchange by NCCL point-to-point sends into the receiver's ghost planes"
                                      % (world, wk.dims[0] // world),
                       "halo_steps": G, "overlap_exchange_with_inner_planes": bool(sw.overlap),
                       "exchange_bytes_per_rank_per_time_step": int(s["exchange_bytes_per_rank_per_time_step"]),
                       "messages_per_rank_per_apply": s["messages_per_rank_per_apply"],
                       "timing": "each apply between barriers, CUDA events on the launching stream, max over ranks",
                       **info},
            "effective_gbs": round(2.0 * wk.itemsize * s["value"], 1),
            "frac_of_measured_hbm_times_n_gpus": round(2.0 * wk.itemsize * s["value"] / (peak * world), 4),
            "gpu_launches": int(launches), "clocks": clocks,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


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
                   "taps": wk.taps(), "time_steps_per_apply": wk.steps, "sample": sample_desc,
                   "input_sha256": wl.sha256(a_host)},
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
    ap.add_argument("--workload", default=None, choices=sorted(wl.WORKLOADS))
    ap.add_argument("--dims", default=None, help="override the grid, e.g. 256,512,512 (profiling on smaller cases)")
    ap.add_argument("--variant", default="auto", choices=["auto", "generic", "stream", "fused"])
    ap.add_argument("--tile-y", dest="tile_y", type=int, default=None)
    ap.add_argument("--rows-per-thread", dest="rows_per_thread", type=int, default=None)
    ap.add_argument("--chunk-z", dest="chunk_z", type=int, default=None)
    ap.add_argument("--stages", type=int, default=None)
    ap.add_argument("--fuse-steps", dest="fuse_steps", type=int, default=None)
    ap.add_argument("--tile-x", dest="tile_x", type=int, default=None, help="region width of fused 3D passes")
    ap.add_argument("--streaming-store", dest="streaming_store", type=int, default=None)
    ap.add_argument("--also", default="cfg1,cfg3,cfg4,cfg5,cfg5L,cfg5L_periodic,cfg5L_f64,box27_iterated,paper2d,paper2d_f64,heat2d", help="other workloads summarised in all_configs")
    ap.add_argument("--also-steps", dest="also_steps", type=int, default=20)
    ap.add_argument("--also-cpu-seconds", dest="also_cpu_seconds", type=float, default=2.0,
                    help="oracle baseline beside every entry of all_configs (0 = off)")
    ap.add_argument("--also-clock-seconds", dest="also_clock_seconds", type=float, default=0.5,
                    help="sustained window (and clock samples) of every entry of all_configs (0 = off)")
    ap.add_argument("--no-all-configs", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-steps", dest="e2e_steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", dest="cpu_seconds", type=float, default=12.0)
    ap.add_argument("--reference-seconds", dest="reference_seconds", type=float, default=90.0)
    ap.add_argument("--clock-seconds", dest="clock_seconds", type=float, default=1.5)
    ap.add_argument("--cudnn", type=int, default=1)
    ap.add_argument("--sharded", action="store_true",
                    help="all ranks share one grid (slabs along the slowest axis, halo exchange over NCCL)")
    ap.add_argument("--halo-steps", dest="halo_steps", type=int, default=2,
                    help="--sharded: time steps between two halo exchanges (1 overlaps the exchange with the inner planes)")
    ap.add_argument("--no-overlap", action="store_true", help="--sharded, halo-steps 1: exchange first, then sweep")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.workload is None:
        args.workload = "cfg5L" if args.sharded else "cfg2"
    if args.impl == "reference":
        run_reference(args)
    elif args.sharded:
        run_sharded(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
