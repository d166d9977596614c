#!/usr/bin/env python
"""Benchmark of the RPS synchronisation step.

    python bench.py [--gpus N] [--steps K] [--warmup W]            # every workload, cfg3 as the headline
    python bench.py --workload cfg5 [--p 0.1] [--kernel 3 ...]     # one workload (sweeps, profiler captures)
    python bench.py --impl reference ...                           # the CPU oracle on the host cores

A step is one pass of the whole hot path (drop masks, local SGD step, masked
average, masked write-back) over all n replicas.  The metric is replica-params
synchronised per second, n*d per step.  Without --workload the line's top-level
fields describe the headline workload (the largest fp32 model) and `workloads`
holds every configuration, the swept ones with each drop probability.  With N > 1 (torchrun, one rank per GPU)
every rank runs an independent replica of the job: the path needs no exchange
between GPUs, so there is no collective on the data path; only the timing is
reduced (max over ranks).  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import sys
import threading
import time
from dataclasses import replace

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "replica_params_synchronised_per_sec"
UNIT = "replica-params/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of one fused-kernel launch (dram__bytes_read.sum + dram__bytes_write.sum) from
# the ncu captures summarised under profiles/, keyed by workload; valid only for the kernel
# sources whose digest is recorded with it.  "bytes_per_launch": mean of 10 consecutive launches
# of this benchmark at full size with the caches left as the launch before left them (one-pass
# capture), which is the state the timed steps run in: a step starts on the columns that the step
# before it touched last, so part of x and b is still in L2 and the traffic is below the
# algorithmic bytes.  "cold_bytes_per_launch": one launch alone at full size with the caches flushed first
# (also a one-pass capture; the writes of the last lines are still in L2 when the launch ends).  Both are bytes PER
# STEP: cfg5's steps go out several per launch, and its figure is one launch of 32 steps divided by 32 (one step per
# launch, --fuse-steps 1, moves the same: 6,415,262,182 B).
NCU_TRAFFIC = {
    "kernel_digest": "0aeaffc63f21b5c0",
    "bytes_per_launch": {"cfg2": 962079770, "cfg3": 4805608013, "cfg4": 1425085158, "cfg5": 6411869744},
    "cold_bytes_per_launch": {"cfg2": 1020622080, "cfg3": 4859442944, "cfg4": 1488037376, "cfg5": 6387771392},
}


# Lane instructions (warp instructions x 32) per replica-param and step of the temporally blocked kernel, from
# ncu's smsp__inst_executed.sum of one launch of `bench.py --block-steps 16` (profiles/), keyed by workload.
BLOCKED_LANE_INSTRUCTIONS = {
    "kernel_digest": "2894f7e15240b1f2",
    "per_replica_param_step": {"cfg2": 19.32, "cfg3": 20.46, "cfg4": 20.97, "cfg5": 20.56},
}


def blocked_kernel_digest() -> str:
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_1810_07766_b200", "csrc")
    for name in ("rps_device.cuh", "rps_blocked.cu"):
        with open(os.path.join(csrc, name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


# rps_options fields that shape the kernels without changing what is computed (command-line flags of the same names)
SHAPE_OPTIONS = ("kernel", "workers_per_lane", "stages", "consumer_warps", "copy_mode", "slice_bytes", "store_mode",
                 "traversal", "l2_policy", "launch_overlap", "block_steps", "team_warps", "early_targets", "fuse_steps")


def kernel_digest() -> str:
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_1810_07766_b200", "csrc")
    # the fused kernels, their arithmetic and the choice of the default shape
    for name in ("rps_device.cuh", "rps_tma.cuh", "rps_staged.cuh", "rps_staged.cu", "rps_ring.cu", "rps_stream.cu",
                 "rps_kernels.cu"):
        with open(os.path.join(csrc, name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def fused_kernel_name(args, w) -> str:
    """Which fused kernel the library picks for this workload (see launch_fused in csrc/rps_kernels.cu)."""
    small = w.n * w.d * w.elem_bytes < 148 * 8192
    if args.kernel == 1 or (args.kernel == 0 and small):
        return "rps_fused_direct_kernel"
    block_cols = -(-w.d // w.n)
    stream_built = (w.n >= 2 and not (args.average_gradients and args.track)
                    and block_cols >= (8 if w.dtype == "bf16" else 4))
    staged_only = args.workers_per_lane or args.copy_mode or args.slice_bytes
    power_of_two = w.n & (w.n - 1) == 0
    padded = 8
    while padded < w.n:
        padded *= 2
    if w.dtype != "bf16":
        streamed = not power_of_two or (not args.average_gradients and (w.n == 2 or (w.n == 4 and args.track)))
    elif args.track:
        streamed = True
    elif args.average_gradients:
        streamed = w.n < 5 or (w.n >= 9 and 5 * w.n <= 4 * padded)
    else:
        streamed = not power_of_two or w.n > 32 or w.n < 8
    if stream_built and (args.kernel == 4 or (args.kernel == 0 and streamed and not staged_only)):
        return "rps_fused_stream_kernel"
    ring_built = w.dtype == "bf16" and w.n > 4 and not args.track
    staged_only = args.workers_per_lane or args.consumer_warps or args.copy_mode or args.slice_bytes
    if ring_built and (args.kernel == 3 or (args.kernel == 0 and not staged_only)):
        return "rps_fused_ring_kernel"
    return "rps_fused_staged_kernel"


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while a region runs."""

    REASONS = {
        0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
        0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
        0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
    }

    def __init__(self, index: int, period_s: float = 0.002):
        self.index, self.period = index, period_s
        self.samples, self.reason_bits, self.power_w = [], 0, []
        self.max_mhz = None
        self._stop = threading.Event()
        self._ready = threading.Event()
        self._thread = None
        self._nvml = None

    def __enter__(self):
        try:
            import pynvml

            pynvml.nvmlInit()
            self._nvml = pynvml
            self._dev = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._dev, pynvml.NVML_CLOCK_SM))
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
            self._ready.wait(timeout=2.0)
        except Exception:
            self._nvml = None
        return self

    def _reasons(self):
        nv = self._nvml
        for fn in ("nvmlDeviceGetCurrentClocksEventReasons", "nvmlDeviceGetCurrentClocksThrottleReasons"):
            if hasattr(nv, fn):
                return int(getattr(nv, fn)(self._dev))
        return 0

    def _run(self):
        nv = self._nvml
        try:  # the first queries of a process can take tens of milliseconds: make them before the region starts
            nv.nvmlDeviceGetClockInfo(self._dev, nv.NVML_CLOCK_SM)
            self._reasons()
            nv.nvmlDeviceGetPowerUsage(self._dev)
        except Exception:
            pass
        self._ready.set()
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._dev, nv.NVML_CLOCK_SM)))
                self.reason_bits |= self._reasons() & ~0x1
                self.power_w.append(nv.nvmlDeviceGetPowerUsage(self._dev) / 1000.0)
            except Exception:
                pass
            time.sleep(self.period)

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2.0)
        return False

    def summary(self):
        reasons = [name for bit, name in self.REASONS.items() if self.reason_bits & bit]
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_min_mhz": min(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(self.samples),
                "power_w_max": max(self.power_w) if self.power_w else None}


# ----------------------------------------------------------------------------- multi-rank plumbing

def dist_env():
    env = os.environ
    return int(env.get("RANK", "0")), int(env.get("LOCAL_RANK", "0")), int(env.get("WORLD_SIZE", "1"))


def max_over_ranks(value: float, device=None) -> float:
    """Largest `value` over all ranks of the default process group (identity without one)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


# ----------------------------------------------------------------------------- the CUDA arm

def timed_steps(torch, stream, fn, device):
    """Device time of fn() in ms: barrier + synchronize on both sides, events on the launch stream."""
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize(device)
    start.record(stream)
    fn()
    stop.record(stream)
    torch.cuda.synchronize(device)
    barrier()
    return max_over_ranks(start.elapsed_time(stop), device)


def in_situ_copy_gbs(torch, device) -> float:
    """Read+write bytes per second of a plain device copy of 1 GiB on this GPU, now (best of 6): the same
    kind of measurement as the recorded peak, taken in this process, because the machine's GPUs differ."""
    a = torch.empty(1 << 29, dtype=torch.bfloat16, device=device)
    c = torch.empty_like(a)
    best = float("inf")
    for _ in range(6):
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        c.copy_(a)
        stop.record()
        torch.cuda.synchronize(device)
        best = min(best, start.elapsed_time(stop))
    del a, c
    torch.cuda.empty_cache()
    return 2 * (1 << 30) / (best * 1e-3) / 1e9


def oracle_baseline(w, b, min_seconds=10.0, max_steps=8):
    """The CPU oracle, as it stands, on full-size steps of the workload (single thread): as many
    consecutive steps from x = 0 as it takes to fill `min_seconds` (one step of cfg3 or cfg5 already does)."""
    import oracle
    from paper_1810_07766_b200 import workloads as wl

    x = wl.make_initial(w)
    steps, t0 = 0, time.perf_counter()
    while steps < max_steps and (steps == 0 or time.perf_counter() - t0 < min_seconds):
        oracle.step(x, b, dtype=w.dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t=steps)
        steps += 1
    dt = time.perf_counter() - t0
    return {"value": w.n * w.d * steps / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{steps} full-size step(s) (n={w.n}, d={w.d}) of the fp64 C oracle, {dt:.2f} s, single thread"}


# The workloads of a default run, the headline first: the largest fp32 model (d >= 11M; its L2 carry-over
# between steps is the smallest of the fp32 workloads), then the other configurations, the swept ones once per
# drop probability of their sweep.
HEADLINE = "cfg3"
DEFAULT_SUITE = ("cfg3", "cfg2", "cfg4", "cfg5")


def resolve_workload(args, name, p=None):
    from paper_1810_07766_b200 import workloads as wl

    w = wl.WORKLOADS[name]
    if p is not None:
        w = replace(w, p=p)
    if args.d is not None:
        w = w.scaled(d=args.d)
    if args.sigma is not None:
        w = replace(w, sigma=args.sigma)
    if args.n is not None:
        w = replace(w, n=args.n, name=f"{w.name}@n={args.n}")
    return w


def measure(args, ctx, w, b, *, with_e2e, with_upwards, p_sweep=()):
    """Times one workload on this rank's GPU.  Returns its entry of the JSON line.

    Pass 1 is W warm-up steps and exactly K timed steps (first, so that nothing but the warm-up precedes the timed
    steps: the largest workload reaches the board's power cap some 50 ms into a run), pass 2 brackets every launch
    with events (per-kernel durations; this serialises what the programmatic launch overlap hides, so the mean
    launch can be longer than the step it is part of; it starts after a second of idle, from the power state pass 1
    started from), pass 3 (optional) the same steps through the host-buffer call.  `p_sweep`: further drop probabilities timed on the same arrays (pass 1 only).
    """
    import numpy as np

    from paper_1810_07766_b200 import binding

    torch, device, rank, local_rank, world = ctx["torch"], ctx["device"], ctx["rank"], ctx["local_rank"], ctx["world"]
    begin, cols, jobs = 0, w.d, world
    if args.shard and world > 1:
        begin, cols = binding.shard_columns(w.d, world, rank)
        if cols == 0:
            raise SystemExit("--shard: the model is too short for this many ranks")
        b = np.ascontiguousarray(b[:, begin:begin + cols])
        jobs = 1
    sharded = jobs != world
    shape = {name: getattr(args, name) for name in SHAPE_OPTIONS}  # all 0 = the library's choice
    bytes_per_step = w.bytes_per_step * cols // w.d

    mask_window = 32  # steps whose masks one launch of the mask kernel generates (rps_options.mask_window)

    def make(p, **more):
        r = binding.RPS(w.n, w.d, p, w.gamma, w.seed, dtype=w.dtype, sigma=w.sigma,
                        average_gradients=args.average_gradients, shard_begin=begin if sharded else 0,
                        shard_cols=cols if sharded else 0, row_skew_lines=args.row_skew_lines, **{**shape, **more})
        r.set_targets(b)
        if args.track:  # every step of the run also records the distance to the optimum and the consensus error
            r.track(2 * max(args.warmup, 3) + 2 * args.steps + args.warmup + 64)
        return r

    def timed_run(r):
        r.step_n(args.warmup)
        before = r.launch_count()
        ms = timed_steps(torch, r.stream, lambda: r.step_n(args.steps), device)
        return ms, r.launch_count() - before

    r = make(w.p)
    # the clocks are sampled over the warm-up and the timed steps (an NVML query takes a millisecond or so)
    with ClockSampler(local_rank) as clocks:
        total_ms, gpu_launches = timed_run(r)
    # a second of idle, so that the next pass starts from the power state the first one started from
    torch.cuda.synchronize(device)
    time.sleep(1.0)
    r.step_n(max(args.warmup, 3))
    r.profile(True)
    profile_steps = max(args.steps, mask_window + 1)  # long enough to see the mask kernel, which runs once per window
    r.step_n(profile_steps)
    fused_ms, fused_n, mask_ms, mask_n = r.profile_read()
    r.profile(False)

    e2e = None
    if with_e2e:
        tdtype = torch.float32 if w.dtype == "f32" else torch.int16  # bf16 bit patterns travel as 16-bit words
        x_host = torch.zeros((w.n, cols), dtype=tdtype).pin_memory()
        b_host = torch.from_numpy(b if w.dtype == "f32" else b.view(np.int16)).pin_memory()
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        for _ in range(2):
            r.step_host(x_host, b_host)
        e2e_ms = timed_steps(torch, r.stream, lambda: [r.step_host(x_host, b_host) for _ in range(e2e_steps)], device)
        e2e = {"value": jobs * w.n * w.d * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "steps": e2e_steps,
               "h2d_bytes_per_step": 2 * w.n * cols * w.elem_bytes, "d2h_bytes_per_step": w.n * cols * w.elem_bytes,
               "call": "rps_step_host (pinned host x and b)"}
        del x_host, b_host
    r.close()

    ms_per_step = total_ms / args.steps
    peak, peak_kind = measured_peak_gbs()
    # a launch may run several steps (rps_options.fuse_steps): bytes per launch = bytes per step x steps per launch
    fused_avg_ms = fused_ms / max(fused_n, 1)
    steps_per_launch = profile_steps / max(fused_n, 1)
    achieved = bytes_per_step * steps_per_launch / (fused_avg_ms * 1e-3) / 1e9
    whole_step = bytes_per_step / (ms_per_step * 1e-3) / 1e9
    traffic = traffic_cold = None
    default_shape = not (any(shape.values()) or args.average_gradients or args.track or sharded or
                         args.row_skew_lines != -1)
    if default_shape and NCU_TRAFFIC["kernel_digest"] == kernel_digest():
        traffic = NCU_TRAFFIC["bytes_per_launch"].get(w.name)
        traffic_cold = NCU_TRAFFIC["cold_bytes_per_launch"].get(w.name)
    roofline = {
        "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
        # per launch, like `achieved`: the recorded bytes are per step
        "traffic": traffic * steps_per_launch if traffic else None, "traffic_per_step": traffic,
        "traffic_cold_cache": traffic_cold, "peak_kind": f"of {peak_kind}",
        "kernel": fused_kernel_name(args, w), "avg_launch_ms": fused_avg_ms, "launches_timed": fused_n,
        "steps_per_launch": steps_per_launch,
        # the same bytes over the time of a whole step inside a train of steps (launch overlap kept, mask kernel in)
        "whole_step_achieved": whole_step, "whole_step_frac": whole_step / peak,
        "whole_step_frac_of_8TBs_nominal": whole_step / 8000.0,
        # what crossed the HBM interface (ncu, when recorded for these sources) over the same times
        "dram_achieved": traffic * steps_per_launch / (fused_avg_ms * 1e-3) / 1e9 if traffic else None,
        "dram_frac": traffic * steps_per_launch / (fused_avg_ms * 1e-3) / 1e9 / peak if traffic else None,
        "dram_whole_step_achieved": traffic / (ms_per_step * 1e-3) / 1e9 if traffic else None,
        "dram_whole_step_frac_of_8TBs_nominal": traffic / (ms_per_step * 1e-3) / 8e12 if traffic else None,
        "note": "avg_launch_ms brackets every launch with events, which serialises the launches and loses the "
                "programmatic launch overlap a train of steps has: it can exceed ms_per_step",
        "mask_kernel_ms_per_launch": mask_ms / max(mask_n, 1) if mask_n else None,
        "mask_kernel_ms_per_step_amortised": mask_ms / mask_n / mask_window if mask_n else None,
        "mask_launches_timed": mask_n,
    }
    entry = {
        "workload": f"{w.name}: n={w.n} workers, d={w.d} {w.dtype}, p={w.p}, gamma={w.gamma}, sigma={w.sigma}, "
                    f"seed={w.seed}; quadratic objective, b_i ~ N({'mu_i' if w.hetero else '0'},1)",
        "n": w.n, "d": w.d, "p": w.p, "dtype": w.dtype, "cols_on_this_gpu": cols,
        "value": jobs * w.n * w.d * args.steps / (total_ms * 1e-3), "unit": UNIT, "ms_per_step": ms_per_step,
        "algorithmic_bytes_per_step": bytes_per_step, "hbm_gbs_whole_step": whole_step,
        "frac_of_8TBs_nominal": whole_step / 8000.0,
        "l2": "inputs larger than L2 (x and b are %.0f MB each)" % (w.n * cols * w.elem_bytes / 1e6),
        "clocks": clocks.summary(), "gpu_launches": gpu_launches, "roofline": roofline, "e2e": e2e,
        "sharded": sharded, "kernel_shape": shape,
    }
    if p_sweep:
        entry["p_sweep"] = {}
        for p in p_sweep:
            rp = make(p)
            ms, _ = timed_run(rp)
            rp.close()
            entry["p_sweep"][str(p)] = {"ms_per_step": ms / args.steps,
                                        "value": jobs * w.n * w.d * args.steps / (ms * 1e-3),
                                        "hbm_gbs_whole_step": bytes_per_step / (ms / args.steps * 1e-3) / 1e9}
    if with_upwards:
        # every step walks the columns upwards: no step starts on what the step before it left in L2
        ru = make(w.p, traversal=1)
        ms, _ = timed_run(ru)
        ru.close()
        entry["traversal_always_upwards"] = {"ms_per_step": ms / args.steps,
                                             "hbm_gbs_whole_step": bytes_per_step / (ms / args.steps * 1e-3) / 1e9,
                                             "frac_of_8TBs_nominal": bytes_per_step / (ms / args.steps * 1e-3) / 8e12}
    torch.cuda.empty_cache()
    return entry


def blocked_roofline(args, ctx, w, cols, entry):
    """Several steps per pass over x and b: the pass is bound by the arithmetic of a step, not by HBM.
    achieved = lane instructions executed per second (ncu's count per replica-param and step, recorded above
    with the digest of the kernel sources, x replica-params x steps per second); peak = one warp instruction of
    32 lanes per scheduler and clock."""
    torch, device = ctx["torch"], ctx["device"]
    old = entry["roofline"]
    fused_avg_ms, fused_n = old["avg_launch_ms"], old["launches_timed"]
    steps_per_launch = old["steps_per_launch"]
    rp_steps_per_s = w.n * cols * steps_per_launch / (fused_avg_ms * 1e-3)
    sm_count = torch.cuda.get_device_properties(device).multi_processor_count
    mhz = entry["clocks"].get("sm_max_mhz") or 1965
    peak_alu = sm_count * 4 * 32 * mhz * 1e6 / 1e12
    instr = None
    if BLOCKED_LANE_INSTRUCTIONS["kernel_digest"] == blocked_kernel_digest():
        instr = BLOCKED_LANE_INSTRUCTIONS["per_replica_param_step"].get(w.name)
    alu = instr * rp_steps_per_s / 1e12 if instr else None
    return {"bound": "alu", "achieved": alu, "peak": peak_alu, "unit": "T lane-instructions/s",
            "frac": alu / peak_alu if alu else None, "traffic": None,
            "peak_kind": "derived: SMs x 4 schedulers x 32 lanes x max SM clock",
            "kernel": "rps_fused_blocked_kernel", "lane_instructions_per_replica_param_step": instr,
            "avg_launch_ms": fused_avg_ms, "launches_timed": fused_n, "steps_per_launch": steps_per_launch,
            "hbm_gbs_moved_per_launch": 3 * w.elem_bytes * w.n * cols / (fused_avg_ms * 1e-3) / 1e9}


def run_cuda(args):
    import torch

    from paper_1810_07766_b200 import build
    from paper_1810_07766_b200 import workloads as wl

    rank, local_rank, world = dist_env()
    if world != args.gpus:
        if world == 1 and args.gpus > 1:
            raise SystemExit("--gpus N > 1 must be launched with torchrun, one rank per GPU")
        raise SystemExit(f"--gpus {args.gpus} does not match WORLD_SIZE {world}")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path for the product arm")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=device)
    build.build()
    ctx = {"torch": torch, "device": device, "rank": rank, "local_rank": local_rank, "world": world}

    # one workload when one is named (tuning sweeps, profiler captures), else the whole suite with the headline first
    names = (args.workload,) if args.workload else DEFAULT_SUITE
    headline = names[0]
    entries, cpu = {}, None
    for name in names:
        sweep = wl.WORKLOADS[name].p_sweep if (args.workload is None and args.p is None) else ()
        w = resolve_workload(args, name, args.p)
        b = wl.make_targets(w)
        first = name == headline
        entry = measure(args, ctx, w, b, with_e2e=first and not args.skip_e2e,
                        with_upwards=first and args.workload is None and args.traversal == 0,
                        p_sweep=tuple(p for p in sweep if p != w.p))
        if args.block_steps > 1:
            entry["roofline"] = blocked_roofline(args, ctx, w, entry["cols_on_this_gpu"], entry)
        if first and rank == 0 and world == 1 and not args.no_cpu_baseline:
            cpu = oracle_baseline(w, b)
        entries[name] = entry
        del b
    copy_gbs = in_situ_copy_gbs(torch, device)

    top = entries[headline]
    line = {
        "metric": METRIC, "value": top["value"], "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": top["ms_per_step"],
        "higher_is_better": True, "scaling": "strong" if top["sharded"] else "weak", "vs_baseline": None,
        "dtype": top["dtype"], "data": "synthetic",
        "config": {
            "workload": top["workload"], "n": top["n"], "d": top["d"], "p": top["p"],
            "replicas": ("one model cut by columns over the GPUs, no collective" if top["sharded"]
                         else "one independent job per GPU, no collective"),
            "kernel_shape": top["kernel_shape"],
            "average": "gradients" if args.average_gradients else "models",
            "tracked": bool(args.track),
            "l2": top["l2"],
            "algorithmic_bytes_per_step": top["algorithmic_bytes_per_step"],
            "hbm_gbs_whole_step": top["hbm_gbs_whole_step"],
            "frac_of_8TBs_nominal": top["frac_of_8TBs_nominal"],
        },
        "clocks": top["clocks"],
        "e2e": top["e2e"],
        "gpu_launches": top["gpu_launches"],
        "roofline": dict(top["roofline"], in_situ_copy_gbs=copy_gbs,
                         frac_of_in_situ_copy=(top["roofline"]["achieved"] / copy_gbs
                                               if top["roofline"]["bound"] == "hbm" else None)),
    }
    if len(entries) > 1:
        # every workload of the run, the headline included, each with its own clocks and roofline
        line["workloads"] = {name: {k: v for k, v in e.items() if k not in ("kernel_shape", "sharded")}
                             for name, e in entries.items()}
    if cpu is not None:
        line["cpu_baseline"] = cpu
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist

        dist.destroy_process_group()


# ----------------------------------------------------------------------------- the reference arm

def run_reference(args):
    """The CPU oracle timed on the host: each step is one oracle step over a prefix of the
    workload's columns (true block and noise indices), sized to keep the run to minutes."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    import numpy as np

    import oracle
    from paper_1810_07766_b200 import workloads as wl

    w = wl.WORKLOADS[args.workload or HEADLINE]
    if args.p is not None:
        w = replace(w, p=args.p)
    cols_n = min(w.d, args.reference_columns)
    sample = wl.Workload(w.name, n=w.n, d=cols_n, dtype=w.dtype, p=w.p, gamma=w.gamma, sigma=w.sigma, seed=w.seed,
                         steps=w.steps, hetero=w.hetero)
    b = wl.make_targets(sample)
    x = wl.make_initial(sample)
    cols = np.arange(cols_n, dtype=np.int64)

    def one(t):
        oracle.step_columns(w.d, cols, x, b, dtype=w.dtype, gamma=w.gamma, sigma=w.sigma, p=w.p, seed=w.seed, t=t)

    for t in range(args.warmup):
        one(t)
    t0 = time.perf_counter()
    for t in range(args.warmup, args.warmup + args.steps):
        one(t)
    dt = time.perf_counter() - t0
    value = w.n * cols_n * args.steps / dt
    sample_txt = f"each step = the first {cols_n} of {w.d} columns, all {w.n} workers, fp64 C oracle, single thread"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name}: n={w.n} workers, d={w.d} {w.dtype}, p={w.p}, gamma={w.gamma}, "
                               f"sigma={w.sigma}, seed={w.seed}", "sample": sample_txt},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample_txt},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=("cuda", "reference"), default="cuda")
    ap.add_argument("--workload", choices=("cfg1", "cfg2", "cfg3", "cfg4", "cfg5"), default=None,
                    help="time this workload only (default: cfg3 as the headline, then cfg2 and cfg4 with every drop "
                         "probability of their sweeps, and cfg5, all in one JSON line)")
    ap.add_argument("--p", type=float, default=None, help="override the drop probability (p sweeps)")
    ap.add_argument("--d", type=int, default=None, help="override the model size (small profiler captures)")
    ap.add_argument("--n", type=int, default=None, help="override the number of workers (shape sweeps)")
    ap.add_argument("--sigma", type=float, default=None,
                    help="override the noise level (0 = no gradient noise: the step as pure data movement)")
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--reference-columns", type=int, default=500_000)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true", help="tuning sweeps only: leave the host-buffer pass out")
    ap.add_argument("--kernel", type=int, default=0,
                    help="0 library's choice, 1 direct loads, 2 staged (producer warp), 3 self-refilling ring (bf16), "
                         "4 workers streamed through a ring per warp")
    ap.add_argument("--team-warps", type=int, default=0, help="ring kernel: warps that share a tile")
    ap.add_argument("--row-skew-lines", type=int, default=-1,
                    help="extra 128-byte lines of padding per device row (-1 = the library's choice)")
    ap.add_argument("--workers-per-lane", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--consumer-warps", type=int, default=0)
    ap.add_argument("--slice-bytes", type=int, default=0, help="staged kernel, bf16: 16 or 8 bytes per lane and row")
    ap.add_argument("--average-gradients", action="store_true",
                    help="time the gradient-averaging comparison of Section 5 instead of RPS (model averaging)")
    ap.add_argument("--traversal", type=int, default=0,
                    help="0: odd steps walk the columns downwards (default); 1: every step upwards")
    ap.add_argument("--l2-policy", type=int, default=0, help="staged kernel: 1 plain loads, 2 targets evict-first")
    ap.add_argument("--launch-overlap", type=int, default=0,
                    help="staged kernel: 1 plain launches, 2 programmatic stream serialization (default)")
    ap.add_argument("--early-targets", type=int, default=0,
                    help="1: every copy waits for the kernel ahead in the stream; 2: the first stages' copies of b do not")
    ap.add_argument("--fuse-steps", type=int, default=0,
                    help="rps_step_n: 1 one launch per step; 2 several steps per launch where the kernel takes them")
    ap.add_argument("--block-steps", type=int, default=0,
                    help="temporal blocking of rps_step_n: this many consecutive steps per pass over x and b (<= 32); "
                         "the pass is then bound by arithmetic, not by HBM (off by default)")
    ap.add_argument("--shard", action="store_true",
                    help="with --gpus N > 1: cut one model by columns over the ranks (strong scaling) instead of "
                         "running one whole model per rank")
    ap.add_argument("--track", action="store_true",
                    help="time tracked steps: distance to the optimum and consensus error as a by-product of the pass")
    ap.add_argument("--store-mode", type=int, default=0, help="staged kernel: 1 register stores, 2 TMA stores")
    ap.add_argument("--copy-mode", type=int, default=0, help="staged kernel: 1 bulk copy per row, 2 TMA boxes")
    args = ap.parse_args(argv)
    if args.steps < 1 or args.warmup < 0:
        raise SystemExit("--steps must be >= 1 and --warmup >= 0")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
