#!/usr/bin/env python
"""Throughput of the K-Means ASGD worker loop on B200: samples/s, achieved HBM GB/s, roofline fraction.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload stream]

One bench "step" is one full pass of every worker over its shard in free-running mode (a single
asgd_run launch: mini-batch draw, assignment, per-centre sums, gradient, receive buffers with the
Parzen test, update, puts).  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "K-Means ASGD samples/s"
UNIT = "samples/s"
CPU_SAMPLE_ROWS = 1 << 25          # prefix of the workload the CPU baseline runs on (all cores)
CPU_SAMPLE_ROWS_ONE_CORE = 1 << 22 # and on one core
NOMINAL_HBM_GBS = 8000.0
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of the worker kernel per algorithmic byte, each from one
# small-case ncu capture of that kernel (a few hundred MB of samples, more than L2 holds; the traffic grows in
# proportion to the rows a launch processes).  A record is valid only for the kernel sources it was taken on.
KERNEL_SOURCES = {
    "fp32-stream": ("asgd_common.cuh", "asgd_step_tail.cuh", "asgd_stream.cuh"),
    "fp32-tiled": ("asgd_common.cuh", "asgd_step_tail.cuh", "asgd_stream.cuh", "asgd_tiled.cuh"),
    "tcgen05-fp16": ("asgd_common.cuh", "asgd_step_tail.cuh", "asgd_stream.cuh", "asgd_tc.cuh"),
    "tcgen05-bf16x3": ("asgd_common.cuh", "asgd_step_tail.cuh", "asgd_stream.cuh", "asgd_tc.cuh"),
}
TRAFFIC_CAPTURES = {
    # (kernel, workload): source key at capture time, captured DRAM bytes / algorithmic bytes
    ("fp32-stream", "stream"): {"kernel_sha1": "f1a5085d74a9", "traffic_per_algorithmic_byte": 671.54 / 663.51},
    ("fp32-tiled", "sweep"): {"kernel_sha1": "b132cff9499b", "traffic_per_algorithmic_byte": 1092.63 / 1091.17},
    # tensor-core path: the samples are read twice by design (16-bit copy for the scores, fp32 master for the sums:
    # 1.5 x), the rest is the workers' states, which L2 does not hold for dense (222 MB) and barely for codebook
    ("tcgen05-fp16", "mid"): {"kernel_sha1": "957b3d9a3d43", "traffic_per_algorithmic_byte": 1645.06 / 1060.86},
    ("tcgen05-fp16", "dense"): {"kernel_sha1": "957b3d9a3d43", "traffic_per_algorithmic_byte": 3101.12 / 1241.51},
    ("tcgen05-fp16", "codebook"): {"kernel_sha1": "957b3d9a3d43", "traffic_per_algorithmic_byte": 1938.29 / 620.76},
}


def kernel_sha1(kernel):
    """First 12 hex digits of the SHA-1 over the sources a worker kernel is compiled from."""
    import hashlib
    h = hashlib.sha1()
    for name in KERNEL_SOURCES.get(kernel, ()):
        with open(os.path.join(ROOT, "paper_1505_04956_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:12]


def stream_kernel_sha1():
    return kernel_sha1("fp32-stream")


def captured_traffic(kernel, workload, algorithmic_bytes):
    """(bytes, how) of the DRAM traffic of one launch scaled from the stored capture, or (None, why not)."""
    rec = TRAFFIC_CAPTURES.get((kernel, workload))
    if rec is None:
        return None, "no capture of this kernel on this workload"
    if rec["kernel_sha1"] != kernel_sha1(kernel):
        return None, "the kernel has changed since its counters were taken"
    return algorithmic_bytes * rec["traffic_per_algorithmic_byte"], "scaled from a small-case ncu capture by the rows processed"


def env_int(name, default):
    try:
        return int(os.environ.get(name, default))
    except ValueError:
        return default


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            pk = json.load(f)
        return float(pk["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """SM clock and throttle-reason samples (NVML, read-only) taken by a thread while the timed region runs."""

    def __init__(self, gpu_index, period_s=0.002):
        self.gpu_index, self.period = gpu_index, period_s
        self.sm, self.reasons, self.sm_max = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._err = None

    def _loop(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.gpu_index)
            self.sm_max = float(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
            names = {
                "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            }
            get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                nv.nvmlDeviceGetCurrentClocksThrottleReasons
            while not self._stop.is_set():
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
                mask = int(get_reasons(h))
                for nm, bit in names.items():
                    if mask & bit:
                        self.reasons.add(nm)
                time.sleep(self.period)
            nv.nvmlShutdown()
        except Exception as exc:          # NVML missing: report it, do not fail the run
            self._err = repr(exc)[:120]

    def start(self):
        self._thread = threading.Thread(target=self._loop, daemon=True)
        self._thread.start()
        time.sleep(0.05)                  # let NVML initialise before the timed region begins

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=5)
        out = {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": self.sm_max,
               "samples": len(self.sm), "reasons": sorted(self.reasons)}
        if self._err:
            out["error"] = self._err
        return out


def algorithmic_bytes_per_pass(wl, steps, partial_rows=0):
    """One read of every used sample (d*4 B) plus the put payloads (rows*d*4 B per recipient per put)."""
    sample_bytes = wl.W * steps * wl.b * wl.d * 4
    puts = wl.W * wl.fanout * (steps // wl.comm_interval if wl.comm_interval > 0 else 0)
    return sample_bytes + puts * (partial_rows if partial_rows > 0 else wl.k) * wl.d * 4


def cpu_baseline(wl, sample_rows, threads=None, min_seconds=0.0):
    """The oracle, as it stands, on a prefix of the workload; returns (samples/s, description, threads)."""
    import numpy as np  # noqa: F401
    from oracle import asgd_oracle as orc
    from paper_1505_04956_b200 import inputs
    sub = wl.scaled(N=min(sample_rows, wl.N))
    X, _ = inputs.make_samples(sub, device="cpu")
    w0 = inputs.initial_centres(sub, X)
    th = threads or min(os.cpu_count() or 1, orc.max_threads(), sub.W)
    o = orc.Oracle(X.numpy(), w0.numpy(), W=sub.W, b=sub.b, eps=sub.eps, comm_interval=sub.comm_interval,
                   fanout=sub.fanout, seed=sub.seed, threads=th)
    rounds = sub.B
    t0 = time.perf_counter()
    done = 0
    while True:
        o.rounds(rounds)
        done += rounds
        dt = time.perf_counter() - t0
        if dt >= min_seconds:
            break
    val = sub.W * done * sub.b / dt
    desc = "first %d rows of the workload (W=%d, b=%d), %d synchronous rounds, %.1f s" % (sub.N, sub.W, sub.b, done, dt)
    o.close()
    return val, desc, o.threads


def run_reference(args):
    """--impl reference: the CPU oracle on bounded samples of the same workload."""
    from paper_1505_04956_b200 import inputs
    rank = env_int("RANK", 0)
    if rank != 0:
        return 0
    from oracle import asgd_oracle as orc
    wl = inputs.WORKLOADS[args.workload]
    sub = wl.scaled(N=min(args.reference_rows, wl.N))
    X, _ = inputs.make_samples(sub, device="cpu")
    w0 = inputs.initial_centres(sub, X)
    th = min(os.cpu_count() or 1, orc.max_threads(), sub.W)
    o = orc.Oracle(X.numpy(), w0.numpy(), W=sub.W, b=sub.b, eps=sub.eps, comm_interval=sub.comm_interval,
                   fanout=sub.fanout, seed=sub.seed, threads=th)
    for _ in range(args.warmup):
        o.rounds(sub.B)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        o.rounds(sub.B)
    dt = time.perf_counter() - t0
    val = sub.W * sub.B * sub.b * args.steps / dt
    sample = "each step = one pass over the first %d rows (W=%d, b=%d, %d rounds)" % (sub.N, sub.W, sub.b, sub.B)
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(1, args.steps), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "N": wl.N, "d": wl.d, "k": wl.k, "W": wl.W, "b": wl.b},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": o.threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)
    return 0


def measure(args, wl, dev, rank, world, dist, keep=False):
    """The timed region for one workload on this rank: W untimed passes, K timed passes (one asgd_run launch each)."""
    import torch
    import paper_1505_04956_b200 as pkg
    from paper_1505_04956_b200 import inputs, metrics
    # each rank owns an independent group of W workers on its own seeded shard (no cross-GPU exchange)
    wl_rank = wl.scaled(seed=dist.shard_seed(wl.seed, rank, world))
    X, mu = inputs.make_samples(wl_rank, device=dev)
    w0 = inputs.initial_centres(wl_rank, X)
    cfg = pkg.make_config(N=wl.N, d=wl.d, k=wl.k, W=wl.W, b=wl.b, eps=wl.eps, comm_interval=wl.comm_interval,
                          fanout=wl.fanout, seed=wl_rank.seed, parzen=0 if args.no_parzen else 1,
                          partial_rows=args.partial_rows, dist_path=args.dist_path)
    ctx = pkg.Asgd(cfg, X, w0)
    steps = wl.B                                   # one pass
    samples_per_pass = wl.W * steps * wl.b

    for _ in range(args.warmup):
        ctx.run(steps)
    ctx.sync()
    sampler = ClockSampler(dev.index)
    l0 = ctx.launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    ev[0].record()
    for s in range(args.steps):
        ctx.run(steps)
        ev[s + 1].record()
    torch.cuda.synchronize()
    dist.barrier()
    clocks = sampler.stop()
    ctx.sync()
    launches = ctx.launch_count() - l0
    per_launch_ms = [ev[s].elapsed_time(ev[s + 1]) for s in range(args.steps)]
    total_ms = dist.max_over_ranks(ev[0].elapsed_time(ev[-1]))
    value = world * samples_per_pass * args.steps / (total_ms * 1e-3)
    E_final = ctx.eval(0)
    E_mean = ctx.eval(-1)
    centre_err, _ = metrics.generator_centre_error(mu.cpu().numpy(), ctx.get_state(0).cpu().numpy())
    msgs = {"sent": 0, "received": 0, "accepted": 0, "overwritten": 0}
    for i in range(wl.W):
        st = ctx.get_stats(i)
        for key in msgs:
            msgs[key] += st[key]

    # roofline of the dominant kernel (the persistent worker kernel: one launch per bench step)
    kernel = ctx.path_name()
    hbm_peak, peak_kind = measured_peaks()
    launch_ms = statistics.mean(per_launch_ms)
    bytes_per_launch = algorithmic_bytes_per_pass(wl, steps, args.partial_rows)
    hbm_gbs = bytes_per_launch / (launch_ms * 1e-3) / 1e9
    traffic, traffic_kind = captured_traffic(kernel, wl.name, bytes_per_launch)
    flops = 2.0 * wl.k * wl.d * samples_per_pass
    common = {"traffic": traffic, "traffic_kind": traffic_kind, "kernel": kernel, "launch_ms": launch_ms,
              "algorithmic_bytes_per_launch": bytes_per_launch}
    dtype = "f32"
    if kernel == "fp32-tiled":
        # bound by the fp32 pipe: 2*k*d flops per sample against SMs x 128 lanes x 2 x max SM clock
        props = torch.cuda.get_device_properties(dev)
        alu_peak = props.multi_processor_count * 128 * 2 * (clocks.get("sm_max_mhz") or 1965.0) * 1e6 / 1e12
        ach = flops / (launch_ms * 1e-3) / 1e12
        roofline = dict(common, bound="alu", achieved=ach, peak=alu_peak, unit="TFLOP/s", frac=ach / alu_peak,
                        peak_kind="SMs x 128 fp32 lanes x 2 x max SM clock", algorithmic_flops_per_launch=flops, hbm_GBs=hbm_gbs)
    elif kernel.startswith("tcgen05"):
        # bound by the tensor pipe: the 2*k*d flops per sample of the -2 X W^T contraction against the measured sustained
        # BF16 rate (FP16 and BF16 share one nominal rate; the kernel is timed inside a long launch)
        tpeak, tkind = 1400.0, "fallback (sustained)"
        ppath = os.path.join(ROOT, "MEASURED_PEAKS.json")
        if os.path.exists(ppath):
            with open(ppath) as f:
                tpeak, tkind = float(json.load(f)["bf16_tflops_sustained"]), "measured (sustained)"
        ach = flops / (launch_ms * 1e-3) / 1e12
        if flops / (tpeak * 1e12) >= bytes_per_launch / (hbm_peak * 1e9):
            roofline = dict(common, bound="tensor", achieved=ach, peak=tpeak, unit="TFLOP/s", frac=ach / tpeak,
                            peak_kind="of " + tkind, algorithmic_flops_per_launch=flops, hbm_GBs=hbm_gbs)
        else:
            # few centres: reading the samples takes longer than the contraction, the launch is bound by HBM
            roofline = dict(common, bound="hbm", achieved=hbm_gbs, peak=hbm_peak, unit="GB/s", frac=hbm_gbs / hbm_peak,
                            peak_kind="of " + peak_kind, frac_of_nominal_8TBs=hbm_gbs / NOMINAL_HBM_GBS,
                            algorithmic_flops_per_launch=flops, tensor_TFLOPs=ach)
        dtype = "f16" if kernel.endswith("fp16") else "bf16"
    else:
        roofline = dict(common, bound="hbm", achieved=hbm_gbs, peak=hbm_peak, unit="GB/s", frac=hbm_gbs / hbm_peak,
                        peak_kind="of " + peak_kind, frac_of_nominal_8TBs=hbm_gbs / NOMINAL_HBM_GBS)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": dtype, "data": "synthetic",
        "config": {"workload": wl.name, "N": wl.N, "d": wl.d, "k": wl.k, "W": wl.W, "b": wl.b, "eps": wl.eps,
                   "comm_interval": wl.comm_interval, "fanout": wl.fanout, "parzen": 0 if args.no_parzen else 1,
                   "partial_rows": args.partial_rows, "mode": "free-running",
                   "steps_per_worker_per_bench_step": steps, "parallelism": "dp%d" % world,
                   "l2": "inputs larger than L2 (%.2f GB per pass)" % (bytes_per_launch / 1e9)},
        "roofline": roofline, "cpu_baseline": None, "e2e": None, "gpu_launches": int(launches), "clocks": clocks,
        "quantization_error_worker0": E_final, "quantization_error_mean_state": E_mean,
        "generator_centre_error_worker0": centre_err, "messages": msgs, "messages_over_passes": args.warmup + args.steps,
    }
    if keep:
        return line, (ctx, cfg, X, w0, steps, samples_per_pass)
    ctx.destroy()
    del ctx, X
    torch.cuda.empty_cache()
    return line, None


# workloads other than the headline one: (name, overrides) in the order of the table they make
OTHER_WORKLOADS = [("mid", {})] + \
    [("sweep", {"W": W, "comm_interval": c}) for W in (148, 296, 592, 1184, 2368) for c in (1, 10, 100)] + \
    [("dense", {}), ("codebook", {})]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="stream")
    ap.add_argument("--all-workloads", action="store_true",
                    help="one line per other workload (mid, the W x c grid of sweep, dense, codebook) instead of the headline line")
    ap.add_argument("--rows", type=int, default=0, help="use only the first ROWS rows (profiling of a small case)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--reference-rows", type=int, default=1 << 23)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    # points of the worker / communication sweep and the ablations (the defaults are the workload's own values)
    ap.add_argument("--workers", type=int, default=0, help="W")
    ap.add_argument("--comm-interval", type=int, default=-1, help="c; 0 = silent (no puts)")
    ap.add_argument("--no-parzen", action="store_true", help="accept every non-empty message (Eq. 3 without Eq. 4)")
    ap.add_argument("--partial-rows", type=int, default=0, help="centre rows per message (Section 4.4); 0 = whole state")
    ap.add_argument("--dist-path", type=int, default=0, help="ASGD_PATH_* (0 = the library's choice)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import paper_1505_04956_b200 as pkg
    from paper_1505_04956_b200 import dist, inputs

    args.warmup = max(args.warmup, 3)
    rank, world, local = dist.init_from_env(backend="nccl")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    pkg.load()

    if args.all_workloads:
        for name, over in OTHER_WORKLOADS:
            line, _ = measure(args, inputs.WORKLOADS[name].scaled(**over), dev, rank, world, dist)
            if rank == 0:
                print(json.dumps(line), flush=True)
        dist.shutdown()
        return 0

    wl = inputs.WORKLOADS[args.workload]
    if args.rows:
        wl = wl.scaled(N=args.rows)
    if args.workers:
        wl = wl.scaled(W=args.workers)
    if args.comm_interval >= 0:
        wl = wl.scaled(comm_interval=args.comm_interval)
    line, (ctx, cfg, X, w0, steps, samples_per_pass) = measure(args, wl, dev, rank, world, dist, keep=True)

    # end to end through the host-buffer entry point: H2D of X and w0, the pass, D2H of w^1
    e2e = None
    if not args.no_e2e:
        try:
            path = ctx.path_name()
            ctx.destroy()
            del ctx
            Xh = torch.empty(X.shape, dtype=torch.float32, pin_memory=True)
            Xh.copy_(X)
            w0h = w0.cpu().pin_memory()
            del X
            torch.cuda.empty_cache()
            out = torch.empty((wl.k, wl.d), dtype=torch.float32).pin_memory()
            scratch = torch.empty(pkg.asgd_fit_host_bytes(cfg) + 256, dtype=torch.uint8, device=dev)
            off = (-scratch.data_ptr()) % 256
            pkg.asgd_fit_host(cfg, Xh, w0h, steps, True, out, scratch[off:])       # warm-up
            dist.barrier()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(args.e2e_steps):
                pkg.asgd_fit_host(cfg, Xh, w0h, steps, True, out, scratch[off:])   # synchronises itself
            dt = dist.max_over_ranks(time.perf_counter() - t0)
            e2e = {"value": world * samples_per_pass * args.e2e_steps / dt, "unit": UNIT,
                   "h2d_bytes_per_step": int(Xh.numel() * 4 + w0h.numel() * 4), "d2h_bytes_per_step": int(out.numel() * 4),
                   "steps": args.e2e_steps, "path": path}
            del scratch, Xh
        except Exception as exc:      # e.g. not enough pinned host memory on this machine
            e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0, "error": repr(exc)[:200]}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, desc, th = cpu_baseline(wl, CPU_SAMPLE_ROWS, min_seconds=2.0)
        v1, desc1, _ = cpu_baseline(wl, CPU_SAMPLE_ROWS_ONE_CORE, threads=1, min_seconds=2.0)
        cpu = {"value": v, "unit": UNIT, "cores": th, "kind": "oracle", "sample": desc,
               "single_core": {"value": v1, "unit": UNIT, "cores": 1, "sample": desc1}}

    if rank == 0:
        line["e2e"] = e2e
        line["cpu_baseline"] = cpu
        print(json.dumps(line), flush=True)
    dist.shutdown()
    return 0


if __name__ == "__main__":
    sys.exit(main())
