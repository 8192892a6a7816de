#!/usr/bin/env python
"""Benchmark of the GAF filter-accumulate hot path (Algorithm 1 + Eq. 5).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one whole gaf_filter_accumulate call over one batch of K synthetic
micro-gradients (seed, K-1 cosine-distance tests, accepts, final division).
The default workload is configuration 2 (ResNet18-sized gradients, D=11,227,812
fp32, K=4, tau=0.97).  The path does not shard, so N > 1 runs N independent
replicas, one per GPU (no collective on the data path); time is the max over
ranks and the value is the aggregate over all replicas.

Rank 0 prints ONE JSON line.  `value` is micro-gradient GB/s: bytes of input
gradients consumed per second (K * elem_bytes * D per step), inputs resident in
HBM.  `roofline` reports the HBM bytes the schedule must move (by its byte model,
for the accept mask actually obtained) per second against the measured copy
bandwidth of the box.  `e2e` is the same metric through the host-buffer entry
point, pinned host memory in, results back to the host, copies inside the timed
region.  `cpu_baseline` is the fp64 CPU oracle timed on the host cores.
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
sys.path.insert(0, ROOT)

METRIC = "gaf_filter_accumulate micro-gradient GB/s"
UNIT = "GB/s"
N_SETS = 4                       # rotating input sets: each step's inputs are cold in L2
SCHED_NAMES = {0: "auto", 1: "stepwise", 2: "gram-first, two launches", 3: "gram-first, one launch"}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", type=int, default=2, choices=[1, 2, 3, 4, 5],
                    help="named configuration (2 is the one the metric is quoted on; 3 times the "
                         "pairwise cosine-distance matrix instead of the filter)")
    ap.add_argument("--D", type=int, default=None,
                    help="shorter vectors of the same recipe (for profiler captures, which must stay small); "
                         "the line then says so in config.workload")
    ap.add_argument("--K", type=int, default=None, help="pairwise workload only: another number of gradients")
    ap.add_argument("--fp32", action="store_true", help="pairwise workload only: binary32 inputs (same recipe)")
    ap.add_argument("--tau", type=float, default=0.97)
    ap.add_argument("--schedule", type=int, default=0, choices=[0, 1, 2, 3],
                    help="0 auto, 1 stepwise (streaming), 2 Gram-first in two launches, 3 Gram-first in one launch")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def schedule_bytes(mask_in_order, K, D, b):
    """HBM bytes the fused streaming schedule moves for a given accept pattern:
    pass 0 reads the seed and candidate 1 and writes the running sum; pass t reads
    the running sum and candidate t+1, plus gradient t and a write-back when t was
    accepted; the last pass reads the running sum (plus the last gradient if
    accepted) and writes g/c."""
    if K == 1:
        return (b + 4) * D
    a = [int(x) for x in mask_in_order]          # a[t] for t = 1..K-1 at index t
    total = 2 * b + 4
    for t in range(1, K - 1):
        total += 4 + b + a[t] * (b + 4)
    total += 8 + a[K - 1] * b
    return total * D


def gram_first_bytes(mask_in_order, K, D, b):
    """HBM bytes of the Gram-first schedule: every gradient once for the Gram matrix,
    the c accepted ones once more for the mean, and the output."""
    if K == 1:
        return (b + 4) * D
    c = sum(int(x) for x in mask_in_order)
    return ((K + c) * b + 4) * D


# DRAM traffic (dram__bytes_read + dram__bytes_write) of one launch of gram_fused_kernel<float,4> at
# configuration 2, by accepted count c, from the ncu capture summarised in
# profiles/gram_fused_config2.md.  Reported only while the kernel sources are the ones that were
# profiled (their hash is checked); otherwise `traffic` is null.
NCU_TRAFFIC = {
    "sources": ["paper_2412_18052_b200/csrc/gaf_fused.cuh", "paper_2412_18052_b200/csrc/gaf_gramfilter.cuh",
                "paper_2412_18052_b200/csrc/gaf_device.cuh"],
    "sha256": "95da4a45db5cb622e2e63d7a7459a62206988c0c94e13d4d291f5692fde26e74",
    "gram_fused_kernel<float,4>": {2: 234.2e6, 3: 261.9e6},
}


def kernel_sources_hash():
    import hashlib
    h = hashlib.sha256()
    for rel in NCU_TRAFFIC["sources"]:
        with open(os.path.join(ROOT, rel), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def ncu_traffic_config2(masks, n_sets, steps):
    """Average DRAM bytes per launch over the rotating input sets, or None."""
    if kernel_sources_hash() != NCU_TRAFFIC["sha256"]:
        return None
    table = NCU_TRAFFIC["gram_fused_kernel<float,4>"]
    per_set = []
    for m in masks:
        c = sum(int(x) for x in m)
        if c not in table:
            return None
        per_set.append(table[c])
    return sum(per_set[i % n_sets] for i in range(steps)) / steps


# ---------------------------------------------------------------- clocks -----

class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the
    timed region runs."""

    def __init__(self, index: int, period: float = 0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def sample(self):
        nv = self.nv
        self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
        bits = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
        for name, bit in (("hw_slowdown", nv.nvmlClocksEventReasonHwSlowdown),
                          ("hw_thermal_slowdown", nv.nvmlClocksEventReasonHwThermalSlowdown),
                          ("sw_thermal_slowdown", nv.nvmlClocksEventReasonSwThermalSlowdown),
                          ("sw_power_cap", nv.nvmlClocksEventReasonSwPowerCap),
                          ("hw_power_brake", nv.nvmlClocksEventReasonHwPowerBrakeSlowdown)):
            if bits & bit:
                self.reasons.add(name)

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            try:
                self.sample()
            except Exception:
                break
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        if self.ok and not self.samples:
            try:
                self.sample()
            except Exception:
                pass
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ---------------------------------------------------------- CPU oracle leg ---

def time_oracle(cfg: int, tau: float, seconds: float):
    """The fp64 CPU oracle, as it stands, on the same workload (single thread)."""
    import numpy as np  # noqa: F401
    from oracle import gaf_oracle as orc
    from paper_2412_18052_b200 import workloads

    if cfg == 3:
        cfg = 2                     # the reference arm times the filter; 3 is the pairwise matrix
    full = {1: 1_000_000, 2: workloads.RESNET18_100_NUMEL, 4: workloads.GPT2_SMALL_NUMEL,
            5: 1_000_000_000}[cfg]
    # configurations 4 and 5 are sampled at reduced D (same recipe) to bound the run
    D = full if cfg in (1, 2) else min(full, 32_000_000)
    w = workloads.config(cfg, device="cpu", D=None if D == full else D)
    grads = [workloads.as_numpy_bits(g) for g in w.grads]
    orc.filter_accumulate(grads, tau)                                  # warm (page in, compile)
    t0 = time.perf_counter()
    reps = 0
    while True:
        orc.filter_accumulate(grads, tau)
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= seconds or reps >= 10_000:
            break
    per_call = dt / reps
    gbs = w.K * w.elem_bytes * w.D / per_call / 1e9
    sample = (f"configuration {cfg} recipe, K={w.K}, D={w.D:,} {w.dtype}"
              f"{'' if D == full else ' (reduced from D=%d)' % full}, whole call repeated {reps}x "
              f"({dt:.1f} s of CPU work)")
    return gbs, per_call, sample


def workload_label(cfg, K, D, dtype, tau):
    return (f"configuration {cfg}: K={K}, D={D}, {dtype} inputs, tau={tau}, shared+private Gaussian mixture" +
            (" with ResNet18 per-tensor scales" if cfg == 2 else ""))


def run_reference(args):
    """Reference arm: the CPU oracle as it stands, one thread, W warm-up + K timed steps.
    A step is one whole oracle call on a bounded sample of the workload: the same recipe at a
    D chosen so that the run ends within about two minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import gaf_oracle as orc
    from paper_2412_18052_b200 import workloads

    cfg = 2 if args.workload == 3 else args.workload
    full = {1: 1_000_000, 2: workloads.RESNET18_100_NUMEL, 4: workloads.GPT2_SMALL_NUMEL, 5: 1_000_000_000}[cfg]
    K = {1: 4, 2: 4, 4: 8, 5: 8}[cfg]
    b = 2 if cfg == 5 else 4
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    # about 2.2 GB/s of gradient bytes on one core: size the sample for ~100 s in all
    budget_s = 100.0
    d_fit = int(budget_s / (steps + warmup) * 2.0e9 / (K * b))
    D = max(50_000, min(full, d_fit))
    w = workloads.config(cfg, device="cpu", D=None if D == full else D)
    grads = [workloads.as_numpy_bits(g) for g in w.grads]
    for _ in range(warmup):
        orc.filter_accumulate(grads, args.tau)
    t0 = time.perf_counter()
    for _ in range(steps):
        orc.filter_accumulate(grads, args.tau)
    dt = time.perf_counter() - t0
    per_call = dt / steps
    gbs = w.K * w.elem_bytes * w.D / per_call / 1e9
    sample = (f"configuration {cfg} recipe, K={w.K}, D={w.D:,} {w.dtype}"
              f"{'' if D == full else ' (reduced from D=%d)' % full}, one oracle call per step, "
              f"{steps} steps, {dt:.1f} s of CPU work")
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": per_call * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": workload_label(cfg, K, full, w.dtype, args.tau), "K": K, "D": full,
                   "input_dtype": w.dtype, "tau": args.tau, "sample_D": w.D},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------- replicas over ranks --

def max_over_ranks(value: float, device: str = "cpu") -> float:
    """The slowest rank sets the time of a multi-replica run (MAX all-reduce; works with the
    gloo backend on CPU tensors and with nccl on CUDA tensors)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_gbs(world: int, bytes_per_replica_step: float, ms_per_step: float) -> float:
    """Whole-job rate of `world` independent replicas that all took `ms_per_step`."""
    return world * bytes_per_replica_step / (ms_per_step * 1e-3) / 1e9


# ------------------------------------------------------------------ ours -----

def run_pairwise(args):
    """Configuration 3: the K x K pairwise cosine-distance matrix (one GPU)."""
    import torch

    import paper_2412_18052_b200 as gaf
    from paper_2412_18052_b200 import workloads

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(0)
    w = workloads.config(3, device="cuda:0", K=args.K, D=args.D)
    named = args.K is None and args.D is None and not args.fp32
    if args.fp32:
        w = workloads.mixture(w.K, w.D, "f32", w.rho, w.seed, device="cuda:0")
    K, D, b = w.K, w.D, w.elem_bytes
    ws = gaf.new_workspace(K, D, gaf.GAF_F32 if args.fp32 else gaf.GAF_BF16, device="cuda:0")
    dist_out = torch.empty(K, K, dtype=torch.float32, device="cuda:0")
    gram = torch.empty(K, K, dtype=torch.float64, device="cuda:0")

    def step():
        gaf.gaf_pairwise_cosdist(w.grads, ws, dist_out=dist_out, gram_out=gram)

    for _ in range(max(3, args.warmup)):
        step()
    launches = gaf.gaf_last_launch_count()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1) / args.steps
    in_bytes = K * b * D
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_kind = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_kind = 6650.0, "fallback"
    achieved = in_bytes / (ms * 1e-3) / 1e9
    line = {
        "metric": "gaf_pairwise_cosdist micro-gradient GB/s", "value": achieved, "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 products, f64 sums" if (args.fp32 or K > 32) else "bf16 x bf16 -> f32 (tensor cores), f64 sums",
        "data": "synthetic",
        "config": {"workload": f"configuration 3: pairwise matrix, K={K}, D={D}, {w.dtype} inputs" +
                               ("" if named else " (NOT the named configuration: size or type overridden)"),
                   "K": K, "D": D,
                   "l2": f"inputs of one call ({in_bytes / 1e6:.0f} MB) exceed the 126 MB L2"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": None, "peak_kind": f"of {peak_kind}",
                     "kernel": ("gram_tc_kernel" if (not args.fp32 and 8 < K <= 32) else
                                "gram_panel_kernel" if K > 8 else "gram_small_kernel") + " + finishing (whole call)",
                     "byte_model": "every gradient read once: K b D", "algorithmic_bytes_per_launch": in_bytes},
        "e2e": None, "gpu_launches": launches * args.steps, "clocks": clocks, "cpu_baseline": None,
    }
    print(json.dumps(line), flush=True)


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2412_18052_b200 as gaf
    from paper_2412_18052_b200 import workloads

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    cfg = args.workload
    n_sets = N_SETS if cfg in (1, 2) else (2 if cfg == 4 else 1)
    sets = [workloads.config(cfg, device=dev, seed=(cfg - 1) + 1000 * i + 17 * rank, D=args.D)
            for i in range(n_sets)]
    w0 = sets[0]
    K, D, b = w0.K, w0.D, w0.elem_bytes
    dtype_code = gaf.GAF_F32 if w0.dtype == "f32" else gaf.GAF_BF16
    ws = gaf.new_workspace(K, D, dtype_code, device=dev)
    macro = torch.empty(D, dtype=torch.float32, device=dev)
    mask = torch.empty(K, dtype=torch.uint8, device=dev)
    dist_out = torch.empty(K, dtype=torch.float32, device=dev)
    count = torch.empty(1, dtype=torch.int32, device=dev)

    def step(i):
        gaf.gaf_filter_accumulate(sets[i % n_sets].grads, args.tau, ws, macro_out=macro, mask_out=mask,
                                  dist_out=dist_out, count_out=count, schedule=args.schedule)

    # which schedule runs (the library says what its own choice was) and its byte model
    step(0)
    sched_used = gaf.gaf_last_schedule()
    model = gram_first_bytes if sched_used in (2, 3) else schedule_bytes
    # accept pattern and byte model per input set (also a warm-up)
    masks, bytes_per_set, launches_per_step = [], [], 0
    for i in range(n_sets):
        step(i)
        launches_per_step = gaf.gaf_last_launch_count()
        torch.cuda.synchronize()
        m = mask.cpu().tolist()
        masks.append(m)
        bytes_per_set.append(model(m, K, D, b))
    for i in range(max(3, args.warmup)):
        step(i)
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()

    steps = args.steps
    sampler = ClockSampler(local)
    barrier()
    torch.cuda.synchronize()
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for i in range(steps):
        step(i)
    ev1.record()
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    elapsed_ms = max_over_ranks(ev0.elapsed_time(ev1), dev)
    ms_per_step = elapsed_ms / steps
    grad_bytes = K * b * D
    value = aggregate_gbs(world, grad_bytes, ms_per_step)

    # dominant kernel, timed per launch with events on the launching stream
    n_launch_timed = min(steps, 200)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
           for _ in range(n_launch_timed)]
    for i, (a, z) in enumerate(evs):
        a.record(); step(i); z.record()
    torch.cuda.synchronize()
    launch_ms = [a.elapsed_time(z) for a, z in evs]
    avg_launch_ms = sum(launch_ms) / len(launch_ms)
    avg_bytes = sum(bytes_per_set[i % n_sets] for i in range(n_launch_timed)) / n_launch_timed

    # "warm" figure for the configurations that partly live in L2: the same input set every call
    warm = None
    if n_sets > 1 and cfg in (1, 2):
        n_warm = min(steps, 500)
        for _ in range(5):
            step(0)
        wev0, wev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        wev0.record()
        for _ in range(n_warm):
            step(0)
        wev1.record()
        torch.cuda.synchronize()
        warm_ms = wev0.elapsed_time(wev1) / n_warm
        warm = {"ms_per_step": warm_ms, "value": grad_bytes / (warm_ms * 1e-3) / 1e9, "unit": UNIT, "steps": n_warm,
                "note": "one input set repeated: whatever of it fits stays in L2 between calls; not the headline"}

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_kind = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_kind = 6650.0, "fallback"
    # Roofline figure: algorithmic bytes per call over the average duration of a call inside the timed
    # region (events on the launching stream around the K back-to-back calls).  With the one-launch
    # schedule a call IS one kernel launch.  The same ratio from one event pair per call is kept beside
    # it: it also contains the event records' own gaps.
    region_bytes = sum(bytes_per_set[i % n_sets] for i in range(steps)) / steps
    achieved = region_bytes / (ms_per_step * 1e-3) / 1e9
    per_call_events = avg_bytes / (avg_launch_ms * 1e-3) / 1e9

    # end to end through the host-buffer entry point
    e2e = None
    if args.e2e_steps > 0:
        n_e2e = args.e2e_steps
        host_sets = [[g.cpu().pin_memory() for g in s.grads] for s in sets[:2]]
        staging = torch.empty(gaf.gaf_host_staging_bytes(K, D, dtype_code), dtype=torch.uint8, device=dev)
        macro_h = torch.empty(D, dtype=torch.float32).pin_memory()
        mask_h = torch.empty(K, dtype=torch.uint8).pin_memory()
        dist_h = torch.empty(K, dtype=torch.float32).pin_memory()
        count_h = torch.empty(1, dtype=torch.int32).pin_memory()

        def e2e_step(i):
            gaf.gaf_filter_accumulate_host(host_sets[i % len(host_sets)], args.tau, staging, ws, macro_h,
                                           mask_h, dist_h, count_h, schedule=args.schedule)
        for i in range(2):
            e2e_step(i)
        barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(n_e2e):
            e2e_step(i)                       # synchronises the stream itself
        torch.cuda.synchronize()
        dt = max_over_ranks(time.perf_counter() - t0, dev)
        e2e = {"value": aggregate_gbs(world, grad_bytes, dt / n_e2e * 1e3), "unit": UNIT,
               "h2d_bytes_per_step": grad_bytes, "d2h_bytes_per_step": 4 * D + K + 4 * K + 4,
               "steps": n_e2e}

    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            gbs, per_call, sample = time_oracle(cfg, args.tau, args.cpu_seconds)
            cpu = {"value": gbs, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {
                "workload": workload_label(cfg, K, D, w0.dtype, args.tau) +
                            (" (REDUCED length, not the named configuration)" if args.D else ""),
                "K": K, "D": D, "input_dtype": w0.dtype, "tau": args.tau,
                "schedule": SCHED_NAMES[args.schedule] +
                            (" -> " + SCHED_NAMES[sched_used] if not args.schedule else ""),
                "parallelism": "replicas only (the path does not shard)" if world > 1 else "1 GPU",
                "l2": f"{n_sets} rotating input sets of {grad_bytes / 1e6:.0f} MB each (inputs of a step "
                      f"exceed the 126 MB L2 and were last touched {n_sets - 1} steps earlier)"
                      if n_sets > 1 else f"inputs of one step ({grad_bytes / 1e9:.1f} GB) exceed L2",
                "accept_masks": masks,
            },
            "roofline": {
                "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "frac_of_nominal_8000": achieved / 8000.0,
                "traffic": (ncu_traffic_config2(masks, n_sets, steps)
                            if (cfg == 2 and sched_used == 3 and abs(args.tau - 0.97) < 1e-12) else None),
                "peak_kind": f"of {peak_kind}",
                "kernel": {3: "gram_fused_kernel (the whole call is this one launch)",
                           2: "Gram kernel + masked_mean_kernel (whole call, both HBM-streaming)",
                           1: "step_kernel x%d (whole call)" % launches_per_step}[sched_used],
                "byte_model": ("Gram-first: ((K + c) b + 4) D" if sched_used in (2, 3)
                               else "streaming: (2b+4) + sum_t [4 + b + a_t (b+4)] + 8 + a_last b, times D"),
                "algorithmic_bytes_per_launch": region_bytes, "avg_launch_ms": ms_per_step,
                "launches_per_call": launches_per_step,
                "per_call_event_pairs": {"achieved": per_call_events, "frac": per_call_events / peak,
                                         "avg_call_ms": avg_launch_ms, "calls": n_launch_timed},
                "min_bytes_per_step": (K * b + 4) * D,
            },
            "e2e": e2e,
            "warm_l2": warm,
            "gpu_launches": launches_per_step * steps,
            "clocks": clocks,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == 3:
        if int(os.environ.get("RANK", "0")) == 0:
            run_pairwise(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
