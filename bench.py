#!/usr/bin/env python
"""Benchmark of the GAF filter-accumulate hot path (Algorithm 1 + Eq. 5).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one whole gaf_filter_accumulate call over one batch of K synthetic
micro-gradients (seed, K-1 cosine-distance tests, accepts, final division).
The headline workload is configuration 2 (ResNet18-sized gradients, D=11,227,812
fp32, K=4, tau=0.97).  The path does not shard, so N > 1 runs N independent
replicas, one per GPU (no collective on the data path); time is the max over
ranks and the value is the aggregate over all replicas.

Rank 0 prints ONE JSON line.  `value` is micro-gradient GB/s: bytes of input
gradients consumed per second (K * elem_bytes * D per step), inputs resident in
HBM.  Three byte counts are set against the measured copy bandwidth of the box,
each under its own name in `roofline`:
  dram_frac       bytes that really crossed HBM (ncu dram__bytes_read + dram__bytes_write of the
                  kernels as committed, per launch) / time / peak -- the HBM utilisation;
  min_bytes_frac  (K b + 4) D, every input read once and the output written once, / time / peak
                  -- what any schedule must move at least;
  model_frac      the bytes the schedule that ran asks of the memory system by its own byte model
                  (part of which shared memory and L2 serve), / time / peak -- an effective rate.
`roofline.frac` is dram_frac where the DRAM traffic of the kernels is on record, else
min_bytes_frac; `roofline.basis` says which.  At N = 1 the same line carries a `configs` block with
the other named configurations (1, 3, 4, 5), a few calls each.  `e2e` is the same metric through
the host-buffer entry point, pinned host memory in, results back to the host, copies inside the
timed region.  `cpu_baseline` is the fp64 CPU oracle timed on the host cores (one thread, and all
cores).
"""
from __future__ import annotations

import argparse
import gc
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
SCHED_NAMES = {0: "auto", 1: "stepwise", 2: "gram-first, two launches", 3: "gram-first, one launch"}
L2_BYTES = 126e6
RAMP_SECONDS = 0.3               # back-to-back calls issued right up to every timed region
FULL_D = {1: 1_000_000, 2: 11_227_812, 3: 11_227_812, 4: 124_439_808, 5: 1_000_000_000}
CONFIG_K = {1: 4, 2: 4, 3: 32, 4: 8, 5: 8}
CONFIG_B = {1: 4, 2: 4, 3: 2, 4: 4, 5: 2}
# rotating input sets per configuration: inputs of a call were last touched n_sets - 1 calls earlier,
# and all sets together exceed L2 (configuration 1: 12 x 16 MB), so every call starts cold in L2
N_SETS = {1: 12, 2: 4, 4: 2, 5: 1}
# calls timed for the entries of the `configs` block
BLOCK_STEPS = {1: 1000, 3: 300, 4: 100, 5: 60}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", type=int, default=2, choices=[1, 2, 3, 4, 5],
                    help="named configuration of the headline line (2 is the one the metric is quoted on; "
                         "3 times the pairwise cosine-distance matrix instead of the filter)")
    ap.add_argument("--D", type=int, default=None,
                    help="shorter vectors of the same recipe (for profiler captures, which must stay small); "
                         "the line then says so in config.workload")
    ap.add_argument("--K", type=int, default=None, help="pairwise workload only: another number of gradients")
    ap.add_argument("--fp32", action="store_true", help="pairwise workload only: binary32 inputs (same recipe)")
    ap.add_argument("--separate", action="store_true",
                    help="pairwise workload only: K separate allocations instead of the rows of one matrix")
    ap.add_argument("--two-gradients", action="store_true",
                    help="instead of a named configuration: the filter on two fp32 gradients of configuration 2's "
                         "recipe (the setting of the paper's experiments); --D for another length")
    ap.add_argument("--tau", type=float, default=0.97)
    ap.add_argument("--schedule", type=int, default=0, choices=[0, 1, 2, 3],
                    help="0 auto, 1 stepwise (streaming), 2 Gram-first in two launches, 3 Gram-first in one launch")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sets", type=int, default=None,
                    help="number of rotating input sets of the headline workload (profiler captures: fewer sets, "
                         "less device memory)")
    ap.add_argument("--no-configs", action="store_true",
                    help="leave out the `configs` block (the other named configurations)")
    return ap.parse_args()


# ------------------------------------------------------------ byte models -----

def schedule_bytes(mask_in_order, K, D, b):
    """HBM bytes the fused streaming schedule asks for, for a given accept pattern:
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
    """Bytes of the Gram-first schedule: every gradient once for the Gram matrix,
    the c accepted ones once more for the mean, and the output."""
    if K == 1:
        return (b + 4) * D
    c = sum(int(x) for x in mask_in_order)
    return ((K + c) * b + 4) * D


def min_bytes(K, D, b):
    """What any schedule moves at least: every input once, the output once."""
    return (K * b + 4) * D


# DRAM traffic (ncu dram__bytes_read.sum + dram__bytes_write.sum per launch, summed over the launches of a
# call) of the kernels as committed, from the captures that the summaries in the profiler folder of this
# repository describe.  Bytes per element index, by accepted count c.  Two captures per entry where they differ:
#   "steady"   caches left as the previous call left them (ncu --cache-control none): what crosses HBM while
#              calls run back to back, as they do in the timed region -- this is `traffic`;
#   "flushed"  ncu's default, caches flushed before every launch: a call that starts with a cold L2.
# At configuration 2 they differ: back to back, about 32 MB of L2 hold the previous call's output (dirty lines
# that the next call overwrites in place, so they never reach HBM) and fewer of the second pass's re-reads hit.
# Captures on a shorter vector of the same recipe scale in proportion (both passes stream; inputs far beyond
# L2).  An entry is used only while the listed kernel sources hash to what was profiled; otherwise null.
NCU_TRAFFIC = {
    # gram_fused_kernel<float,4> at configuration 2 itself (D = 11,227,812)
    (2, 3): {"sources": ["gaf_fused.cuh", "gaf_gramfilter.cuh", "gaf_device.cuh"],
             "sha256": "c818aa29bb0ab3cfd20979d4de48b461b64f5638d0d403cbeae6950f4970cd2f",
             "steady": {2: 262.6e6 / 11227812, 3: 296.4e6 / 11227812},
             "flushed": {2: 230.3e6 / 11227812, 3: 257.8e6 / 11227812}},
    # gram_small_kernel<float,8> + masked_mean_kernel<float>, captured at D = 80,000,000
    (4, 2): {"sources": ["gaf_gramfilter.cuh", "gaf_device.cuh"],
             "sha256": "707df4a1adb38d5c23a4b0a9334cb7ee98408cb34984959ae16d9bc13231b65d",
             "steady": {4: (2563.4e6 + 1573.5e6) / 80e6, 1: (2563.9e6 + 591.2e6) / 80e6}},
    # gram_mma_kernel<8> + masked_mean_kernel<bf16>, captured at D = 100,000,000
    (5, 2): {"sources": ["gaf_gram_mma.cuh", "gaf_gramfilter.cuh", "gaf_device.cuh"],
             "sha256": "9e4d0496b3660411997f70119a65ea597629d6649e27b79cad70329530722984",
             "steady": {4: (1604.5e6 + 1169.0e6) / 100e6}},
}


def kernel_sources_hash(names):
    import hashlib
    h = hashlib.sha256()
    for name in names:
        with open(os.path.join(ROOT, "paper_2412_18052_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def ncu_traffic(cfg, sched_used, masks, D, n_sets, steps, which="steady"):
    """Average DRAM bytes per call over the rotating input sets, or None when no capture of the
    committed kernels is on record for this configuration and schedule."""
    entry = NCU_TRAFFIC.get((cfg, sched_used))
    if not entry or kernel_sources_hash(entry["sources"]) != entry["sha256"]:
        return None
    table = entry.get(which) or entry["steady"]
    per_set = []
    for m in masks:
        c = sum(int(x) for x in m)
        if c not in table:
            return None
        per_set.append(table[c] * D)
    return sum(per_set[i % n_sets] for i in range(steps)) / steps


def peak_bandwidth():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["hbm_gbs"]), "of measured"
    return 6650.0, "of fallback"


# ---------------------------------------------------------------- clocks -----

class Nvml:
    """NVML handle of one GPU, initialised once, before any warm-up (initialising it with the GPU
    idle right in front of a timed region costs the first calls of that region their clocks)."""

    REASONS = (("hw_slowdown", "nvmlClocksEventReasonHwSlowdown"),
               ("hw_thermal_slowdown", "nvmlClocksEventReasonHwThermalSlowdown"),
               ("sw_thermal_slowdown", "nvmlClocksEventReasonSwThermalSlowdown"),
               ("sw_power_cap", "nvmlClocksEventReasonSwPowerCap"),
               ("hw_power_brake", "nvmlClocksEventReasonHwPowerBrakeSlowdown"))

    def __init__(self, index: int):
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.max_mhz = None

    def read(self):
        """(SM MHz, set of active slowdown reasons)."""
        nv = self.nv
        mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
        bits = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
        return mhz, {name for name, attr in self.REASONS if bits & getattr(nv, attr)}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons while a timed region runs."""

    def __init__(self, nvml: Nvml, period: float = 0.005):
        super().__init__(daemon=True)
        self.nvml, self.period = nvml, period
        self.samples, self.reasons = [], set()
        self._stop_evt = threading.Event()

    def sample(self):
        if not self.nvml.ok:
            return
        try:
            mhz, reasons = self.nvml.read()
        except Exception:
            return
        self.samples.append(mhz)
        self.reasons |= reasons

    def run(self):
        while not self._stop_evt.is_set():
            self.sample()
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.nvml.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ---------------------------------------------------------- CPU oracle leg ---

def oracle_sample_workload(cfg):
    """The workload the CPU legs run: the named configuration, configurations 4 and 5 at a reduced
    D of the same recipe so that the run stays bounded."""
    from paper_2412_18052_b200 import workloads
    if cfg == 3:
        cfg = 2                     # the CPU legs time the filter; 3 is the pairwise matrix
    full = FULL_D[cfg]
    D = full if cfg in (1, 2) else min(full, 32_000_000)
    w = workloads.config(cfg, device="cpu", D=None if D == full else D)
    return cfg, full, w, [workloads.as_numpy_bits(g) for g in w.grads]


def time_oracle(cfg: int, tau: float, seconds: float):
    """The fp64 CPU oracle, as it stands, on the same workload: one thread, then the same loops split
    over all host cores by chunks of D."""
    from oracle import gaf_oracle as orc

    cfg, full, w, grads = oracle_sample_workload(cfg)
    gbytes = w.K * w.elem_bytes * w.D

    def run(fn, budget):
        fn()                                                       # warm (page in, compile)
        t0 = time.perf_counter()
        reps = 0
        while True:
            fn()
            reps += 1
            dt = time.perf_counter() - t0
            if dt >= budget or reps >= 10_000:
                break
        return gbytes / (dt / reps) / 1e9, reps, dt

    one, reps1, dt1 = run(lambda: orc.filter_accumulate(grads, tau), seconds)
    cores = orc.host_cores()
    many, repsn, dtn = run(lambda: orc.filter_accumulate_all_cores(grads, tau, n_threads=cores), seconds / 2)
    sample = (f"configuration {cfg} recipe, K={w.K}, D={w.D:,} {w.dtype}"
              f"{'' if w.D == full else ' (reduced from D=%d)' % full}, whole call repeated {reps1}x on one "
              f"thread ({dt1:.1f} s) and {repsn}x on {cores} threads ({dtn:.1f} s)")
    return {"value": one, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
            "all_cores": {"value": many, "unit": UNIT, "cores": cores,
                          "how": "the same loops, every pass over D cut into one chunk per thread, "
                                 "sums combined in chunk order"}}


def workload_label(cfg, K, D, dtype, tau):
    return (f"configuration {cfg}: K={K}, D={D}, {dtype} inputs, tau={tau}, shared+private Gaussian mixture" +
            (" with ResNet18 per-tensor scales" if cfg == 2 else ""))


def config_dict(cfg, K, D, dtype, tau, schedule, parallelism, l2, extra=None):
    """The `config` object: the same keys from both arms."""
    d = {"workload": workload_label(cfg, K, D, dtype, tau), "K": K, "D": D, "input_dtype": dtype, "tau": tau,
         "schedule": schedule, "parallelism": parallelism, "l2": l2}
    d.update(extra or {})
    return d


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
    full = FULL_D[cfg]
    K = CONFIG_K[cfg]
    b = CONFIG_B[cfg]
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    # about 2 GB/s of gradient bytes on one core: size the sample for ~100 s in all
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
        "config": config_dict(cfg, K, full, w.dtype, args.tau, "CPU oracle (Algorithm 1 as written, one thread)",
                              "host cores", f"each step runs on D={w.D} elements of the recipe",
                              {"accept_masks": None}),
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


# ------------------------------------------------------------- timing core ----

def timed_region(torch, step, steps, warmup, nvml, barrier=None, ramp_seconds=RAMP_SECONDS, n_pairs=None):
    """W warm-up calls, a ramp of back-to-back calls right up to the region, then exactly `steps`
    calls between two events on the launching stream, bracketed by barrier + synchronize.  Clocks are
    sampled while the region runs.  Afterwards the same calls once more with one event pair each,
    for the median.  Returns a dict."""
    for i in range(max(3, warmup)):
        step(i)
    torch.cuda.synchronize()
    # ramp: the first calls after an idle stretch run below the steady clocks
    ramp_calls, t0 = 0, time.perf_counter()
    while time.perf_counter() - t0 < ramp_seconds:
        for _ in range(16):
            step(ramp_calls)
            ramp_calls += 1
        if ramp_calls % 256 == 0:
            torch.cuda.synchronize()                 # bound the queue; the GPU stays busy to within one call
    sampler = ClockSampler(nvml)
    if barrier:
        barrier()
    torch.cuda.synchronize()
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for i in range(steps):
        step(i)
    ev1.record()
    sampler.sample()                                 # the queue is still draining: a sample under load
    torch.cuda.synchronize()
    if barrier:
        barrier()
    clocks = sampler.stop()
    ms_region = ev0.elapsed_time(ev1)
    # one event pair per call (the pairs' own gaps are part of what they measure)
    n_pairs = n_pairs or max(20, min(steps, 200))
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_pairs)]
    for i, (a, z) in enumerate(evs):
        a.record(); step(i); z.record()
    torch.cuda.synchronize()
    per_call = [a.elapsed_time(z) for a, z in evs]
    return {"ms_region": ms_region, "ms_per_step": ms_region / steps, "ramp_calls": ramp_calls,
            "clocks": clocks, "per_call_ms": per_call}


def fractions(ms, traffic, model_b, min_b, peak, traffic_flushed=None):
    """The three byte counts over one time, as GB/s and as fractions of `peak`."""
    def rate(nbytes):
        return None if nbytes is None else nbytes / (ms * 1e-3) / 1e9
    dram, model, least, cold = rate(traffic), rate(model_b), rate(min_b), rate(traffic_flushed)
    return {"dram_gbs": dram, "dram_frac": None if dram is None else dram / peak,
            "dram_frac_flushed_caches": None if cold is None else cold / peak,
            "model_gbs": model, "model_frac": model / peak,
            "min_bytes_gbs": least, "min_bytes_frac": least / peak}


def measure_filter(torch, gaf, workloads, cfg, dev, tau, schedule, steps, warmup, nvml, rank=0, D=None,
                   barrier=None, want_warm=False, want_c_loop=False, n_sets=None):
    """One named configuration of the filter on one GPU: timed region, byte counts, fractions."""
    n_sets = n_sets or N_SETS[cfg]
    sets = [workloads.config(cfg, device=dev, seed=(cfg - 1) + 1000 * i + 17 * rank, D=D) for i in range(n_sets)]
    w0 = sets[0]
    K, D, b = w0.K, w0.D, w0.elem_bytes
    dtype_code = gaf.GAF_F32 if w0.dtype == "f32" else gaf.GAF_BF16
    ws = gaf.new_workspace(K, D, dtype_code, device=dev)
    macro = torch.empty(D, dtype=torch.float32, device=dev)
    mask = torch.empty(K, dtype=torch.uint8, device=dev)
    dist_out = torch.empty(K, dtype=torch.float32, device=dev)
    count = torch.empty(1, dtype=torch.int32, device=dev)

    def step(i):
        gaf.gaf_filter_accumulate(sets[i % n_sets].grads, tau, ws, macro_out=macro, mask_out=mask,
                                  dist_out=dist_out, count_out=count, schedule=schedule)

    # which schedule runs (the library says what its own choice was), accept pattern per input set
    step(0)
    sched_used = gaf.gaf_last_schedule()
    model = gram_first_bytes if sched_used in (2, 3) else schedule_bytes
    masks, bytes_per_set, launches_per_step = [], [], 0
    for i in range(n_sets):
        step(i)
        launches_per_step = gaf.gaf_last_launch_count()
        torch.cuda.synchronize()
        m = mask.cpu().tolist()
        masks.append(m)
        bytes_per_set.append(model(m, K, D, b))
    status = gaf.gaf_read_status(ws)

    t = timed_region(torch, step, steps, warmup, nvml, barrier)
    grad_bytes = K * b * D
    model_b = sum(bytes_per_set[i % n_sets] for i in range(steps)) / steps
    out = {"K": K, "D": D, "b": b, "dtype": w0.dtype, "n_sets": n_sets, "grad_bytes": grad_bytes, "masks": masks,
           "sched_used": sched_used, "launches_per_step": launches_per_step, "status": status,
           "model_bytes": model_b, "min_bytes": min_bytes(K, D, b),
           "traffic": ncu_traffic(cfg, sched_used, masks, D, n_sets, steps) if abs(tau - 0.97) < 1e-12 else None,
           "traffic_flushed": (ncu_traffic(cfg, sched_used, masks, D, n_sets, steps, "flushed")
                               if abs(tau - 0.97) < 1e-12 else None),
           "timing": t, "sets": sets, "ws": ws, "outputs": (macro, mask, dist_out, count), "dtype_code": dtype_code}

    if want_warm:
        # the same input set every call: whatever of it fits stays in L2 between calls
        n_warm = min(max(steps, 200), 500)
        for _ in range(5):
            step(0)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(n_warm):
            step(0)
        e1.record()
        torch.cuda.synchronize()
        warm_ms = e0.elapsed_time(e1) / n_warm
        out["warm_l2"] = {"ms_per_step": warm_ms, "value": grad_bytes / (warm_ms * 1e-3) / 1e9, "unit": UNIT,
                          "steps": n_warm,
                          "note": "one input set repeated: whatever of it fits stays in L2 between calls; "
                                  "not the headline"}
    if want_c_loop:
        # the same calls issued by a loop in C inside the library: the interpreter's per-call cost is out
        n_c = max(steps, 1000)
        grads_sets = [s.grads for s in sets]
        gaf.gaf_filter_accumulate_repeat(200, grads_sets, tau, ws, macro, mask, dist_out, count, schedule=schedule)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        gaf.gaf_filter_accumulate_repeat(n_c, grads_sets, tau, ws, macro, mask, dist_out, count, schedule=schedule)
        e1.record()
        torch.cuda.synchronize()
        out["c_loop"] = {"ms_per_step": e0.elapsed_time(e1) / n_c, "steps": n_c,
                         "note": "the same calls from a loop in C (gaf_filter_accumulate_repeat)"}
    return out


def block_entry(m, peak, peak_kind, tau, schedule):
    """One entry of the `configs` block from a measure_filter result."""
    t = m["timing"]
    ms = t["ms_per_step"]
    fr = fractions(ms, m["traffic"], m["model_bytes"], m["min_bytes"], peak, m["traffic_flushed"])
    per_call = t["per_call_ms"]
    mhz = t["clocks"]["sm_mhz"]
    e = {"workload": workload_label(m["cfg"], m["K"], m["D"], m["dtype"], tau),
         "schedule": SCHED_NAMES[schedule] + (" -> " + SCHED_NAMES[m["sched_used"]] if not schedule else ""),
         "steps": m["steps"], "ramp_calls": t["ramp_calls"], "ms_per_call": ms,
         "ms_per_call_median_of_event_pairs": statistics.median(per_call), "event_pairs": len(per_call),
         "value": m["grad_bytes"] / (ms * 1e-3) / 1e9, "unit": UNIT,
         "launches_per_call": m["launches_per_step"], "accept_masks": m["masks"],
         "l2": f"{m['n_sets']} rotating input sets of {m['grad_bytes'] / 1e6:.0f} MB each"
               if m["n_sets"] > 1 else f"inputs of one call ({m['grad_bytes'] / 1e9:.1f} GB) exceed L2",
         "model_bytes_per_call": m["model_bytes"], "min_bytes_per_call": m["min_bytes"],
         "traffic": m["traffic"], "peak": peak, "peak_kind": peak_kind, "clocks": t["clocks"],
         "ms_x_sm_mhz": None if mhz is None else ms * mhz}
    e.update(fr)
    for key in ("warm_l2", "c_loop"):
        if key in m:
            e[key] = m[key]
    return e


def measure_pairwise(torch, gaf, workloads, dev, steps, warmup, nvml, K=None, D=None, fp32=False, stacked=True):
    """Configuration 3: the K x K pairwise cosine-distance matrix.  ``stacked``: the gradients are the rows of one
    matrix (row distance D rounded up to 128 elements: what an all-gather of padded flat micro-gradients leaves), which
    lets the tensor-memory kernel fetch them by tensor copies; otherwise K separate allocations."""
    w = workloads.config(3, device=dev, K=K, D=D, stacked=stacked)
    if fp32:
        w = workloads.mixture(w.K, w.D, "f32", w.rho, w.seed, device=dev, stacked=stacked)
    K, D, b = w.K, w.D, w.elem_bytes
    ws = gaf.new_workspace(K, D, gaf.GAF_F32 if fp32 else gaf.GAF_BF16, device=dev)
    dist_out = torch.empty(K, K, dtype=torch.float32, device=dev)
    gram = torch.empty(K, K, dtype=torch.float64, device=dev)

    def step(_i):
        gaf.gaf_pairwise_cosdist(w.grads, ws, dist_out=dist_out, gram_out=gram)

    step(0)
    launches = gaf.gaf_last_launch_count()
    loader = gaf.gaf_last_gram_loader()
    t = timed_region(torch, step, steps, warmup, nvml)
    return {"K": K, "D": D, "b": b, "dtype": w.dtype, "grad_bytes": K * b * D, "launches": launches, "timing": t,
            "placement": "rows of one matrix" if stacked else "separate allocations",
            "gram_loader": {0: None, 1: "16-byte asynchronous copies", 2: "tensor copies (TMA)"}[loader],
            "kernel": ("gram_tc_kernel" if (not fp32 and 16 < K <= 64) else
                       "gram_mma_wide_kernel" if (not fp32 and 8 < K <= 16) else
                       "gram_panel_kernel" if K > 8 else "gram_small_kernel") + " + finishing (whole call)"}


def measure_cosdist(torch, gaf, workloads, dev, D, steps, nvml, peak, peak_kind):
    """gaf_cosdist (Eq. 4 between two buffers) on two gradients of configuration 2's recipe at length D."""
    w = workloads.config(2 if D == FULL_D[2] else 4, device=dev, K=2, D=D)
    ws = gaf.new_workspace(2, D, gaf.GAF_F32, device=dev)
    dist_out = torch.empty(1, dtype=torch.float32, device=dev)
    stats = torch.empty(3, dtype=torch.float64, device=dev)
    n_sets = 4 if 2 * 4 * D * 4 < 4e9 else 1
    pairs = [w.grads] + [[g.clone() for g in w.grads] for _ in range(n_sets - 1)]

    def step(i):
        x, y = pairs[i % n_sets]
        gaf.gaf_cosdist(x, y, ws, dist_out=dist_out, stats_out=stats)

    t = timed_region(torch, step, steps, 5, nvml)
    ms = t["ms_per_step"]
    nbytes = 2 * 4 * D
    rate = nbytes / (ms * 1e-3) / 1e9
    return {"workload": f"gaf_cosdist, D={D}, f32 inputs ({n_sets} rotating pairs of {nbytes / 1e6:.0f} MB)",
            "op": "gaf_cosdist", "steps": steps, "ramp_calls": t["ramp_calls"], "ms_per_call": ms,
            "ms_per_call_median_of_event_pairs": statistics.median(t["per_call_ms"]), "value": rate, "unit": UNIT,
            "launches_per_call": 1, "min_bytes_per_call": nbytes, "model_bytes_per_call": nbytes,
            "byte_model": "both buffers read once: 2 b D (= the minimum)", "min_bytes_frac": rate / peak,
            "model_frac": rate / peak, "dram_frac": None, "traffic": None, "peak": peak, "peak_kind": peak_kind,
            "clocks": t["clocks"]}


def measure_two_gradients(torch, gaf, workloads, dev, D, steps, nvml, peak, peak_kind):
    """The filter on two fp32 micro-gradients (the setting of the paper's experiments, Section 4) of configuration 2's
    recipe at length D, four rotating input sets: a stream of calls that all accept the second gradient (tau = 2), one
    that all reject it (tau = 0), and one in which the outcome changes with every call."""
    n_sets = 4 if 3 * 4 * D * 4 < 6e9 else 1
    sets = [workloads.config(2 if D == FULL_D[2] else 4, device=dev, K=2, D=D, seed=1 + 1000 * i).grads
            for i in range(n_sets)]
    ws = gaf.new_workspace(2, D, gaf.GAF_F32, device=dev)
    macro, mask, dist, count = gaf.gaf_filter_accumulate(sets[0], 2.0, ws)
    min_b = (2 * 4 + 4) * D
    out = {"workload": f"gaf_filter_accumulate, K=2, D={D}, f32 inputs ({n_sets} rotating sets)",
           "op": "gaf_filter_accumulate", "unit": UNIT, "min_bytes_per_call": min_b,
           "byte_model": "both gradients read once, the output written once when the outcome of the latest two calls "
                         "repeats: (2 b + 4) D (= the minimum); two passes (16 D or 20 D) while outcomes alternate",
           "peak": peak, "peak_kind": peak_kind}
    for name, taus in (("all_accepted", (2.0,)), ("all_rejected", (0.0,)), ("alternating", (2.0, 0.0))):
        def step(i, taus=taus):
            gaf.gaf_filter_accumulate(sets[i % n_sets], taus[i % len(taus)], ws, macro_out=macro, mask_out=mask,
                                      dist_out=dist, count_out=count)
        step(0)
        launches = gaf.gaf_last_launch_count()
        t = timed_region(torch, step, steps, 5, nvml)
        ms = t["ms_per_step"]
        rate = min_b / (ms * 1e-3) / 1e9
        out[name] = {"steps": steps, "ms_per_call": ms, "launches_per_call": launches,
                     "ms_per_call_median_of_event_pairs": statistics.median(t["per_call_ms"]),
                     "value": 2 * 4 * D / (ms * 1e-3) / 1e9, "min_bytes_frac": rate / peak, "clocks": t["clocks"]}
    return out


def measure_variants(torch, gaf, workloads, dev, steps, nvml, peak, peak_kind):
    """The other forms of the filter at configuration 2 (K=4, D=11,227,812 fp32, tau 0.97, four rotating sets): the
    order-indifferent variant, the bucketed variant with ResNet18's 62 parameter tensors as buckets, and the
    streaming form (one call per arriving gradient)."""
    import numpy as np
    sets = [workloads.config(2, device=dev, seed=1 + 1000 * i).grads for i in range(4)]
    K, D = len(sets[0]), sets[0][0].numel()
    ws = gaf.new_workspace(K, D, gaf.GAF_F32, device=dev)
    macro = torch.empty(D, dtype=torch.float32, device=dev)
    bounds = [0] + [int(x) // 8 * 8 for x in np.cumsum(workloads.resnet18_tensor_sizes(100))[:-1]] + [D]
    bounds = sorted(set(bounds))
    min_b = (K * 4 + 4) * D

    def any_seed(i):
        gaf.gaf_filter_accumulate_any_seed(sets[i % 4], 0.97, ws, macro_out=macro)

    def bucketed(i):
        gaf.gaf_filter_accumulate_bucketed(sets[i % 4], 0.97, bounds, ws, macro_out=macro)

    def streaming(i):
        g = sets[i % 4]
        gaf.gaf_stream_begin(g[0], macro, ws)
        for t in range(1, K):
            gaf.gaf_stream_push(g[t], t, 0.97, macro, ws)
        gaf.gaf_stream_end(K, macro, ws)

    out = {"workload": f"configuration 2 recipe, K={K}, D={D}, f32 inputs (4 rotating sets)", "unit": UNIT,
           "min_bytes_per_call": min_b, "peak": peak, "peak_kind": peak_kind}
    for name, op, step in (("any_seed", "gaf_filter_accumulate_any_seed", any_seed),
                           ("bucketed", f"gaf_filter_accumulate_bucketed, {len(bounds) - 1} buckets", bucketed),
                           ("streaming", "gaf_stream_begin + 3 gaf_stream_push + gaf_stream_end", streaming)):
        t = timed_region(torch, step, steps, 5, nvml)
        ms = t["ms_per_step"]
        out[name] = {"op": op, "steps": steps, "ms_per_call": ms,
                     "ms_per_call_median_of_event_pairs": statistics.median(t["per_call_ms"]),
                     "value": K * 4 * D / (ms * 1e-3) / 1e9, "min_bytes_frac": min_b / (ms * 1e-3) / 1e9 / peak,
                     "clocks": t["clocks"]}
    return out


def pairwise_entry(m, peak, peak_kind, steps):
    t = m["timing"]
    ms = t["ms_per_step"]
    achieved = m["grad_bytes"] / (ms * 1e-3) / 1e9
    mhz = t["clocks"]["sm_mhz"]
    return {"workload": f"configuration 3: pairwise matrix, K={m['K']}, D={m['D']}, {m['dtype']} inputs",
            "op": "gaf_pairwise_cosdist", "steps": steps, "ramp_calls": t["ramp_calls"], "ms_per_call": ms,
            "ms_per_call_median_of_event_pairs": statistics.median(t["per_call_ms"]),
            "event_pairs": len(t["per_call_ms"]), "value": achieved, "unit": UNIT,
            "launches_per_call": m["launches"], "kernel": m["kernel"], "placement": m["placement"],
            "gram_loader": m["gram_loader"],
            "l2": f"inputs of one call ({m['grad_bytes'] / 1e6:.0f} MB) exceed the 126 MB L2",
            "model_bytes_per_call": m["grad_bytes"], "min_bytes_per_call": m["grad_bytes"],
            "byte_model": "every gradient read once: K b D (= the minimum)",
            "model_gbs": achieved, "model_frac": achieved / peak, "min_bytes_gbs": achieved,
            "min_bytes_frac": achieved / peak, "dram_gbs": None, "dram_frac": None, "traffic": None,
            "peak": peak, "peak_kind": peak_kind, "clocks": t["clocks"],
            "ms_x_sm_mhz": None if mhz is None else ms * mhz}


# ------------------------------------------------------------------ ours -----

def run_pairwise(args):
    """--workload 3: the pairwise matrix as the headline line (one GPU)."""
    import torch

    import paper_2412_18052_b200 as gaf
    from paper_2412_18052_b200 import workloads

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(0)
    nvml = Nvml(0)
    named = args.K is None and args.D is None and not args.fp32
    m = measure_pairwise(torch, gaf, workloads, "cuda:0", args.steps, args.warmup, nvml, K=args.K, D=args.D,
                         fp32=args.fp32, stacked=not args.separate)
    peak, peak_kind = peak_bandwidth()
    e = pairwise_entry(m, peak, peak_kind, args.steps)
    K = m["K"]
    line = {
        "metric": "gaf_pairwise_cosdist micro-gradient GB/s", "value": e["value"], "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": e["ms_per_call"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 products, f64 sums" if (args.fp32 or K > 64) else "bf16 x bf16 -> f32 (tensor cores), f64 sums",
        "data": "synthetic",
        "config": {"workload": e["workload"] + ("" if named else " (NOT the named configuration: size or type overridden)"),
                   "K": K, "D": m["D"], "l2": e["l2"], "placement": m["placement"], "gram_loader": m["gram_loader"]},
        "roofline": {"bound": "hbm", "achieved": e["value"], "peak": peak, "unit": "GB/s", "frac": e["value"] / peak,
                     "basis": "min_bytes (= byte model: every gradient read once)", "traffic": None,
                     "peak_kind": peak_kind, "kernel": m["kernel"], "algorithmic_bytes_per_launch": m["grad_bytes"],
                     "model_frac": e["model_frac"], "min_bytes_frac": e["min_bytes_frac"], "dram_frac": None},
        "ramp_calls": e["ramp_calls"], "ms_per_call_median_of_event_pairs": e["ms_per_call_median_of_event_pairs"],
        "e2e": None, "gpu_launches": m["launches"] * args.steps, "clocks": e["clocks"], "cpu_baseline": None,
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
    nvml = Nvml(local)                        # before any warm-up
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    def barrier():
        if world > 1:
            dist.barrier()

    cfg, steps = args.workload, args.steps
    peak, peak_kind = peak_bandwidth()
    m = measure_filter(torch, gaf, workloads, cfg, dev, args.tau, args.schedule, steps, args.warmup, nvml,
                       rank=rank, D=args.D, barrier=barrier, want_warm=cfg in (1, 2), want_c_loop=True,
                       n_sets=args.sets)
    t = m["timing"]
    K, D, b, grad_bytes = m["K"], m["D"], m["b"], m["grad_bytes"]
    ms_per_step = max_over_ranks(t["ms_region"], dev) / steps
    value = aggregate_gbs(world, grad_bytes, ms_per_step)
    fr = fractions(ms_per_step, m["traffic"], m["model_bytes"], m["min_bytes"], peak, m["traffic_flushed"])
    per_call = t["per_call_ms"]

    # end to end through the host-buffer entry point
    e2e = None
    if args.e2e_steps > 0:
        n_e2e = args.e2e_steps
        host_sets = [[g.cpu().pin_memory() for g in s.grads] for s in m["sets"][:2]]
        staging = torch.empty(gaf.gaf_host_staging_bytes(K, D, m["dtype_code"]), dtype=torch.uint8, device=dev)
        macro_h = torch.empty(D, dtype=torch.float32).pin_memory()
        mask_h = torch.empty(K, dtype=torch.uint8).pin_memory()
        dist_h = torch.empty(K, dtype=torch.float32).pin_memory()
        count_h = torch.empty(1, dtype=torch.int32).pin_memory()

        def e2e_step(i):
            gaf.gaf_filter_accumulate_host(host_sets[i % len(host_sets)], args.tau, staging, m["ws"], macro_h,
                                           mask_h, dist_h, count_h, schedule=args.schedule)
        for i in range(3):
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
        del host_sets, staging, macro_h, e2e_step

    # the other named configurations, a few calls each (one GPU, the default line only)
    block = None
    if world == 1 and cfg == 2 and args.D is None and not args.no_configs:
        sched_used_main = m["sched_used"]
        m_keep = {k: v for k, v in m.items() if k not in ("sets", "ws", "outputs")}
        del m
        gc.collect()
        torch.cuda.empty_cache()
        m = m_keep
        m["sched_used"] = sched_used_main
        block = {}
        for c in (1, 3, 4, 5):
            try:
                if c == 3:
                    r = measure_pairwise(torch, gaf, workloads, dev, BLOCK_STEPS[3], 5, nvml)
                    block["3"] = pairwise_entry(r, peak, peak_kind, BLOCK_STEPS[3])
                    r = None
                    gc.collect()
                    torch.cuda.empty_cache()
                    r = measure_pairwise(torch, gaf, workloads, dev, BLOCK_STEPS[3], 5, nvml, stacked=False)
                    other = pairwise_entry(r, peak, peak_kind, BLOCK_STEPS[3])
                    block["3"]["separate_allocations"] = {k: other[k] for k in (
                        "placement", "gram_loader", "ms_per_call", "ms_per_call_median_of_event_pairs", "value",
                        "min_bytes_frac", "ms_x_sm_mhz")}
                else:
                    r = measure_filter(torch, gaf, workloads, c, dev, 0.97, 0, BLOCK_STEPS[c], 5, nvml,
                                       want_warm=(c == 1), want_c_loop=(c == 1))
                    r["cfg"], r["steps"] = c, BLOCK_STEPS[c]
                    block[str(c)] = block_entry(r, peak, peak_kind, 0.97, 0)
            except Exception as exc:      # a configuration that cannot run here is reported, not hidden
                block[str(c)] = {"error": f"{type(exc).__name__}: {exc}"}
            r = None
            gc.collect()
            torch.cuda.empty_cache()
        for key, D_c, n in (("cosdist_D11.2M", FULL_D[2], 1000), ("cosdist_D124M", FULL_D[4], 200)):
            try:
                block[key] = measure_cosdist(torch, gaf, workloads, dev, D_c, n, nvml, peak, peak_kind)
            except Exception as exc:
                block[key] = {"error": f"{type(exc).__name__}: {exc}"}
            gc.collect()
            torch.cuda.empty_cache()

        try:
            block["variants_config2"] = measure_variants(torch, gaf, workloads, dev, 500, nvml, peak, peak_kind)
        except Exception as exc:
            block["variants_config2"] = {"error": f"{type(exc).__name__}: {exc}"}
        gc.collect()
        torch.cuda.empty_cache()
        for key, D_c, n in (("two_gradients_D11.2M", FULL_D[2], 1000), ("two_gradients_D124M", FULL_D[4], 100)):
            try:
                block[key] = measure_two_gradients(torch, gaf, workloads, dev, D_c, n, nvml, peak, peak_kind)
            except Exception as exc:
                block[key] = {"error": f"{type(exc).__name__}: {exc}"}
            gc.collect()
            torch.cuda.empty_cache()

    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            cpu = time_oracle(cfg, args.tau, args.cpu_seconds)
        sched_used = m["sched_used"]
        n_sets = m["n_sets"]
        basis = "dram" if fr["dram_frac"] is not None else "min_bytes"
        achieved = fr["dram_gbs"] if basis == "dram" else fr["min_bytes_gbs"]
        mhz = t["clocks"]["sm_mhz"]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_dict(
                cfg, K, D, m["dtype"], args.tau,
                SCHED_NAMES[args.schedule] + (" -> " + SCHED_NAMES[sched_used] if not args.schedule else ""),
                "replicas only (the path does not shard)" if world > 1 else "1 GPU",
                (f"{n_sets} rotating input sets of {grad_bytes / 1e6:.0f} MB each (inputs of a step "
                 f"exceed the 126 MB L2 and were last touched {n_sets - 1} steps earlier)"
                 if n_sets > 1 and grad_bytes > L2_BYTES else
                 f"{n_sets} rotating input sets of {grad_bytes / 1e6:.0f} MB each ({n_sets * grad_bytes / 1e6:.0f} MB "
                 f"in all, more than the 126 MB L2)" if n_sets > 1 else
                 f"inputs of one step ({grad_bytes / 1e9:.1f} GB) exceed L2"),
                {"accept_masks": m["masks"],
                 **({"note": "REDUCED length, not the named configuration"} if args.D else {})}),
            "roofline": {
                "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "basis": ("dram: bytes that cross HBM per call while calls run back to back (ncu --cache-control none, "
                          "`traffic`) / time; dram_frac_flushed_caches takes ncu's default capture (caches flushed "
                          "before the launch) instead" if basis == "dram" else
                          "min_bytes: (K b + 4) D / time (no DRAM traffic on record for the kernels as committed)"),
                "traffic": m["traffic"], "traffic_flushed_caches": m["traffic_flushed"], "peak_kind": peak_kind,
                "dram_frac": fr["dram_frac"], "dram_frac_flushed_caches": fr["dram_frac_flushed_caches"], "min_bytes_frac": fr["min_bytes_frac"], "model_frac": fr["model_frac"],
                "dram_gbs": fr["dram_gbs"], "min_bytes_gbs": fr["min_bytes_gbs"], "model_gbs": fr["model_gbs"],
                "frac_of_nominal_8000": achieved / 8000.0,
                "kernel": {3: "gram_fused_kernel (the whole call is this one launch)",
                           2: "Gram kernel + masked_mean_kernel (whole call, both HBM-streaming)",
                           1: "step_kernel x%d (whole call)" % m["launches_per_step"]}[sched_used],
                "byte_model": ("Gram-first: ((K + c) b + 4) D; part of it is served by shared memory and L2, "
                               "so model_frac is an effective rate, not HBM utilisation" if sched_used in (2, 3)
                               else "streaming: (2b+4) + sum_t [4 + b + a_t (b+4)] + 8 + a_last b, times D"),
                "model_bytes_per_launch": m["model_bytes"], "min_bytes_per_step": m["min_bytes"],
                "algorithmic_bytes_per_launch": m["min_bytes"],
                "avg_launch_ms": ms_per_step, "launches_per_call": m["launches_per_step"],
                "per_call_event_pairs": {"median_ms": statistics.median(per_call),
                                         "mean_ms": sum(per_call) / len(per_call), "calls": len(per_call)},
                "ms_x_sm_mhz": None if mhz is None else ms_per_step * mhz,
            },
            "ramp_calls": t["ramp_calls"],
            "e2e": e2e,
            "warm_l2": m.get("warm_l2"),
            "c_loop": m.get("c_loop"),
            "gpu_launches": m["launches_per_step"] * steps,
            "clocks": t["clocks"],
            "cpu_baseline": cpu,
            "configs": block,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_two_gradients(args):
    """--two-gradients: the K = 2 lines of the configs block alone (one GPU), the repeating-outcome stream as the
    headline value."""
    import torch

    import paper_2412_18052_b200 as gaf
    from paper_2412_18052_b200 import workloads

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(0)
    nvml = Nvml(0)
    peak, peak_kind = peak_bandwidth()
    D = args.D or FULL_D[2]
    m = measure_two_gradients(torch, gaf, workloads, "cuda:0", D, args.steps, nvml, peak, peak_kind)
    head = m["all_accepted"]
    line = {
        "metric": "gaf_filter_accumulate micro-gradient GB/s", "value": head["value"], "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": head["ms_per_call"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32 products, f64 sums",
        "data": "synthetic",
        "config": {"workload": m["workload"] + " (NOT a named configuration: two gradients, as in the paper's "
                               "experiments); headline = the stream of calls that all accept"},
        "roofline": {"bound": "hbm", "achieved": head["min_bytes_frac"] * peak, "peak": peak, "unit": "GB/s",
                     "frac": head["min_bytes_frac"], "basis": "min_bytes: (2 b + 4) D", "traffic": None,
                     "peak_kind": peak_kind, "kernel": "gram_fused_kernel<float, 2>",
                     "algorithmic_bytes_per_launch": m["min_bytes_per_call"]},
        "two_gradients": m, "e2e": None, "gpu_launches": head["launches_per_call"] * args.steps,
        "clocks": head["clocks"], "cpu_baseline": None,
    }
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.two_gradients:
        if int(os.environ.get("RANK", "0")) == 0:
            run_two_gradients(args)
    elif args.workload == 3:
        if int(os.environ.get("RANK", "0")) == 0:
            run_pairwise(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
