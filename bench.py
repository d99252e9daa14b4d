"""Benchmark of the HADFL round hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c2]
                    [--min-seconds 0.5] [--sweep default|full|none] [--no-cpu-baseline]
    python bench.py --table saved_line.json                               (markdown tables of its sweep)
    python bench.py --profile-case [--pc-fused] [--pc-steps 1,8] ...      (target of ncu captures)

A "step" is one round of the whole hot path over one synthetic workload: local update of every
device with its own step count, selection (host), aggregation with write-back, version update and
per-replica statistics - one hadfl_round call, one kernel launch.  Prints ONE JSON line (rank 0).

  value     rounds/s with everything resident in HBM.  A timed region is exactly K rounds between a
            barrier + synchronize on both sides, timed with CUDA events on the library's stream,
            max over ranks.  The region is repeated until --min-seconds have been timed (so that
            the clock sampler sees the GPU under load whatever K is); value is the median over the
            repeats, value_min / value_max the spread.
  kernels / separate_calls   the same rounds as separate calls (hadfl_local_step, hadfl_select,
            hadfl_aggregate, hadfl_stats_enqueue) with CUDA events around every launch: the
            bandwidth of each kernel on its own; plus the local update at one step per device
            (its memory-bound regime).
  e2e       the same rounds through the C ABI with HOST buffers: every round also reads the
            statistics (2N floats) and the aggregated model (P floats, the coordinator's model
            backup) into pinned host memory.  Median of three regions, spread reported.
  roofline  for the kernel of the timed region (the fused round): algorithmic bytes per launch /
            average launch time (CUDA events around each launch) against the measured copy
            bandwidth of the B200 (MEASURED_PEAKS.json), or - when arithmetic is the higher floor -
            element-steps per second against the busiest arithmetic pipe (see PIPE_CYCLES below).
  sweep     the metric against P: the bandwidth sweep (N=16, k=4, P = 2^20 .. 2^27, fp32 and bf16
            storage, one step per device and step ratios 1,1,2,2,4,4,8,8) plus the VGG-16- and
            ResNet-50-sized workloads: rounds/s of the fused round and GB/s of every kernel.
            Outside the timed region; N = 1 only.
  cpu_baseline  the CPU checker (single thread, as it stands) on a column sample of the same
            workload, scaled to the full vector; beside it the same sample on all host cores
            (the checker's -fopenmp build).

N > 1 runs N independent replicas of the workload, one process per GPU (launched by torchrun):
the path does not shard across GPUs and has no exchange step, so there is no collective in it.
--impl reference times the CPU checker instead (rank 0 only).
"""
import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2111_08274_b200 import workloads  # noqa: E402

METRIC = "aggregation_rounds_per_sec"
UNIT = "rounds/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
SM_COUNT, SUBPARTITIONS_PER_SM, SM_MAX_MHZ = 148, 4, 1965.0
ORACLE_NS_PER_ELEM_STEP = 45e-9   # rough cost of the CPU checker, used only to size its sample

# Arithmetic roofline of the local update (and of the fused round, whose step loop is the same
# code).  With several steps per device the launch is bound by the arithmetic pipes of the SM, not
# by HBM.  The figures are busy cycles of each pipe per SM sub-partition and per element-step
# (one SGD step of one parameter of one device), measured with ncu on k_local_step at 4 and at 8
# steps per device (difference of the two launches / element-steps between them; summary and
# command under profiles/k_local_step_pipes_N8_P4M.md).  A sub-partition cannot process an
# element-step in fewer cycles than its busiest pipe needs, so
#   peak = SMs x 4 sub-partitions x SM clock / max(PIPE_CYCLES)      [element-steps per second]
# with the SM clock sampled during the timed region.  "fmaheavy" counts only what no scheduling can
# move off that pipe, the 36 32x32->64-bit multiplies of Philox per step and 8-parameter pack at 4
# cycles each (with the packed FP32 instructions the hardware runs there it is busy 0.69); "issue"
# is the warp scheduler's issue slot (one instruction per cycle: 132.8 warp instructions per step
# and pack).
PIPE_CYCLES_PER_ELEM_STEP = {"fmaheavy": 0.5625, "issue": 0.5186, "xu": 0.5000, "alu": 0.3572, "fmalite": 0.1925}
PIPE_CYCLES_SOURCE = "profiles/k_local_step_pipes_N8_P4M.md"

# DRAM bytes per unit of work moved by one launch, from the ncu captures summarised under profiles/
# (dram__bytes_read.sum and dram__bytes_write.sum on a smaller case of the same kernel, N=8,
# P=4 194 306).  Reads grow in proportion to the units processed.  Writes are a LOWER BOUND: in the
# small capture up to 126 MB of written lines are still dirty in L2 when the kernel ends and are
# not counted.  Unit: (device, parameter) for the round, the local update and the statistics, one
# element of a selected row for the aggregation.  None = not captured for the kernel as it stands.
NCU_DRAM_READ_PER_UNIT = {"round": 8.00, "local_step": 8.00, "aggregate": 4.00, "stats": 4.00}
NCU_DRAM_WRITE_PER_UNIT = {"round": 6.12, "local_step": 6.12, "aggregate": 0.26, "stats": 0.003}
NCU_DRAM_SOURCE = "profiles/kernels_small_case_N8_P4M.md"


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def describe(wl):
    steps = "uniform[%d,%d] per device per round" % (wl.steps_lo, wl.steps_hi) \
        if wl.steps_rule == "uniform" else "fixed %s" % (list(wl.steps_fixed),)
    return {"workload": wl.name, "n_devices": wl.n_devices, "n_params": wl.n_params, "k": wl.k,
            "local_steps": steps, "lr": wl.lr, "momentum": wl.momentum,
            "weight_decay": wl.weight_decay, "grad_std": wl.grad_std,
            "storage": "bf16" if wl.dtype else "fp32",
            "arena_bytes": wl.n_devices * wl.n_params * (6 if wl.dtype else 8),
            "l2": "arena is larger than L2 (126 MB): no flush between rounds",
            "multi_gpu": "replicas only (no sharding, no collective)"}


def mean_steps_per_device(wl, rounds=8):
    return float(np.mean([wl.steps_for_round(r).sum() for r in range(rounds)])) / wl.n_devices


def spread(values):
    v = [float(x) for x in values]
    return {"median": float(np.median(v)), "min": min(v), "max": max(v), "n": len(v)}


# ---- CPU checker timing ------------------------------------------------------------------------
def time_oracle(wl, frac_cols, rounds, openmp=False):
    """Rounds of the CPU checker on the first `frac_cols` of the column groups; returns
    (seconds per full-vector round for each round, description of the sample, threads used)."""
    import oracle
    n_groups = (wl.n_params + 3) // 4
    take = min(n_groups, max(64, int(n_groups * frac_cols)))
    groups = np.arange(take, dtype=np.uint32)
    sim = oracle.Sim(wl.n_devices, wl.n_params, dtype=wl.dtype, momentum=wl.momentum,
                     weight_decay=wl.weight_decay, grad_std=wl.grad_std, init_std=wl.init_std,
                     seed=wl.seed, version_scale=wl.version_scale, weight_mode=wl.weight_mode,
                     groups=groups, openmp=openmp)
    ids = wl.device_ids()
    per_round = []
    for r in range(rounds):
        t0 = time.perf_counter()
        sim.local_step(ids, wl.steps_for_round(r), wl.lr)
        sel = sim.select(r, wl.k, wl.select_seed())
        sim.aggregate(sel)
        sim.stats(int(sel[0]))
        per_round.append(time.perf_counter() - t0)
    sim.close()
    scale = n_groups / float(take)
    what = "%d round(s) on the first %d of %d column groups (%.3f%% of the vector), scaled by %.1f" % (
        rounds, take, n_groups, 100.0 / scale, scale)
    return [t * scale for t in per_round], what, oracle.threads(openmp), [t for t in per_round]


def cpu_model():
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except Exception:
        pass
    return "unknown"


def run_reference(args, wl):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    # Bounded sample: size the column sample so that the whole run takes about a minute.
    total = args.warmup + args.steps
    full_round_s = wl.n_devices * wl.n_params * mean_steps_per_device(wl) * ORACLE_NS_PER_ELEM_STEP
    frac = min(1.0 / 8.0, 60.0 / (total * full_round_s))
    times, what, threads, raw = time_oracle(wl, frac, total)
    sec = float(np.mean(times[args.warmup:]))
    value = 1.0 / sec
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": sec * 1e3,
            "ms_per_step_is": "time of one round on the column sample x (vector / sample): an "
                              "extrapolation to the full vector, linear because every operation of "
                              "the round is elementwise in the column index",
            "sample_ms_per_step": float(np.mean(raw[args.warmup:])) * 1e3,
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": describe(wl),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": what},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---- clocks --------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU while the timed region runs (NVML, read
    only)."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index, period=0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        if not self.ok:
            return
        while not self._halt.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.dev, self.nv.NVML_CLOCK_SM)))
                bits = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.dev))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._halt.set()
        if self.is_alive():
            self.join(timeout=2.0)
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def physical_gpu_index(local_index):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


def max_over_ranks(value, world):
    """Max of a host scalar over all ranks (the job is as slow as its slowest rank)."""
    if world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def repeats_for(first_region_s, min_seconds, cap=400):
    """How many K-round regions to time in all so that at least min_seconds are timed; a pure
    function of a value that is the same on every rank (the max over ranks of the first region)."""
    if first_region_s <= 0.0:
        return 1
    return int(max(1, min(cap, math.ceil(min_seconds / first_region_s))))


# ---- per-kernel figures ----------------------------------------------------------------------------
def gbs_entry(nbytes, ms, peak, frac_key):
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"avg_ms": ms, "algorithmic_bytes": nbytes, "achieved_gbs": gbs, frac_key: gbs / peak,
            "frac_of_8TBs": gbs / NOMINAL_HBM_GBS}


def traffic_entry(kernel, units):
    rd, wr = NCU_DRAM_READ_PER_UNIT[kernel], NCU_DRAM_WRITE_PER_UNIT[kernel]
    if rd is None or wr is None:
        return {"traffic": None}
    return {"traffic": (rd + wr) * units, "traffic_read": rd * units,
            "traffic_write_lower_bound": wr * units,
            "traffic_is": "DRAM bytes per unit from the ncu capture of a smaller case of this kernel "
                          "(%s) x the units of this launch; reads scale in proportion, writes are a "
                          "lower bound (lines still dirty in the 126 MB L2 at kernel end are not "
                          "counted in the small capture)" % NCU_DRAM_SOURCE}


def measure_case(wl, rounds, peak, frac_key, warmup=3):
    """One point of the sweep: median launch time of every kernel over `rounds` rounds run as
    separate calls, then the same rounds through the fused kernel (CUDA events around each launch)."""
    import torch
    from paper_2111_08274_b200 import runtime
    arena = runtime.Arena(wl)
    h = arena.h
    N, P, k = wl.n_devices, wl.n_params, wl.k
    ew, em = (2 if wl.dtype else 4), (2 if wl.m_dtype else 4)
    r = 0
    for _ in range(warmup):
        arena.run_round(r)
        r += 1
    names = ("local_step", "aggregate", "stats")
    ev = {n: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(rounds)] for n in names}
    steps = [wl.steps_for_round(r + i) for i in range(rounds)]
    torch.cuda.synchronize()
    for i in range(rounds):
        a, b = ev["local_step"][i]
        a.record(); h.local_step(arena.ids, steps[i], wl.lr); b.record()
        sel = h.select(r + i, k, arena.select_seed)
        a, b = ev["aggregate"][i]
        a.record(); h.aggregate(sel); b.record()
        a, b = ev["stats"][i]
        a.record(); h.stats_enqueue(int(sel[0])); b.record()
    torch.cuda.synchronize()
    ms = {n: float(np.median([a.elapsed_time(b) for a, b in ev[n]])) for n in names}
    r += rounds
    for i in range(warmup):
        arena.run_round_fused(r + i)
    r += warmup
    evf = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(rounds)]
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    for i in range(rounds):
        a, b = evf[i]
        a.record(); arena.run_round_fused(r + i); b.record()
    torch.cuda.synchronize()
    fused_ms = float(np.median([a.elapsed_time(b) for a, b in evf]))
    r += rounds
    # rounds/s with 8 rounds enqueued per library call (hadfl_rounds): small vectors then show the
    # kernel and not the per-call overhead of the caller, while the launch queue stays shallow
    def rounds_by_calls_of_8(r0):
        arena.run_rounds_fused(r0, 8)  # untimed: the first launch of a kind starts on the previous kernel's cache contents
        r0 += 8
        launches0 = h.launch_count()
        torch.cuda.synchronize()
        start.record()
        for i in range(0, 4 * rounds, 8):
            arena.run_rounds_fused(r0 + i, min(8, 4 * rounds - i))
        end.record()
        torch.cuda.synchronize()
        return start.elapsed_time(end) / (4 * rounds), 4 * rounds / (h.launch_count() - launches0)
    fused_wall_ms, rounds_per_launch = rounds_by_calls_of_8(r)
    r += 4 * rounds + 8
    # where the library put several rounds into one launch: the same with one launch per round
    single_wall_ms = fused_wall_ms
    if rounds_per_launch > 1:
        h.set_round_batch(1)
        single_wall_ms, _ = rounds_by_calls_of_8(r)
    grid = h.round_grid()
    arena.close()
    nbytes = {"local_step": N * P * 2 * (ew + em), "aggregate": 2 * k * P * ew, "stats": N * P * ew,
              "round": N * P * 2 * (ew + em)}
    mean_steps = float(np.mean([s.mean() for s in steps]))
    res = {"workload": wl.name, "N": N, "P": P, "k": k,
           "storage": ("bf16" if wl.dtype else "fp32") + ("+bf16 m" if wl.m_dtype else ""),
           "mean_steps_per_device": mean_steps, "arena_mb": N * P * (ew + em) / 1e6,
           "rounds_per_s": 1e3 / fused_wall_ms, "round_ms": fused_wall_ms, "round_grid_blocks": grid,
           "rounds_per_launch": rounds_per_launch, "rounds_per_s_one_round_per_launch": 1e3 / single_wall_ms,
           "separate_calls_rounds_per_s": 1e3 / (ms["local_step"] + ms["aggregate"] + ms["stats"]),
           "hbm_bound": bool(N * P * (ew + em) > 126e6),
           "kernels": {"round": gbs_entry(nbytes["round"], fused_ms, peak, frac_key)}}
    res["kernels"]["round"]["gelem_steps_per_s"] = N * P * mean_steps / (fused_ms * 1e-3) / 1e9
    for n in names:
        res["kernels"][n] = gbs_entry(nbytes[n], ms[n], peak, frac_key)
    return res


def measure_sync(wl, peak, frac_key, reps=30):
    """Global synchronisation from device 0 to the N - k others: overwrite and beta-mix."""
    import torch
    from paper_2111_08274_b200 import runtime
    arena = runtime.Arena(wl)
    h = arena.h
    ew = 2 if wl.dtype else 4
    dst = np.arange(wl.k, wl.n_devices, dtype=np.int32)
    out = {"workload": wl.name, "N": wl.n_devices, "P": wl.n_params, "receivers": len(dst),
           "storage": "bf16" if wl.dtype else "fp32", "kernels": {}}
    for name, call, nbytes in (("broadcast", lambda: h.broadcast(0, dst), (1 + len(dst)) * wl.n_params * ew),
                               ("integrate", lambda: h.integrate(0, dst, 0.5), (1 + 2 * len(dst)) * wl.n_params * ew)):
        for _ in range(3):
            call()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            call()
        b.record()
        torch.cuda.synchronize()
        out["kernels"][name] = gbs_entry(nbytes, a.elapsed_time(b) / reps, peak, frac_key)
    arena.close()
    return out


def sweep_cases(which):
    """default: the bandwidth sweep at five sizes, both storages, one step per device and step ratios
    1,1,2,2,4,4,8,8, plus the VGG-16- and ResNet-50-sized workloads.  full: every size 2^16 .. 2^27, all
    five workloads with k in {2, 8, 16}, the ResNet-18 size at one step per device, and the
    reduced-precision variants (bf16 momentum, stochastic rounding)."""
    from dataclasses import replace
    cases = [workloads.c3(), workloads.c4(8)]
    sizes = (20, 22, 24, 26, 27)
    if which == "full":
        cases = [workloads.c1(), workloads.c2(), workloads.c3(), workloads.c4(2), workloads.c4(8), workloads.c4(16),
                 workloads.Workload("c2_steps1", 8, 11_173_962, 4, 50, "fixed", (1,) * 8, seed=workloads.BASE_SEED + 2)]
        sizes = tuple(range(16, 28))
    for dtype in (0, 1):
        for hetero in (False, True):
            for lp in sizes:
                cases.append(workloads.c5(lp, dtype=dtype, hetero=hetero))
    if which == "full":
        for hetero in (False, True):
            for m_dtype, rounding in ((0, 1), (1, 0), (1, 1)):
                base = workloads.c5(25, dtype=1, hetero=hetero)
                name = base.name + ("_m16" if m_dtype else "") + ("_sr" if rounding else "")
                cases.append(replace(base, name=name, m_dtype=m_dtype, rounding=rounding))
    return cases


def run_sweep(peak, frac_key, which="default", rounds=12):
    """The metric against P (bandwidth sweep) and the larger CNN-sized workloads."""
    import torch
    out = []
    for wl in sweep_cases(which):
        out.append(measure_case(wl, rounds, peak, frac_key))
        torch.cuda.empty_cache()
    sync = []
    if which == "full":
        for wl in (workloads.c2(), workloads.c3(), workloads.c4(8), workloads.c5(25, dtype=1)):
            sync.append(measure_sync(wl, peak, frac_key))
            torch.cuda.empty_cache()
    return out, sync


def print_tables(path):
    """Markdown tables of the sweep carried by a saved JSON line of this benchmark."""
    with open(path) as f:
        line = json.loads(f.read().strip().splitlines()[-1])
    sw = line["sweep"]
    peak = sw["peak_gbs"]
    key = "frac_of_%s_hbm" % sw["peak_kind"]

    def cell(k):
        return "%.1f | %.0f (%.0f / %.0f)" % (k["avg_ms"] * 1e3, k["achieved_gbs"], 100 * k[key], 100 * k["frac_of_8TBs"])
    print("GB/s = algorithmic bytes / time; percentages: of the %s %.0f GB/s / of the nominal 8000 GB/s.\n" % (sw["peak_kind"], peak))
    print("| workload | N | P | k | storage | mean steps | K1 µs | K1 GB/s (% meas / % 8T) | K2 µs | K2 GB/s (%/%) | K3 µs | K3 GB/s (%/%) "
          "| separate calls rounds/s | fused `hadfl_round` µs | fused GB/s (%/%) | fused rounds/s, one round per launch "
          "| `hadfl_rounds` rounds/s (rounds per launch) | G element-steps/s |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|")
    for p in sw["points"]:
        ks = p["kernels"]
        print("| %s | %d | %d | %d | %s | %.2f | %s | %s | %s | %.0f | %s | %.0f | %.0f (%.3g) | %.0f |" % (
            p["workload"], p["N"], p["P"], p["k"], p["storage"], p["mean_steps_per_device"], cell(ks["local_step"]),
            cell(ks["aggregate"]), cell(ks["stats"]), p["separate_calls_rounds_per_s"], cell(ks["round"]),
            p["rounds_per_s_one_round_per_launch"], p["rounds_per_s"], p["rounds_per_launch"],
            ks["round"]["gelem_steps_per_s"]))
    if sw.get("sync"):
        print("\n| workload | N | P | receivers | storage | broadcast µs | GB/s (%/%) | integrate µs | GB/s (%/%) |")
        print("|---|---|---|---|---|---|---|---|---|")
        for p in sw["sync"]:
            print("| %s | %d | %d | %d | %s | %s | %s |" % (p["workload"], p["N"], p["P"], p["receivers"], p["storage"],
                                                         cell(p["kernels"]["broadcast"]), cell(p["kernels"]["integrate"])))


# ---- our arm ---------------------------------------------------------------------------------------
def run_ours(args, wl):
    import torch
    import torch.distributed as dist
    from paper_2111_08274_b200 import runtime

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU implementation")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus != world:
        raise SystemExit("--gpus %d does not match WORLD_SIZE %d (launch with torch.distributed.run)"
                         % (args.gpus, world))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    runtime.ensure_built()

    arena = runtime.Arena(wl, device="cuda:%d" % local)
    h = arena.h
    N, P, k = wl.n_devices, wl.n_params, wl.k
    elem_w = 2 if wl.dtype else 4
    warmup = max(args.warmup, 3)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    r = 0
    for _ in range(warmup):
        arena.run_round(r)
        r += 1

    K = args.steps
    ids, seed = arena.ids, arena.select_seed
    peak, peak_kind = measured_peak()
    frac_key = "frac_of_%s_hbm" % peak_kind

    # ---- timed regions: exactly K rounds each, every round ONE call of the public API
    # (hadfl_round: local steps of every device, selection, aggregation with write-back, version
    # update, statistics); repeated until --min-seconds have been timed ---------------------------
    def timed_region(r0):
        ev_round = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                    for _ in range(K)]
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        step_lists = [wl.steps_for_round(r0 + i) for i in range(K)]
        syncs = [bool(wl.sync_every) and (r0 + i + 1) % wl.sync_every == 0 for i in range(K)]
        barrier()
        start.record()
        for i in range(K):
            a, b = ev_round[i]
            a.record(); h.round(ids, step_lists[i], wl.lr, r0 + i, k, seed, sync_all=syncs[i]); b.record()
        end.record()
        barrier()
        region_ms = max_over_ranks(start.elapsed_time(end), world)
        launch_ms = [a.elapsed_time(b) for a, b in ev_round]
        return region_ms, launch_ms, float(np.sum([s.sum() for s in step_lists]))

    sampler = ClockSampler(physical_gpu_index(local))
    launches0 = h.launch_count()
    sampler.start()
    region_ms, launch_ms, step_sum = [], [], 0.0
    first_ms, lm, ss = timed_region(r)
    r += K
    region_ms.append(first_ms); launch_ms += lm; step_sum += ss
    for _ in range(repeats_for(first_ms * 1e-3, args.min_seconds) - 1):
        ms_, lm, ss = timed_region(r)
        r += K
        region_ms.append(ms_); launch_ms += lm; step_sum += ss
    clocks = sampler.stop()
    launches = h.launch_count() - launches0
    elapsed_ms = float(np.median(region_ms))
    per_region = [world * K / (ms_ * 1e-3) for ms_ in region_ms]
    mean_steps = step_sum / (len(region_ms) * K) / N
    round_ms = float(np.mean(launch_ms))
    round_bytes = N * P * (2 * elem_w + 8)             # w and m read and written once per round
    round_gbs = round_bytes / (round_ms * 1e-3) / 1e9

    # ---- the same rounds as separate calls, to time each kernel on its own ---------------------
    Ks = max(3, min(K, 200))
    names = ("local_step", "aggregate", "stats")
    ev = {n: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(Ks)] for n in names}
    sstart, send = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sep_steps = [wl.steps_for_round(r + i) for i in range(Ks)]
    barrier()
    sstart.record()
    for i in range(Ks):
        a, b = ev["local_step"][i]
        a.record(); h.local_step(ids, sep_steps[i], wl.lr); b.record()
        sel = h.select(r + i, k, seed)
        a, b = ev["aggregate"][i]
        a.record(); h.aggregate(sel); b.record()
        a, b = ev["stats"][i]
        a.record(); h.stats_enqueue(int(sel[0])); b.record()
    send.record()
    barrier()
    r += Ks
    sep_ms = max_over_ranks(sstart.elapsed_time(send), world) / Ks
    kern_ms = {n: float(np.mean([a.elapsed_time(b) for a, b in ev[n]])) for n in names}
    sep_mean_steps = float(np.mean([s.sum() for s in sep_steps])) / N
    alg_bytes = {"local_step": N * P * (2 * elem_w + 8),       # read + write w and m, once per call
                 "aggregate": 2 * k * P * elem_w,              # k rows read, k rows written
                 "stats": N * P * elem_w}                      # every row read once
    units = {"local_step": N * P, "aggregate": k * P, "stats": N * P}
    kernels = {"round": gbs_entry(round_bytes, round_ms, peak, frac_key)}
    kernels["round"].update({"mean_steps_per_device": mean_steps, "grid_blocks": h.round_grid(),
                             "gelem_steps_per_s": N * P * mean_steps / (round_ms * 1e-3) / 1e9})
    kernels["round"].update(traffic_entry("round", N * P))
    for n in names:
        kernels[n] = gbs_entry(alg_bytes[n], kern_ms[n], peak, frac_key)
        kernels[n]["share_of_separate_round"] = kern_ms[n] / sep_ms
        kernels[n].update(traffic_entry(n, units[n]))
    # ---- the local update in its memory-bound regime: one step per device per call ---------------
    Kb = max(3, min(K, 100))
    ones = np.ones(N, dtype=np.int32)
    ev1 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(Kb)]
    for _ in range(3):
        h.local_step(ids, ones, wl.lr)
    barrier()
    for a, b in ev1:
        a.record(); h.local_step(ids, ones, wl.lr); b.record()
    barrier()
    one_ms = float(np.mean([a.elapsed_time(b) for a, b in ev1]))
    kernels["local_step_1_step_per_device"] = gbs_entry(alg_bytes["local_step"], one_ms, peak, frac_key)
    kernels["local_step_1_step_per_device"].update(traffic_entry("local_step", N * P))
    kernels["local_step"]["mean_steps_per_device"] = sep_mean_steps
    kernels["local_step"]["gelem_steps_per_s"] = N * P * sep_mean_steps / (kern_ms["local_step"] * 1e-3) / 1e9
    separate = {"rounds_per_s": world * 1e3 / sep_ms, "ms_per_round": sep_ms, "rounds": Ks,
                "what": "hadfl_local_step + hadfl_select + hadfl_aggregate + hadfl_stats_enqueue"}

    # ---- roofline of the timed kernel -----------------------------------------------------------------
    sm_mhz = clocks["sm_mhz"] or SM_MAX_MHZ
    busiest = max(PIPE_CYCLES_PER_ELEM_STEP, key=PIPE_CYCLES_PER_ELEM_STEP.get)
    alu_peak = SM_COUNT * SUBPARTITIONS_PER_SM * sm_mhz * 1e6 / PIPE_CYCLES_PER_ELEM_STEP[busiest] / 1e9
    alu_achieved = kernels["round"]["gelem_steps_per_s"]
    hbm_src = ("of measured (copy bandwidth, MEASURED_PEAKS.json)" if peak_kind == "measured"
               else "of fallback (6650 GB/s)")
    alu_src = ("derived from counters: %d SMs x %d sub-partitions x %.0f MHz (median SM clock sampled "
               "in the timed region) / %.4f busy cycles of the busiest pipe (%s) per element-step "
               "(%s)" % (SM_COUNT, SUBPARTITIONS_PER_SM, sm_mhz, PIPE_CYCLES_PER_ELEM_STEP[busiest],
                         busiest, PIPE_CYCLES_SOURCE))
    # which floor is higher for this launch: bytes / HBM peak or element-steps / arithmetic peak?
    t_hbm, t_alu = round_bytes / (peak * 1e9), N * P * mean_steps / (alu_peak * 1e9)
    if t_alu > t_hbm:
        roofline = {"kernel": "k_round (the whole round in one launch)", "bound": "alu",
                    "achieved": alu_achieved, "peak": alu_peak, "unit": "Gelem-step/s",
                    "frac": alu_achieved / alu_peak, "peak_source": alu_src,
                    "hbm_achieved_gbs": round_gbs, "hbm_peak_gbs": peak,
                    "hbm_frac": round_gbs / peak, "hbm_peak_source": hbm_src}
    else:
        roofline = {"kernel": "k_round (the whole round in one launch)", "bound": "hbm",
                    "achieved": round_gbs, "peak": peak, "unit": "GB/s", "frac": round_gbs / peak,
                    "peak_source": hbm_src, "alu_achieved_gelem_steps": alu_achieved,
                    "alu_peak_gelem_steps": alu_peak, "alu_frac": alu_achieved / alu_peak,
                    "alu_peak_source": alu_src}
    roofline["floor_ms"] = {"hbm": t_hbm * 1e3, "alu": t_alu * 1e3, "measured": round_ms}
    roofline["pipe_cycles_per_elem_step"] = PIPE_CYCLES_PER_ELEM_STEP
    roofline.update(traffic_entry("round", N * P))
    roofline["note"] = ("algorithmic bytes = 16 per (device, parameter) whatever the step count; "
                        "mean steps per device here: %.2f; the bandwidth-bound kernels (local update "
                        "at 1 step, aggregation, statistics) are listed under `kernels`" % mean_steps)

    # ---- end to end: host buffers, results read back every round -----------------------------
    # Every round: hadfl_round (its inputs are host arrays), the statistics read back (2N floats),
    # and the aggregated model copied to pinned host memory (the coordinator's model backup).
    # (a) overlapped: hadfl_backup_begin / hadfl_backup_wait move the model on a copy stream while
    #     the next round runs; (b) blocking: hadfl_read_params waits for the transfer every round.
    Ke = max(3, min(K, 200))
    host_model = [torch.empty(P, dtype=torch.float32).pin_memory() for _ in range(2)]
    h2d = 4 * N + 4 * N + 4 * k + 4            # ids, step counts, selected ids, lr (launch parameters)
    d2h = 2 * N * 4 + P * 4                    # statistics + the aggregated model

    def e2e_overlapped(r0):
        barrier()
        t0 = time.perf_counter()
        for i in range(Ke):
            sel = arena.run_round_fused(r0 + i)
            if i > 0:
                h.backup_wait()                    # the previous round's model has arrived
            h.stats_read()
            h.backup_begin(int(sel[0]), host_model[i % 2])
        h.backup_wait()
        torch.cuda.synchronize()
        return world * Ke / max_over_ranks(time.perf_counter() - t0, world)

    def e2e_blocking(r0):
        barrier()
        t0 = time.perf_counter()
        for i in range(Ke):
            sel = arena.run_round_fused(r0 + i)
            h.stats_read()
            h.read_params(int(sel[0]), out=host_model[0])
        torch.cuda.synchronize()
        return world * Ke / max_over_ranks(time.perf_counter() - t0, world)

    def e2e_stats_only(r0):
        barrier()
        t0 = time.perf_counter()
        for i in range(Ke):
            arena.run_round_fused(r0 + i)
            h.stats_read()                 # waits for the round: no launch runs ahead of the host
        torch.cuda.synchronize()
        return world * Ke / max_over_ranks(time.perf_counter() - t0, world)

    e2e_runs = {}
    for name, fn in (("overlapped", e2e_overlapped), ("blocking", e2e_blocking), ("stats_only", e2e_stats_only)):
        vals = []
        for _ in range(3):
            vals.append(fn(r))
            r += Ke
        e2e_runs[name] = spread(vals)
    e2e = {"value": e2e_runs["overlapped"]["median"], "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "steps": Ke, "spread": e2e_runs["overlapped"],
           "what": "hadfl_round + hadfl_stats_read + hadfl_backup_begin/wait(selected[0]) into pinned "
                   "host memory, the model transfer overlapping the next round; median of 3 regions",
           "blocking_value": e2e_runs["blocking"]["median"], "blocking_spread": e2e_runs["blocking"],
           "blocking_what": "the same with hadfl_read_params (waits for the transfer every round)",
           "stats_only_value": e2e_runs["stats_only"]["median"], "stats_only_spread": e2e_runs["stats_only"],
           "stats_only_what": "hadfl_round + hadfl_stats_read only (2N floats back per round, no model copy)"}

    line = {"metric": METRIC, "value": float(np.median(per_region)), "unit": UNIT,
            "n_gpus": world, "steps": K, "warmup": warmup,
            "ms_per_step": elapsed_ms / K, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": describe(wl),
            "value_is": "median over `repeats` timed regions of exactly `steps` rounds each",
            "repeats": len(region_ms), "value_min": min(per_region), "value_max": max(per_region),
            "timed_seconds": float(np.sum(region_ms)) * 1e-3,
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "kernels": kernels, "separate_calls": separate}

    arena.close()
    del host_model
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and args.sweep != "none":
        points, sync = run_sweep(peak, frac_key, args.sweep)
        line["sweep"] = {"what": "fused round (rounds/s, one hadfl_round call per round, CUDA events) and "
                                 "every kernel's algorithmic GB/s against P; 12 rounds per point, medians",
                         "peak_gbs": peak, "peak_kind": peak_kind, "points": points}
        if sync:
            line["sweep"]["sync"] = sync
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        times, what, threads, _ = time_oracle(wl, 1.0 / 2.0, 3)
        base = {"value": 1.0 / float(np.mean(times)), "unit": UNIT, "cores": threads,
                "kind": "oracle", "sample": what, "nproc": os.cpu_count(), "cpu_model": cpu_model()}
        try:
            times_all, _, threads_all, _ = time_oracle(wl, 1.0 / 2.0, 3, openmp=True)
            base["value_all_cores"] = 1.0 / float(np.mean(times_all))
            base["cores_all"] = threads_all
            base["all_cores_is"] = "the same sample with the checker's -fopenmp build (loops split over column blocks)"
        except Exception as e:           # no OpenMP runtime on the host: the 1-thread figure stands
            base["value_all_cores"] = None
            base["all_cores_error"] = str(e)
        line["cpu_baseline"] = base
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# ---- small fixed case for profiler captures --------------------------------------------------------
def run_profile_case(a):
    """Runs a small, fixed case of every kernel a few times: the target of `ncu` captures.  The arena
    (N * P * 8 bytes for fp32) should exceed the 126 MB L2 so that DRAM counters mean something, and
    stay at a few hundred MB so that a multi-pass capture ends quickly.  Launch order per repetition:
    local update once per entry of --pc-steps (all devices that many steps), aggregation of k
    devices, statistics, broadcast to the other devices, the same as a mix (beta = 1/2).  With
    --pc-fused: one hadfl_round launch per entry of --pc-steps instead; with --pc-batch R also one
    hadfl_rounds call of R rounds per entry (one launch of R rounds where the library batches them)."""
    from paper_2111_08274_b200 import runtime
    wl = workloads.Workload("profile", a.pc_n, a.pc_p, a.pc_k, 1, "fixed", (1,) * a.pc_n, dtype=a.pc_dtype,
                            seed=workloads.BASE_SEED)
    runtime.ensure_built()
    ar = runtime.Arena(wl)
    ids = wl.device_ids()
    sel = ids[: a.pc_k]
    steps = [int(t) for t in a.pc_steps.split(",")]
    for rep in range(a.pc_reps):
        if a.pc_fused:
            for s in steps:
                ar.h.round(ids, np.full(a.pc_n, s, dtype=np.int32), wl.lr, rep, a.pc_k, 1)
            for s in steps if a.pc_batch > 1 else ():
                ar.h.rounds(100 * rep, np.full((a.pc_batch, a.pc_n), s, dtype=np.int32), wl.lr, a.pc_k, 1)
            continue
        for s in steps:
            ar.h.local_step(ids, np.full(a.pc_n, s, dtype=np.int32), wl.lr)
        ar.h.aggregate(sel)
        ar.h.stats_enqueue(int(sel[0]))
        ar.h.broadcast(int(sel[0]), ids[a.pc_k:])
        ar.h.integrate(int(sel[0]), ids[a.pc_k:], 0.5)
    ar.h.synchronize()
    n2, _ = ar.h.stats_read()
    print("ok: launches=%d norm2[0]=%.6g" % (ar.h.launch_count(), n2[0]))
    ar.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--min-seconds", type=float, default=0.5,
                    help="the K-round timed region is repeated until this much has been timed")
    ap.add_argument("--sweep", default="default", choices=["default", "full", "none"],
                    help="which set of workloads the sweep against P covers (see sweep_cases)")
    ap.add_argument("--no-sweep", action="store_true", help="same as --sweep none")
    ap.add_argument("--table", default="", help="print the markdown tables of a saved JSON line and exit")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile-case", action="store_true", help="run the small case for ncu and exit")
    ap.add_argument("--pc-n", type=int, default=8)
    ap.add_argument("--pc-p", type=int, default=4 * 1024 * 1024 + 2)
    ap.add_argument("--pc-k", type=int, default=4)
    ap.add_argument("--pc-steps", type=str, default="1,8")
    ap.add_argument("--pc-dtype", type=int, default=0)
    ap.add_argument("--pc-reps", type=int, default=2)
    ap.add_argument("--pc-fused", action="store_true", help="hadfl_round instead of the separate calls")
    ap.add_argument("--pc-batch", type=int, default=0, help="with --pc-fused: also hadfl_rounds calls of that many rounds")
    args = ap.parse_args()
    if args.no_sweep:
        args.sweep = "none"
    if args.table:
        print_tables(args.table)
        return
    if args.profile_case:
        run_profile_case(args)
        return
    wl = workloads.by_name(args.workload)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
