"""Benchmark of the HADFL round hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c2]

A "step" is one round of the whole hot path over one synthetic workload: local update of every
device with its own step count, selection (host), aggregation with write-back, version update and
per-replica statistics - one hadfl_round call, one kernel launch.  Prints ONE JSON line (rank 0).

  value     rounds/s with everything resident in HBM; timed with CUDA events on the library's
            stream, barrier + synchronize on both sides, max over ranks.
  kernels / separate_calls   the same rounds as separate calls (hadfl_local_step, hadfl_select,
            hadfl_aggregate, hadfl_stats_enqueue) with CUDA events around every launch: the
            bandwidth of each kernel on its own; plus the local update at one step per device
            (its memory-bound regime).
  e2e       the same rounds through the C ABI with HOST buffers: every round also reads the
            statistics (2N floats) and the aggregated model (P floats, the coordinator's model
            backup) into pinned host memory.
  roofline  for the kernel of the timed region (the fused round): algorithmic bytes per launch /
            average launch time (CUDA events around each launch), against the measured copy
            bandwidth of the B200 (MEASURED_PEAKS.json).
  cpu_baseline  the CPU checker (single thread, as it stands) on a column sample of the same
            workload, scaled to the full vector.

N > 1 runs N independent replicas of the workload, one process per GPU (launched by torchrun):
the path does not shard across GPUs and has no exchange step, so there is no collective in it.
--impl reference times the CPU checker instead (rank 0 only).
"""
import argparse
import json
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
# Arithmetic roofline of the local update: instruction issue.  One step of one Philox block
# (4 parameters) needs at least 76 warp instructions (9 Philox rounds x (2 wide multiplies +
# 2 three-input xors) = 36, Box-Muller for two pairs = 24, the rare-case test = 2, the update = 12,
# step loop = 2), i.e. 19 per parameter and step (ncu counts 78 in the kernel as it stands); an
# SM issues 4 x 32 = 128 lane-instructions per clock.
ALU_INSTR_PER_ELEM_STEP = 19.0
# The same count weighted by issue cost: integer and conversion instructions run on 16-lane pipes
# (64 results per clock and SM), so each holds the issue slot of its scheduler for two cycles.  Per
# Philox block and step: 18 wide multiplies + 18 xors + 2 compares + 1 add + 4 conversions = 43
# such instructions (86 slots) + 24 FP32 + 8 special-function + 1 branch = 119 slots, 29.75 per
# parameter and step.  ncu measures 117 cycles per block and step in the local-update kernel.
ALU_ISSUE_SLOTS_PER_ELEM_STEP = 29.75
SM_COUNT, LANES_PER_CLK_PER_SM, SM_MAX_GHZ = 148, 128, 1.965
ORACLE_NS_PER_ELEM_STEP = 45e-9   # rough cost of the CPU checker, used only to size its sample

# DRAM bytes per (device, parameter) moved by one launch, from the ncu captures summarised under
# profiles/ (dram__bytes_read.sum + dram__bytes_write.sum on a smaller case of the same kernel;
# reads grow in proportion to the elements processed; writes are undercounted by whatever is still
# dirty in the 126 MB L2 when the kernel ends).  None = not captured for the kernel as it stands.
NCU_DRAM_BYTES_PER_ELEM = {"round": 14.26, "local_step": 14.29, "aggregate": 4.58, "stats": 4.11}


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


# ---- CPU checker timing ------------------------------------------------------------------------
def time_oracle(wl, frac_cols, rounds):
    """Rounds of the CPU checker on the first `frac_cols` of the column groups; returns
    (seconds per full-vector round for each round, description of the sample)."""
    import oracle
    n_groups = (wl.n_params + 3) // 4
    take = min(n_groups, max(64, int(n_groups * frac_cols)))
    groups = np.arange(take, dtype=np.uint32)
    sim = oracle.Sim(wl.n_devices, wl.n_params, dtype=wl.dtype, momentum=wl.momentum,
                     weight_decay=wl.weight_decay, grad_std=wl.grad_std, init_std=wl.init_std,
                     seed=wl.seed, version_scale=wl.version_scale, weight_mode=wl.weight_mode,
                     groups=groups)
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
    return [t * scale for t in per_round], what


def run_reference(args, wl):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    # Bounded sample: size the column sample so that the whole run takes about a minute.
    total = args.warmup + args.steps
    full_round_s = wl.n_devices * wl.n_params * mean_steps_per_device(wl) * ORACLE_NS_PER_ELEM_STEP
    frac = min(1.0 / 8.0, 60.0 / (total * full_round_s))
    times, what = time_oracle(wl, frac, total)
    sec = float(np.mean(times[args.warmup:]))
    value = 1.0 / sec
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": describe(wl),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
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

    def __init__(self, index, period=0.02):
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

    # ---- timed region: K rounds, each ONE call of the public API (hadfl_round: local steps of
    # every device, selection, aggregation with write-back, version update, statistics) ----------
    ev_round = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                for _ in range(K)]
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(physical_gpu_index(local))
    step_lists = [wl.steps_for_round(r + i) for i in range(K)]
    syncs = [bool(wl.sync_every) and (r + i + 1) % wl.sync_every == 0 for i in range(K)]
    barrier()
    launches0 = h.launch_count()
    sampler.start()
    start.record()
    for i in range(K):
        a, b = ev_round[i]
        a.record(); h.round(ids, step_lists[i], wl.lr, r + i, k, seed, sync_all=syncs[i]); b.record()
    end.record()
    barrier()
    clocks = sampler.stop()
    launches = h.launch_count() - launches0
    r += K
    elapsed_ms = max_over_ranks(start.elapsed_time(end), world)
    mean_steps = float(np.mean([s.sum() for s in step_lists])) / N
    round_ms = float(np.mean([a.elapsed_time(b) for a, b in ev_round]))
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
    kernels = {"round": {"avg_ms": round_ms, "algorithmic_bytes": round_bytes,
                         "achieved_gbs": round_gbs, frac_key: round_gbs / peak,
                         "frac_of_8TBs": round_gbs / 8000.0, "mean_steps_per_device": mean_steps,
                         "gelem_steps_per_s": N * P * mean_steps / (round_ms * 1e-3) / 1e9,
                         "traffic": None if NCU_DRAM_BYTES_PER_ELEM["round"] is None
                         else NCU_DRAM_BYTES_PER_ELEM["round"] * N * P}}
    for n in names:
        gbs = alg_bytes[n] / (kern_ms[n] * 1e-3) / 1e9
        per_elem = NCU_DRAM_BYTES_PER_ELEM[n]
        kernels[n] = {"avg_ms": kern_ms[n], "algorithmic_bytes": alg_bytes[n], "achieved_gbs": gbs,
                      frac_key: gbs / peak, "frac_of_8TBs": gbs / 8000.0,
                      "share_of_separate_round": kern_ms[n] / sep_ms,
                      "traffic": None if per_elem is None else per_elem * units[n]}
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
    one_gbs = alg_bytes["local_step"] / (one_ms * 1e-3) / 1e9
    kernels["local_step_1_step_per_device"] = {
        "avg_ms": one_ms, "algorithmic_bytes": alg_bytes["local_step"], "achieved_gbs": one_gbs,
        frac_key: one_gbs / peak, "frac_of_8TBs": one_gbs / 8000.0,
        "traffic": NCU_DRAM_BYTES_PER_ELEM["local_step"] * N * P}
    kernels["local_step"]["mean_steps_per_device"] = sep_mean_steps
    kernels["local_step"]["gelem_steps_per_s"] = N * P * sep_mean_steps / (kern_ms["local_step"] * 1e-3) / 1e9
    separate = {"rounds_per_s": world * 1e3 / sep_ms, "ms_per_round": sep_ms, "rounds": Ks,
                "what": "hadfl_local_step + hadfl_select + hadfl_aggregate + hadfl_stats_enqueue"}
    alu_peak = SM_COUNT * LANES_PER_CLK_PER_SM * SM_MAX_GHZ / ALU_INSTR_PER_ELEM_STEP   # Gelem-step/s
    alu_achieved = kernels["round"]["gelem_steps_per_s"]
    alu_peak_weighted = SM_COUNT * LANES_PER_CLK_PER_SM * SM_MAX_GHZ / ALU_ISSUE_SLOTS_PER_ELEM_STEP
    hbm_src = ("of measured (copy bandwidth, MEASURED_PEAKS.json)" if peak_kind == "measured"
               else "of fallback (6650 GB/s)")
    # which floor is higher for this launch: bytes / HBM peak or element-steps / issue peak?
    t_hbm, t_alu = round_bytes / (peak * 1e9), N * P * mean_steps / (alu_peak * 1e9)
    if t_alu > t_hbm:
        roofline = {"kernel": "k_round (the whole round in one launch)", "bound": "alu",
                    "achieved": alu_achieved, "peak": alu_peak, "unit": "Gelem-step/s",
                    "frac": alu_achieved / alu_peak,
                    "peak_source": "derived: 148 SMs x 128 lane-instr/clk x 1.965 GHz / 19 "
                                   "instructions per parameter and step (instruction issue)",
                    "hbm_achieved_gbs": round_gbs, "hbm_peak_gbs": peak,
                    "hbm_frac": round_gbs / peak, "hbm_peak_source": hbm_src}
    else:
        roofline = {"kernel": "k_round (the whole round in one launch)", "bound": "hbm",
                    "achieved": round_gbs, "peak": peak, "unit": "GB/s", "frac": round_gbs / peak,
                    "peak_source": hbm_src, "alu_achieved_gelem_steps": alu_achieved,
                    "alu_peak_gelem_steps": alu_peak, "alu_frac": alu_achieved / alu_peak}
    roofline["alu_peak_half_rate_integer_gelem_steps"] = alu_peak_weighted
    roofline["alu_frac_half_rate_integer"] = alu_achieved / alu_peak_weighted
    roofline["traffic"] = kernels["round"]["traffic"]
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
    barrier()
    t0 = time.perf_counter()
    for i in range(Ke):
        sel = arena.run_round_fused(r + i)
        if i > 0:
            h.backup_wait()                    # the previous round's model has arrived
        n2, d2 = h.stats_read()
        h.backup_begin(int(sel[0]), host_model[i % 2])
    h.backup_wait()
    torch.cuda.synchronize()
    e2e_s = max_over_ranks(time.perf_counter() - t0, world)
    r += Ke
    barrier()
    t0 = time.perf_counter()
    for i in range(Ke):
        sel = arena.run_round_fused(r + i)
        n2, d2 = h.stats_read()
        h.read_params(int(sel[0]), out=host_model[0])
    torch.cuda.synchronize()
    blocking_s = max_over_ranks(time.perf_counter() - t0, world)
    r += Ke
    barrier()
    t0 = time.perf_counter()
    for i in range(Ke):
        arena.run_round_fused(r + i)
        n2, d2 = h.stats_read()            # waits for the round: no launch runs ahead of the host
    torch.cuda.synchronize()
    stats_only_s = max_over_ranks(time.perf_counter() - t0, world)
    r += Ke
    e2e = {"value": world * Ke / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "steps": Ke,
           "what": "hadfl_round + hadfl_stats_read + hadfl_backup_begin/wait(selected[0]) into pinned "
                   "host memory, the model transfer overlapping the next round",
           "blocking_value": world * Ke / blocking_s,
           "blocking_what": "the same with hadfl_read_params (waits for the transfer every round)",
           "stats_only_value": world * Ke / stats_only_s,
           "stats_only_what": "hadfl_round + hadfl_stats_read only (2N floats back per round, no model copy)"}

    line = {"metric": METRIC, "value": world * K / (elapsed_ms * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": K, "warmup": warmup,
            "ms_per_step": elapsed_ms / K, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": describe(wl),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "kernels": kernels, "separate_calls": separate}

    arena.close()
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        times, what = time_oracle(wl, 1.0 / 2.0, 3)
        line["cpu_baseline"] = {"value": 1.0 / float(np.mean(times)), "unit": UNIT, "cores": 1,
                                "kind": "oracle", "sample": what}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    wl = workloads.by_name(args.workload)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
