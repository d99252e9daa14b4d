"""Bandwidth and rounds/s tables over the workloads (the metric is quoted against P).

    python -m paper_2111_08274_b200.sweep [--what c5|configs|variants|sync|all] [--rounds 30] [--json out.json]

For every case: warm-up rounds, then `--rounds` timed rounds with CUDA events around each launch.
Prints markdown tables: per kernel the median launch time and the algorithmic GB/s (bytes that
must move / time), the rounds/s of the round as separate calls, and the rounds/s of the same
round through the fused kernel (its GB/s counts 16 bytes per device and parameter).  Small vectors (arena below the 126 MB L2)
are L2- and launch-bound and are reported as such, not as HBM bandwidth.
"""
import argparse
import json

import numpy as np
import torch

from . import runtime, workloads


def measure(wl, rounds, warmup=3):
    arena = runtime.Arena(wl)
    h = arena.h
    N, P, k = wl.n_devices, wl.n_params, wl.k
    ew = 2 if wl.dtype else 4
    em = 2 if wl.m_dtype else 4
    r = 0
    for _ in range(warmup):
        arena.run_round(r)
        r += 1
    names = ("local_step", "aggregate", "stats")
    ev = {n: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(rounds)] for n in names}
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    steps = [wl.steps_for_round(r + i) for i in range(rounds)]
    torch.cuda.synchronize()
    start.record()
    for i in range(rounds):
        a, b = ev["local_step"][i]
        a.record(); h.local_step(arena.ids, steps[i], wl.lr); b.record()
        sel = h.select(r + i, k, arena.select_seed)
        a, b = ev["aggregate"][i]
        a.record(); h.aggregate(sel); b.record()
        a, b = ev["stats"][i]
        a.record(); h.stats_enqueue(int(sel[0])); b.record()
    end.record()
    torch.cuda.synchronize()
    ms = {n: float(np.median([a.elapsed_time(b) for a, b in ev[n]])) for n in names}
    total_ms = start.elapsed_time(end) / rounds
    r += rounds
    # the same rounds through the fused kernel
    for i in range(warmup):
        arena.run_round_fused(r + i)
    r += warmup
    torch.cuda.synchronize()
    start.record()
    for i in range(0, rounds, 8):              # 8 rounds per library call: the per-call overhead is
        arena.run_rounds_fused(r + i, min(8, rounds - i))   # amortised, the launch queue stays shallow
    end.record()
    torch.cuda.synchronize()
    fused_ms = start.elapsed_time(end) / rounds
    bytes_ = {"local_step": N * P * 2 * (ew + em), "aggregate": 2 * k * P * ew, "stats": N * P * ew}
    arena.close()
    storage = ("bf16" if wl.dtype else "fp32") + ("+bf16 m" if wl.m_dtype else "") + (" sr" if wl.rounding else "")
    res = {"workload": wl.name, "N": N, "P": P, "k": k, "storage": storage,
           "mean_steps": float(np.mean([s.mean() for s in steps])),
           "arena_mb": N * P * (ew + em) / 1e6, "round_ms": total_ms, "rounds_per_s": 1e3 / total_ms,
           "fused_round_ms": fused_ms, "fused_rounds_per_s": 1e3 / fused_ms,
           "fused_gbs": N * P * 2 * (ew + em) / fused_ms / 1e6}
    for n in names:
        res[n + "_us"] = ms[n] * 1e3
        res[n + "_gbs"] = bytes_[n] / ms[n] / 1e6
    return res


def measure_sync(wl, reps=30):
    """Global synchronisation from device 0 to the N - k others: overwrite and beta-mix."""
    arena = runtime.Arena(wl)
    h = arena.h
    ew = 2 if wl.dtype else 4
    dst = np.arange(wl.k, wl.n_devices, dtype=np.int32)
    out = {"workload": wl.name, "N": wl.n_devices, "P": wl.n_params, "receivers": len(dst),
           "storage": "bf16" if wl.dtype else "fp32"}
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
        ms = a.elapsed_time(b) / reps
        out[name + "_us"] = ms * 1e3
        out[name + "_gbs"] = nbytes / ms / 1e6
    arena.close()
    return out


def table(rows, peak):
    out = ["| workload | N | P | k | storage | mean steps | arena MB | K1 µs | K1 GB/s (%% of %.0f) | K2 µs | K2 GB/s (%%) | K3 µs | K3 GB/s (%%) | round ms | rounds/s | fused round ms | fused rounds/s | fused GB/s (%%) |" % peak,
           "|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|"]
    for r in rows:
        out.append("| %s | %d | %d | %d | %s | %.2f | %.0f | %.1f | %.0f (%.0f) | %.1f | %.0f (%.0f) | %.1f | %.0f (%.0f) | %.3f | %.0f | %.3f | %.0f | %.0f (%.0f) |" % (
            r["workload"], r["N"], r["P"], r["k"], r["storage"], r["mean_steps"], r["arena_mb"],
            r["local_step_us"], r["local_step_gbs"], 100 * r["local_step_gbs"] / peak,
            r["aggregate_us"], r["aggregate_gbs"], 100 * r["aggregate_gbs"] / peak,
            r["stats_us"], r["stats_gbs"], 100 * r["stats_gbs"] / peak,
            r["round_ms"], r["rounds_per_s"], r["fused_round_ms"], r["fused_rounds_per_s"],
            r["fused_gbs"], 100 * r["fused_gbs"] / peak))
    return "\n".join(out)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--what", default="all", choices=["c5", "configs", "variants", "sync", "all"])
    ap.add_argument("--rounds", type=int, default=30)
    ap.add_argument("--peak", type=float, default=0.0, help="HBM GB/s to quote fractions of")
    ap.add_argument("--json", default="")
    a = ap.parse_args()
    peak = a.peak
    if not peak:
        try:
            import os
            with open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))),
                                   "MEASURED_PEAKS.json")) as f:
                peak = float(json.load(f)["hbm_gbs"])
        except Exception:
            peak = 6650.0
    runtime.ensure_built()
    rows = []
    if a.what in ("configs", "all"):
        for wl in (workloads.c1(), workloads.c2(), workloads.c3(), workloads.c4(2), workloads.c4(8),
                   workloads.c4(16)):
            rows.append(measure(wl, a.rounds))
        ones = workloads.Workload("c2_steps1", 8, 11_173_962, 4, 50, "fixed", (1,) * 8,
                                  seed=workloads.BASE_SEED + 2)
        rows.append(measure(ones, a.rounds))
    if a.what in ("c5", "all"):
        for dtype in (0, 1):
            for hetero in (False, True):
                for lp in range(16, 28):
                    rows.append(measure(workloads.c5(lp, dtype=dtype, hetero=hetero), a.rounds))
    if a.what in ("variants", "all"):
        # reduced-precision state next to bf16 parameters: bf16 momentum, stochastic rounding
        from dataclasses import replace
        for hetero in (False, True):
            for m_dtype, rounding in ((0, 0), (0, 1), (1, 0), (1, 1)):
                base = workloads.c5(25, dtype=1, hetero=hetero)
                name = base.name + ("_m16" if m_dtype else "") + ("_sr" if rounding else "")
                rows.append(measure(replace(base, name=name, m_dtype=m_dtype, rounding=rounding), a.rounds))
    sync_rows = []
    if a.what in ("sync", "all"):
        for wl in (workloads.c2(), workloads.c3(), workloads.c4(8), workloads.c5(25, dtype=1)):
            sync_rows.append(measure_sync(wl))
    if rows:
        print(table(rows, peak))
    if sync_rows:
        print("\n| workload | N | P | receivers | storage | broadcast µs | GB/s (%% of %.0f) | integrate µs | GB/s (%%) |" % peak)
        print("|---|---|---|---|---|---|---|---|---|")
        for r in sync_rows:
            print("| %s | %d | %d | %d | %s | %.1f | %.0f (%.0f) | %.1f | %.0f (%.0f) |" % (
                r["workload"], r["N"], r["P"], r["receivers"], r["storage"], r["broadcast_us"],
                r["broadcast_gbs"], 100 * r["broadcast_gbs"] / peak, r["integrate_us"],
                r["integrate_gbs"], 100 * r["integrate_gbs"] / peak))
        rows = rows + sync_rows
    if a.json:
        with open(a.json, "w") as f:
            json.dump(rows, f, indent=1)


if __name__ == "__main__":
    main()
