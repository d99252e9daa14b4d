"""Runs a workload round by round on one GPU and logs what the coordinator of the paper would see.

    python -m paper_2111_08274_b200.run [--workload c1] [--rounds R] [--n-params P] [--separate]
                                        [--predict ALPHA] [--jsonl out.jsonl]

Every round is one hadfl_round call (or, with --separate, the four separate calls).  Per round one
JSON line: the selected devices in draw order, every device's version and step counter, the
selection probabilities of Eq. 8 the draw was made from, per-replica squared norm and squared
distance to the aggregate, and the time the round took on the GPU (CUDA events).

--predict ALPHA plans the selection with predicted instead of actual versions, as the paper's
strategy generator does (Section "Runtime information prediction", Eq. 7): each device's version
history is smoothed twice with factor ALPHA and extrapolated one round ahead (hadfl_predict_version);
the first two rounds use the actual versions.  Arithmetic happens in the library; this module
only moves arrays and writes the log.
"""
import argparse
import json
import sys

import numpy as np
import torch

from . import binding, runtime, workloads


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c1")
    ap.add_argument("--rounds", type=int, default=0, help="0 = the workload's own round count")
    ap.add_argument("--n-params", type=int, default=0, help="0 = the workload's own vector length")
    ap.add_argument("--separate", action="store_true", help="four separate calls instead of hadfl_round")
    ap.add_argument("--predict", type=float, default=0.0, help="smoothing factor of Eq. 7 (0 = use actual versions)")
    ap.add_argument("--jsonl", default="", help="file to write (default: standard output)")
    a = ap.parse_args(argv)

    wl = workloads.by_name(a.workload)
    if a.n_params or a.rounds:
        wl = workloads.shrink(wl, a.n_params or wl.n_params, a.rounds or wl.rounds)
    runtime.ensure_built()
    arena = runtime.Arena(wl)
    h = arena.h
    out = open(a.jsonl, "w") if a.jsonl else sys.stdout
    history = [[] for _ in range(wl.n_devices)]
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for r in range(wl.rounds):
        steps = wl.steps_for_round(r)
        planned = None
        if a.predict > 0.0 and r >= 2:
            # what each device's version is expected to be when this round synchronises
            planned = np.array([binding.hadfl_predict_version(history[i], a.predict, 1.0)
                                for i in range(wl.n_devices)], dtype=np.float64)
        sync = bool(wl.sync_every) and (r + 1) % wl.sync_every == 0
        start.record(arena.stream)
        if a.separate:
            h.local_step(arena.ids, steps, wl.lr)
            probs = h.select_probs(planned)
            sel = h.select(r, wl.k, arena.select_seed, planned)
            h.aggregate(sel, planned)
            if sync:
                others = np.setdiff1d(arena.ids, sel).astype(np.int32)
                if wl.sync_beta == 1.0:
                    h.broadcast(int(sel[0]), others)
                else:
                    h.integrate(int(sel[0]), others, wl.sync_beta)
            h.stats_enqueue(int(sel[0]))
        else:
            probs = h.select_probs(planned) if planned is not None else h.select_probs_after(arena.ids, steps)
            sel = h.round(arena.ids, steps, wl.lr, r, wl.k, arena.select_seed, versions=planned,
                          sync_all=sync)
        end.record(arena.stream)
        n2, d2 = h.stats_read()
        versions, counters = h.get_versions()
        for i in range(wl.n_devices):
            history[i].append(float(versions[i]))
        json.dump({"round": r, "selected": [int(s) for s in sel], "steps": [int(s) for s in steps],
                   "versions": [int(v) for v in versions], "step_counters": [int(c) for c in counters],
                   "planned_versions": None if planned is None else [float(x) for x in planned],
                   "selection_probabilities": [float(p) for p in probs],
                   "norm2": [float(x) for x in n2], "divergence2": [float(x) for x in d2],
                   "global_sync": sync, "gpu_ms": float(start.elapsed_time(end))}, out)
        out.write("\n")
    if a.jsonl:
        out.close()
    arena.close()


if __name__ == "__main__":
    main()
