"""Runs a small, fixed case of every kernel a few times: the target of `ncu` captures.

    python -m paper_2111_08274_b200.profile_case [--n 8] [--p 4194306] [--k 4] [--steps 1,8]
                                                 [--dtype 0] [--reps 2]

The arena (N * P * 8 bytes for fp32) should exceed the 126 MB L2 so that DRAM counters mean
something, and stay at a few hundred MB so that a multi-pass capture ends quickly.
Launch order per repetition: local update once per entry of --steps (all devices that many
steps), aggregation of k devices, statistics, broadcast to the other devices, the same as a mix
(beta = 1/2).  With --fused: one
hadfl_round launch per entry of --steps instead.
"""
import argparse

import numpy as np

from . import runtime, workloads


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--n", type=int, default=8)
    ap.add_argument("--p", type=int, default=4 * 1024 * 1024 + 2)
    ap.add_argument("--k", type=int, default=4)
    ap.add_argument("--steps", type=str, default="1,8")
    ap.add_argument("--dtype", type=int, default=0)
    ap.add_argument("--reps", type=int, default=2)
    ap.add_argument("--fused", action="store_true", help="run hadfl_round instead of the separate calls")
    a = ap.parse_args()
    wl = workloads.Workload("profile", a.n, a.p, a.k, 1, "fixed", (1,) * a.n, dtype=a.dtype,
                            seed=workloads.BASE_SEED)
    runtime.ensure_built()
    ar = runtime.Arena(wl)
    ids = wl.device_ids()
    sel = ids[: a.k]
    for rep in range(a.reps if a.fused else 0):
        for s in [int(t) for t in a.steps.split(",")]:
            ar.h.round(ids, np.full(a.n, s, dtype=np.int32), wl.lr, rep, a.k, 1)
    for _ in range(0 if a.fused else a.reps):
        for s in [int(t) for t in a.steps.split(",")]:
            ar.h.local_step(ids, np.full(a.n, s, dtype=np.int32), wl.lr)
        ar.h.aggregate(sel)
        ar.h.stats_enqueue(int(sel[0]))
        ar.h.broadcast(int(sel[0]), ids[a.k:])
        ar.h.integrate(int(sel[0]), ids[a.k:], 0.5)
    ar.h.synchronize()
    n2, d2 = ar.h.stats_read()
    print("ok: launches=%d norm2[0]=%.6g" % (ar.h.launch_count(), n2[0]))
    ar.close()


if __name__ == "__main__":
    main()
