"""Drives the CPU oracle through the rounds of a workload (test-side only)."""
import numpy as np


def oracle_round(sim, wl, r):
    sim.local_step(wl.device_ids(), wl.steps_for_round(r), wl.lr)
    sel = sim.select(r, wl.k, wl.select_seed())
    sim.aggregate(sel)
    if wl.sync_every and (r + 1) % wl.sync_every == 0:
        others = np.setdiff1d(wl.device_ids(), sel).astype(np.int32)
        if wl.sync_beta == 1.0:
            sim.broadcast(int(sel[0]), others)
        else:
            sim.integrate(int(sel[0]), others, wl.sync_beta)
    return sel


def make_sim(oracle, wl, groups=None, openmp=False):
    """openmp=True: the oracle's -fopenmp build (same source, same results bit for bit -
    tests/test_oracle_openmp.py -, its column loops split over the host cores), for column samples
    too large for one core to follow in seconds."""
    return oracle.Sim(wl.n_devices, wl.n_params, dtype=wl.dtype, momentum=wl.momentum,
                      weight_decay=wl.weight_decay, grad_std=wl.grad_std, init_std=wl.init_std,
                      seed=wl.seed, version_scale=wl.version_scale, weight_mode=wl.weight_mode,
                      groups=groups, m_dtype=wl.m_dtype, rounding=wl.rounding, openmp=openmp)
