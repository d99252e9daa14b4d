"""Shared helpers of the GPU parity tests."""
import numpy as np
import pytest
import torch

from oracle_driver import make_sim, oracle_round

TOL_REL = 2e-6      # max|gpu - cpu| <= TOL_REL * max|x| for fp32 parameters


def require_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2111_08274_b200 import runtime
    runtime.ensure_built()


def assert_close_params(got, want, what=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    scale = np.abs(want).max()
    err = np.abs(got - want).max() if got.size else 0.0
    assert err <= TOL_REL * scale, "%s: max err %.3e > %.1e * %.3e" % (what, err, TOL_REL, scale)
    return err / scale if scale > 0 else 0.0


def bf16_ulp(x):
    """Spacing of bf16 numbers at |x| (fp32 array in, fp64 array out)."""
    bits = np.abs(np.asarray(x, dtype=np.float32)).view(np.uint32) & np.uint32(0x7F800000)
    e = (bits >> 23).astype(np.int32) - 127
    return np.ldexp(1.0, np.maximum(e, -126) - 7)


def columns_of(groups, n_params):
    cols = (4 * groups.astype(np.int64)[:, None] + np.arange(4)[None, :]).reshape(-1)
    return cols, cols < n_params


def compare_sample(arena, sim, groups, what):
    wl = arena.wl
    cols, live = columns_of(groups, wl.n_params)
    idx = torch.from_numpy(np.where(live, cols, 0)).to(arena.device)
    worst = 0.0
    for i in range(wl.n_devices):
        got = arena.w[i, idx].float().cpu().numpy()[live]
        want = sim.read_cols(i)[live]
        if wl.dtype == 0:
            worst = max(worst, assert_close_params(got, want, "%s w[%d]" % (what, i)))
        else:
            # A rounding decision that went the other way leaves a difference of one bf16 step of the
            # value at that time, which persists while the value itself moves on: bound it by two
            # steps at the largest magnitude in the row, and require such elements to be rare.
            assert np.abs(got - want).max() <= 2 * bf16_ulp(np.abs(want).max()), (what, i)
            assert np.mean(got != want) < 0.01, (what, i)
        gm = arena.m[i, idx].cpu().numpy()[live]
        # momentum sees the generator's error directly (not scaled by lr); with bf16 storage a
        # moved rounding of w also enters through weight decay
        m_tol = wl.grad_std * 1e-5 / (1.0 - wl.momentum) + (wl.weight_decay * 0.004 / (1.0 - wl.momentum) if wl.dtype else 0.0)
        assert np.abs(gm - sim.read_momentum_cols(i)[live]).max() <= m_tol, (what, i)
    return worst


def run_and_compare(oracle, wl, groups, check_rounds, stats_rounds=(), fused=False, openmp=False):
    from paper_2111_08274_b200 import runtime
    arena = runtime.Arena(wl)
    sim = make_sim(oracle, wl, groups, openmp=openmp)
    full = groups is None
    g = np.arange((wl.n_params + 3) // 4, dtype=np.uint32) if full else groups
    worst = 0.0
    for r in range(wl.rounds):
        sel = arena.run_round_fused(r) if fused else arena.run_round(r)
        want_sel = oracle_round(sim, wl, r)
        assert np.array_equal(sel, want_sel), "round %d: selection %s != %s" % (r, sel, want_sel)
        v, s = arena.h.get_versions()
        ov, os_ = sim.get_versions()
        assert np.array_equal(v, ov) and np.array_equal(s, os_), "round %d: counters differ" % r
        if r in check_rounds or r == wl.rounds - 1:
            worst = max(worst, compare_sample(arena, sim, g, "%s round %d" % (wl.name, r)))
        if full and (r in stats_rounds or r == wl.rounds - 1):
            n2, d2 = arena.h.stats_read()
            wn2, wd2 = sim.stats(int(sel[0]))
            assert np.allclose(n2, wn2, rtol=1e-5) and np.allclose(d2, wd2, rtol=1e-5, atol=1e-12)
    n2, d2 = arena.h.stats_read()
    assert np.all(np.isfinite(n2)) and np.all(d2 >= 0) and d2[int(sel[0])] == 0.0
    launches = arena.h.launch_count()
    arena.h.debug_check()      # debug build: no kernel skipped an out-of-range access (no-op otherwise)
    arena.close()
    print("%s: %d rounds ok, max err / max|x| = %.2e, %d launches" % (wl.name, wl.rounds, worst, launches))
    return worst
