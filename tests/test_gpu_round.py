"""The fused round kernel (hadfl_round) against the separate calls it replaces and against the CPU
oracle: selections, versions, parameters and momentum must equal the unfused sequence bit for bit;
its statistics agree with the oracle's double-precision sums to 1e-5."""
import numpy as np
import pytest
import torch

from gpu_common import assert_close_params, bf16_ulp, require_gpu
from oracle_driver import make_sim, oracle_round
from paper_2111_08274_b200 import binding, runtime, workloads
from paper_2111_08274_b200.workloads import Workload

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def wl_of(n, P, k, dtype=0, steps=None, sync_every=0, **kw):
    steps = tuple(1 + (3 * i) % 5 for i in range(n)) if steps is None else steps
    return Workload("rt", n, P, k, 6, "fixed", steps, grad_std=1e-2, dtype=dtype,
                    seed=workloads.BASE_SEED + 31 * n + P, sync_every=sync_every, **kw)


def assert_same_state(a, b, n):
    for i in range(n):
        assert np.array_equal(a.h.read_params(i), b.h.read_params(i)), i
        assert np.array_equal(a.h.read_momentum(i), b.h.read_momentum(i)), i
    va, vb = a.h.get_versions(), b.h.get_versions()
    assert np.array_equal(va[0], vb[0]) and np.array_equal(va[1], vb[1])


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("n,P,k", [(4, 100_003, 2), (8, 70_001, 4), (16, 33_333, 1), (32, 9_999, 16),
                                   (32, 4_099, 32), (1, 5, 1), (5, 1, 3), (6, 300_007, 3)])
def test_fused_round_equals_separate_calls(oracle, n, P, k, dtype):
    wl = wl_of(n, P, k, dtype=dtype, sync_every=3)
    fused, plain = runtime.Arena(wl), runtime.Arena(wl)
    sim = make_sim(oracle, wl)
    for r in range(wl.rounds):
        sf = fused.run_round_fused(r)
        sp = plain.run_round(r)
        so = oracle_round(sim, wl, r)
        assert np.array_equal(sf, sp) and np.array_equal(sf, so), r
        n2, d2 = fused.h.stats_read()
        pn2, pd2 = plain.h.stats_read()
        on2, od2 = sim.stats(int(so[0]))
        assert np.allclose(n2, pn2, rtol=2e-6) and np.allclose(d2, pd2, rtol=2e-6, atol=1e-30), r
        if dtype == 0:
            assert np.allclose(n2, on2, rtol=1e-5) and np.allclose(d2, od2, rtol=1e-5, atol=1e-12), r
        assert all(d2[int(s)] == 0.0 for s in sf)
    assert_same_state(fused, plain, n)
    if dtype == 0:
        for i in range(n):
            assert_close_params(fused.h.read_params(i), sim.read_params(i), "w[%d]" % i)
    else:
        for i in range(n):
            got, want = fused.h.read_params(i), sim.read_params(i)
            assert np.abs(got - want).max() <= 2 * bf16_ulp(np.abs(want).max()) and np.mean(got != want) < 0.02
    fused.close()
    plain.close()


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("n,P,k,beta", [(6, 50_003, 2, 0.25), (8, 9_999, 4, 0.5), (5, 7, 1, 0.9), (4, 3_001, 4, 0.3)])
def test_fused_round_with_mixed_global_synchronisation(oracle, n, P, k, beta, dtype):
    """Global-synchronisation rounds that mix the aggregate into the unselected devices' own models
    (hadfl_set_sync_beta) instead of overwriting them: the fused kernel against the separate calls
    (hadfl_integrate) bit for bit, selections and versions against the oracle."""
    wl = wl_of(n, P, k, dtype=dtype, sync_every=2, sync_beta=beta)
    fused, plain = runtime.Arena(wl), runtime.Arena(wl)
    sim = make_sim(oracle, wl)
    for r in range(wl.rounds):
        sf, sp, so = fused.run_round_fused(r), plain.run_round(r), oracle_round(sim, wl, r)
        assert np.array_equal(sf, sp) and np.array_equal(sf, so), r
        assert np.array_equal(fused.h.get_versions()[0], sim.get_versions()[0]), r
        n2, d2 = fused.h.stats_read()
        pn2, pd2 = plain.h.stats_read()
        assert np.allclose(n2, pn2, rtol=2e-6) and np.allclose(d2, pd2, rtol=2e-6, atol=1e-30), r
    assert_same_state(fused, plain, n)
    for i in range(n):
        got, want = fused.h.read_params(i), sim.read_params(i)
        if dtype == 0:
            assert_close_params(got, want, "w[%d]" % i)
        else:
            assert np.abs(got - want).max() <= 2 * bf16_ulp(np.abs(want).max()) and np.mean(got != want) < 0.02
    with pytest.raises(binding.HadflError):
        fused.h.set_sync_beta(1.5)
    fused.close()
    plain.close()


@pytest.mark.parametrize("dtype,m_dtype,rounding", [(0, 0, 0), (1, 0, 0), (1, 1, 0), (1, 0, 1), (1, 1, 1)])
@pytest.mark.parametrize("n,P,k,beta", [(6, 70_003, 2, 1.0), (16, 9_999, 4, 0.5), (3, 300_007, 3, 1.0), (5, 7, 1, 0.25)])
def test_fused_round_when_no_device_runs_more_than_two_steps(oracle, n, P, k, beta, dtype, m_dtype, rounding):
    """At most two steps per device is the memory-bound regime, for which the library picks other
    launch shapes (one row per block in the local update; with bf16 parameters a build of the fused
    round that loads the next row ahead).  Some devices run no step at all; every second round is a
    global synchronisation (overwrite or mix).  Fused round against the separate calls bit for bit,
    selections and versions against the oracle, parameters within the storage's tolerance."""
    steps = tuple((i * 5 + 1) % 3 for i in range(n))          # 0, 1 and 2 steps
    wl = wl_of(n, P, k, dtype=dtype, steps=steps, sync_every=2, sync_beta=beta, m_dtype=m_dtype, rounding=rounding)
    fused, plain = runtime.Arena(wl), runtime.Arena(wl)
    sim = make_sim(oracle, wl)
    for r in range(wl.rounds):
        sf, sp, so = fused.run_round_fused(r), plain.run_round(r), oracle_round(sim, wl, r)
        assert np.array_equal(sf, sp) and np.array_equal(sf, so), r
        assert np.array_equal(fused.h.get_versions()[0], sim.get_versions()[0]), r
        n2, d2 = fused.h.stats_read()
        pn2, pd2 = plain.h.stats_read()
        assert np.allclose(n2, pn2, rtol=2e-6) and np.allclose(d2, pd2, rtol=2e-6, atol=1e-30), r
    assert_same_state(fused, plain, n)
    for i in range(n):
        got, want = fused.h.read_params(i), sim.read_params(i)
        if dtype == 0:
            assert_close_params(got, want, "w[%d]" % i)
        else:
            assert np.abs(got - want).max() <= 2 * bf16_ulp(np.abs(want).max()) and np.mean(got != want) < 0.02
    fused.h.debug_check()
    fused.close()
    plain.close()


@pytest.mark.parametrize("dtype,steps_hi", [(0, 8), (1, 8), (1, 2)])
def test_a_run_of_rounds_in_one_call_equals_the_rounds_one_by_one(dtype, steps_hi):
    from dataclasses import replace
    wl = replace(workloads.shrink(workloads.c2(), 30_011, rounds=9), dtype=dtype, sync_every=4, steps_hi=steps_hi)
    one, many = runtime.Arena(wl), runtime.Arena(wl)
    want = np.stack([one.run_round_fused(r) for r in range(wl.rounds)])
    got = np.concatenate([many.run_rounds_fused(0, 5), many.run_rounds_fused(5, 4)])
    assert np.array_equal(got, want)
    assert_same_state(one, many, wl.n_devices)
    a, b = one.h.stats_read(), many.h.stats_read()
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert many.h.rounds(9, np.zeros((0, wl.n_devices), dtype=np.int32), wl.lr, wl.k, 1).shape == (0, wl.k)
    with pytest.raises(binding.HadflError):
        many.h.rounds(9, np.ones((2, wl.n_devices + 1), dtype=np.int32), wl.lr, wl.k, 1)
    with pytest.raises(binding.HadflError):
        many.h.rounds(9, np.ones((2, wl.n_devices), dtype=np.int32), wl.lr, wl.n_devices + 1, 1)
    one.close()
    many.close()


def test_fused_round_subset_of_devices_zero_steps_mask_and_versions(oracle):
    """Only some devices step, one of them zero steps; an availability mask; caller-supplied versions."""
    wl = wl_of(6, 20_003, 2)
    fused, plain = runtime.Arena(wl), runtime.Arena(wl)
    mask = [1, 1, 0, 1, 1, 1]
    for ar in (fused, plain):
        ar.h.set_available(mask)
    ids, steps = [4, 0, 2], [3, 0, 2]
    pv = [2.0, 2.5, 9.0, 1.0, 3.0, 3.0]
    for r, versions in ((0, None), (1, pv), (2, None)):
        sf = fused.h.round(ids, steps, 0.01, r, 2, 77, versions=versions)
        plain.h.local_step(ids, steps, 0.01)
        sp = plain.h.select(r, 2, 77, versions)
        plain.h.aggregate(sp, versions)
        plain.h.stats_enqueue(int(sp[0]))
        assert np.array_equal(sf, sp) and 2 not in sf
        a, b = fused.h.stats_read(), plain.h.stats_read()
        assert np.allclose(a[0], b[0], rtol=2e-6) and np.allclose(a[1], b[1], rtol=2e-6, atol=1e-30)
    assert_same_state(fused, plain, 6)
    fused.close()
    plain.close()


def test_fused_round_version_weighted_mode():
    wl = wl_of(8, 12_345, 4, weight_mode=1, version_scale=0.5)
    fused, plain = runtime.Arena(wl), runtime.Arena(wl)
    for r in range(4):
        assert np.array_equal(fused.run_round_fused(r), plain.run_round(r))
    assert_same_state(fused, plain, 8)
    fused.close()
    plain.close()


def test_fused_round_is_reproducible_and_rejects_bad_arguments():
    wl = wl_of(8, 50_001, 4)
    a, b = runtime.Arena(wl), runtime.Arena(wl)
    for r in range(3):
        a.run_round_fused(r)
        b.run_round_fused(r)
        sa, sb = a.h.stats_read(), b.h.stats_read()
        assert np.array_equal(sa[0], sb[0]) and np.array_equal(sa[1], sb[1])     # bit for bit
    assert_same_state(a, b, 8)
    before = a.h.read_params(3)
    E = binding.HadflError
    for ids, steps, k in (([0, 0], [1, 1], 2), ([8], [1], 2), ([0], [-1], 2), ([0], [1], 0), ([0], [1], 9), ([], [], 2)):
        with pytest.raises(E):
            a.h.round(ids, steps, 0.01, 5, k, 1)
    assert np.array_equal(a.h.read_params(3), before)
    a.close()
    b.close()


def test_fused_round_counter_crossing_falls_back_to_separate_kernels():
    wl = wl_of(3, 4_099, 2)
    fused, plain = runtime.Arena(wl), runtime.Arena(wl)
    start = np.array([2**32 - 2, 5, 2**33 - 1], dtype=np.uint64)
    for ar in (fused, plain):
        ar.h.set_versions(step_counts=start)
    sf = fused.run_round_fused(0)
    sp = plain.run_round(0)
    assert np.array_equal(sf, sp)
    assert_same_state(fused, plain, 3)
    fused.close()
    plain.close()


# ---- several rounds per launch ---------------------------------------------------------------------
def _launches(ar, fn):
    before = ar.h.launch_count()
    out = fn()
    return out, ar.h.launch_count() - before


@pytest.mark.parametrize("dtype,m_dtype,rounding", [(0, 0, 0), (1, 0, 0), (1, 1, 0), (1, 0, 1), (1, 1, 1)])
@pytest.mark.parametrize("n,P,k,sync_every,beta", [(4, 100_003, 2, 0, 1.0), (8, 70_001, 4, 3, 0.5),
                                                  (16, 9_999, 1, 4, 1.0), (32, 2_049, 16, 0, 1.0), (5, 7, 5, 2, 0.25)])
def test_batched_rounds_equal_the_rounds_launched_one_by_one(n, P, k, sync_every, beta, dtype, m_dtype, rounding):
    """A small arena: hadfl_rounds puts up to 8 rounds into one launch.  Parameters, momentum, counters,
    selections and EVERY round's statistics must equal those of single launches, bit for bit."""
    steps = tuple((5 * i + 1) % 4 for i in range(n))  # 0 .. 3 steps, some devices idle
    wl = wl_of(n, P, k, dtype=dtype, steps=steps, sync_every=sync_every, sync_beta=beta, m_dtype=m_dtype,
               rounding=rounding)
    single, batched = runtime.Arena(wl), runtime.Arena(wl)
    assert batched.h.round_batch() == 8
    single.h.set_round_batch(1)
    stats_single = []
    want = []
    for r in range(19):
        want.append(single.run_round_fused(r))
        stats_single.append(single.h.stats_read())
    got = []
    for first, count in ((0, 8), (8, 8), (16, 3)):
        sel, launches = _launches(batched, lambda: batched.run_rounds_fused(first, count))
        assert launches == 1
        got.append(sel)
        for back in range(count):
            a = batched.h.stats_read_round(back)
            b = stats_single[first + count - 1 - back]
            assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]), (first, back)
        with pytest.raises(binding.HadflError):
            batched.h.stats_read_round(count)
    assert np.array_equal(np.concatenate(got), np.stack(want))
    assert_same_state(single, batched, n)
    # the same through hadfl_rounds with batching switched off: one launch per round
    off = runtime.Arena(wl)
    off.h.set_round_batch(1)
    sel, launches = _launches(off, lambda: off.run_rounds_fused(0, 19))
    assert launches == 19 and np.array_equal(sel, np.stack(want))
    assert_same_state(single, off, n)
    for ar in (single, batched, off):
        ar.h.debug_check()  # debug build: no kernel skipped an out-of-range access (no-op otherwise)
        ar.close()


@pytest.mark.parametrize("dtype", [0, 1])
def test_batching_rule_on_an_arena_larger_than_the_small_arena_bound(dtype):
    """Beyond 64 MiB only rounds in which no device runs more than two steps are batched."""
    n, P, k = 8, 1_300_003, 4  # fp32: 83 MB, bf16 parameters: 62 MB of parameters and momentum
    if dtype == 1:
        P = 2_000_003  # 96 MB
    light = np.array([1, 2, 0, 1, 2, 2, 1, 1], dtype=np.int32)
    heavy = np.array([1, 3, 0, 1, 2, 2, 1, 1], dtype=np.int32)
    steps = np.stack([light, light, light, heavy, light, light, heavy, heavy, light])
    # launches: [0 1 2] [3] [4 5] [6] [7] [8]
    wl = Workload("rule", n, P, k, 9, "fixed", tuple(light), grad_std=1e-2, dtype=dtype, seed=workloads.BASE_SEED + 77,
                  sync_every=4)
    single, batched = runtime.Arena(wl), runtime.Arena(wl)
    want = np.stack([single.h.round(single.ids, steps[r], wl.lr, r, k, single.select_seed,
                                    sync_all=(r + 1) % 4 == 0) for r in range(9)])
    got, launches = _launches(batched, lambda: batched.h.rounds(0, steps, wl.lr, k, batched.select_seed, 4))
    assert launches == 6
    assert np.array_equal(got, want)
    batched.h.synchronize()
    single.h.synchronize()
    assert torch.equal(single.w, batched.w) and torch.equal(single.m, batched.m)
    a, b = single.h.stats_read(), batched.h.stats_read()
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    batched.h.set_round_batch(2)
    _, launches = _launches(batched, lambda: batched.h.rounds(9, steps[:3], wl.lr, k, batched.select_seed, 4))
    assert launches == 2
    for bad in (0, 9, -1):
        with pytest.raises(binding.HadflError):
            batched.h.set_round_batch(bad)
    assert batched.h.round_batch() == 2
    single.close()
    batched.close()
    if dtype == 0:  # fp32, at most 1.5 steps per device on average: the batch takes packs of 4 columns
        ones = np.ones((5, n), dtype=np.int32)
        a4, a1 = runtime.Arena(wl), runtime.Arena(wl)
        a1.h.set_round_batch(1)
        assert a4.h.last_round_pack() == 0
        got, launches = _launches(a4, lambda: a4.h.rounds(0, ones, wl.lr, k, a4.select_seed, 2))
        assert launches == 1 and a4.h.last_round_pack() == 4
        want = a1.h.rounds(0, ones, wl.lr, k, a1.select_seed, 2)
        assert a1.h.last_round_pack() == 8 and np.array_equal(got, want)
        a4.h.synchronize()
        a1.h.synchronize()
        assert torch.equal(a4.w, a1.w) and torch.equal(a4.m, a1.m)
        for back in range(5):
            x, y = a4.h.stats_read_round(back), (a1.h.stats_read() if back == 0 else None)
            assert np.all(np.isfinite(x[0])) and np.all(x[1] >= 0)
            if y is not None:
                assert np.allclose(x[0], y[0], rtol=2e-6) and np.allclose(x[1], y[1], rtol=2e-6, atol=1e-30)
        a4.h.rounds(5, steps[:2], wl.lr, k, a4.select_seed, 2)  # 1.25 steps per device on average: still packs of 4
        assert a4.h.last_round_pack() == 4
        a4.h.rounds(7, np.full((2, n), 2, dtype=np.int32), wl.lr, k, a4.select_seed, 2)  # two steps each: packs of 8
        assert a4.h.last_round_pack() == 8
        a4.h.debug_check()
        a4.close()
        a1.close()
    if dtype == 1:  # stochastic rounding draws a second random block per pack: launched one by one
        from dataclasses import replace
        sr = runtime.Arena(replace(wl, rounding=1))
        _, launches = _launches(sr, lambda: sr.h.rounds(0, steps[:3], wl.lr, k, sr.select_seed, 4))
        assert launches == 3
        sr.close()


def test_batched_rounds_with_a_step_counter_crossing_2_to_the_32():
    """The round in which a counter crosses a multiple of 2^32 leaves the batch (separate kernels); the
    rounds before and after it are batched around it."""
    wl = wl_of(3, 4_099, 2, steps=(2, 1, 3))
    batched, plain = runtime.Arena(wl), runtime.Arena(wl)
    start = np.array([2**32 - 5, 5, 2**33 - 7], dtype=np.uint64)  # device 0 crosses in round 2, device 2 in round 2
    for ar in (batched, plain):
        ar.h.set_versions(step_counts=start)
    got, launches = _launches(batched, lambda: batched.run_rounds_fused(0, 6))
    want = np.stack([plain.run_round(r) for r in range(6)])
    assert np.array_equal(got, want)
    assert_same_state(batched, plain, 3)
    assert launches > 2  # two batches and the kernels of the crossing round in between
    batched.close()
    plain.close()
