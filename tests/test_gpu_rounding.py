"""GPU parity of the reduced-precision state (bf16 momentum, stochastic rounding of the local
update's bf16 stores; a workload variant outside the paper, which trains in fp32) against the CPU
oracle.  Without gradient noise both sides run the same fp32 arithmetic and draw the same rounding
bits, so every stored value must agree bit for bit; with noise the generator's last-bit
differences can flip a rounding decision, which the tests bound as for plain bf16 storage."""
import numpy as np
import pytest
import torch

from gpu_common import bf16_ulp, require_gpu
from oracle_driver import make_sim, oracle_round
from paper_2111_08274_b200 import binding, runtime, workloads
from paper_2111_08274_b200.workloads import Workload

pytestmark = pytest.mark.gpu

MODES = [(0, 1), (1, 0), (1, 1)]      # (m_dtype, rounding); (0, 0) is covered by the other files


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def wl_of(n, P, m_dtype, rounding, **kw):
    args = dict(name="r", n_devices=n, n_params=P, k=min(2, n), rounds=4, steps_rule="fixed",
                steps_fixed=tuple(1 + (2 * i) % 5 for i in range(n)), grad_std=1e-2, dtype=1,
                m_dtype=m_dtype, rounding=rounding, seed=0xBF16 + 7 * P + m_dtype + 2 * rounding)
    args.update(kw)
    return Workload(**args)


def load_rows(h, sim, rows, momentum=None):
    for i in range(rows.shape[0]):
        h.write_params(i, rows[i])
        sim.write_params(i, rows[i])
        if momentum is not None:
            h.write_momentum(i, momentum[i])
            sim.write_momentum(i, momentum[i])


def test_rounding_words_are_the_generator_on_the_stated_counter(oracle):
    h = binding.Hadfl(1, 8)
    seed = 0x0123456789ABCDEF
    key = np.array([seed & 0xFFFFFFFF, seed >> 32], dtype=np.uint32)
    cases = [(0, 0, 0), (5, 17, 3), (2**32 - 1, 2**40 + 9, 31), (77, 2**32 - 1, 1)]
    ctr = np.array([[g, s & 0xFFFFFFFF, d, 0x52000000 | (s >> 32)] for g, s, d in cases], dtype=np.uint32)
    got = h.debug_philox(ctr, key)
    for row, (g, s, d) in zip(got, cases):
        assert np.array_equal(row, oracle.rounding_words(seed, g, s, d))


@pytest.mark.parametrize("m_dtype,rounding", MODES)
@pytest.mark.parametrize("P", [1, 6, 1023, 4099, 70_001])
def test_local_step_without_noise_is_bit_exact(oracle, P, m_dtype, rounding):
    """grad_std = 0: pure fp32 fma arithmetic, then the rounding under test - every stored bit of
    the parameters and of the momentum must equal the oracle's, call after call."""
    n = 4
    wl = wl_of(n, P, m_dtype, rounding, grad_std=0.0, weight_decay=0.3, momentum=0.9)
    h, sim = binding.Hadfl.from_workload(wl), make_sim(oracle, wl)
    rows = workloads.random_rows(n, P, seed=P + 1)
    mom = workloads.random_rows(n, P, seed=P + 2, std=0.01)
    load_rows(h, sim, rows, mom)
    # step counters next to a multiple of 2^32 (without crossing it) and beyond it: the rounding
    # block is indexed by the last step of the call
    start = np.array([2**32 - 9, 2**40 + 3, 0, 5], dtype=np.uint64)
    h.set_versions(step_counts=start)
    sim.set_versions(step_counts=start)
    for ids, steps in [([0, 1, 2, 3], [1, 2, 3, 4]), ([2, 0], [5, 0]), ([3], [1]), ([1, 3, 0, 2], [2, 1, 2, 7])]:
        h.local_step(ids, steps, 0.05)
        sim.local_step(ids, steps, 0.05)
        for i in range(n):
            assert np.array_equal(h.read_params(i), sim.read_params(i)), (ids, i)
            assert np.array_equal(h.read_momentum(i), sim.read_momentum(i)), (ids, i)
    assert np.array_equal(h.get_versions()[1], sim.get_versions()[1])


@pytest.mark.parametrize("m_dtype,rounding", [(0, 0)] + MODES)
def test_a_call_that_crosses_a_multiple_of_two_to_the_32_steps_rounds_where_it_is_split(oracle, m_dtype, rounding):
    """The kernels take the high word of a device's step index as fixed per launch, so a call whose
    step counter crosses a multiple of 2^32 runs as two launches - and with bf16 storage the values
    are rounded at the end of each.  The documented behaviour is therefore that of the SAME steps
    given as two calls (up to the crossing, beyond it): pinned here bit for bit, without gradient
    noise, against the oracle driven that way; the oracle's single call (one rounding) may differ
    from it by at most one bf16 step."""
    n, P = 3, 4099
    wl = wl_of(n, P, m_dtype, rounding, grad_std=0.0, weight_decay=0.3, momentum=0.9)
    h, two_calls, one_call = binding.Hadfl.from_workload(wl), make_sim(oracle, wl), make_sim(oracle, wl)
    rows = workloads.random_rows(n, P, seed=91)
    mom = workloads.random_rows(n, P, seed=92, std=0.01)
    for sim in (two_calls, one_call):
        load_rows(h, sim, rows, mom)
    start = np.array([2**32 - 2, 7, 2**33 - 1], dtype=np.uint64)
    for x in (h, two_calls, one_call):
        x.set_versions(step_counts=start)
    ids, steps = [0, 1, 2], [5, 3, 4]
    h.local_step(ids, steps, 0.05)
    two_calls.local_step(ids, [2, 3, 1], 0.05)          # up to the crossing (device 1 does not cross)
    two_calls.local_step([0, 2], [3, 3], 0.05)          # beyond it
    one_call.local_step(ids, steps, 0.05)
    assert np.array_equal(h.get_versions()[1], two_calls.get_versions()[1])
    assert np.array_equal(h.get_versions()[1], one_call.get_versions()[1])
    for i in range(n):
        got_w, got_m = h.read_params(i), h.read_momentum(i)
        assert np.array_equal(got_w, two_calls.read_params(i)), i
        assert np.array_equal(got_m, two_calls.read_momentum(i)), i
        once = one_call.read_params(i)
        assert np.abs(got_w - once).max() <= bf16_ulp(np.abs(once).max()), i
    assert np.array_equal(h.read_params(1), one_call.read_params(1))       # no crossing, no split
    h.destroy()


def test_stochastic_rounding_moves_where_nearest_even_stalls(oracle):
    """Weight decay only, lr wd = 1e-3 < half a bf16 spacing: nearest-even storage never moves,
    stochastic storage follows the oracle bit for bit (whose mean is pinned to the closed form)."""
    n, lr, wd, T = 4000, 0.1, 0.01, 40
    base = dict(grad_std=0.0, momentum=0.0, weight_decay=wd, steps_fixed=(1,), k=1)
    w0 = np.full(n, 0.4, dtype=np.float32)
    for rounding in (0, 1):
        wl = wl_of(1, n, 0, rounding, **base)
        h, sim = binding.Hadfl.from_workload(wl), make_sim(oracle, wl)
        load_rows(h, sim, w0[None, :])
        start = h.read_params(0).copy()
        for _ in range(T):
            h.local_step([0], [1], lr)
            sim.local_step([0], [1], lr)
        got = h.read_params(0)
        assert np.array_equal(got, sim.read_params(0))
        if rounding == 0:
            assert np.array_equal(got, start)
        else:
            assert got.mean() < 0.99 * start[0] and got.std() > 0


@pytest.mark.parametrize("m_dtype,rounding", MODES)
@pytest.mark.parametrize("P", [3, 4099, 70_001])
def test_local_step_parity_with_noise(oracle, P, m_dtype, rounding):
    n = 5
    wl = wl_of(n, P, m_dtype, rounding)
    h, sim = binding.Hadfl.from_workload(wl), make_sim(oracle, wl)
    rows = workloads.random_rows(n, P, seed=P)
    load_rows(h, sim, rows)
    for ids, steps in [([0, 1, 2, 3, 4], [1, 2, 3, 4, 8]), ([3, 1], [5, 0]), ([2, 0, 4, 1, 3], [2, 2, 1, 7, 3])]:
        h.local_step(ids, steps, 0.01)
        sim.local_step(ids, steps, 0.01)
        for i in range(n):
            got, want = h.read_params(i), sim.read_params(i)
            assert np.abs(got - want).max() <= 2 * bf16_ulp(np.abs(want).max()), i
            assert np.mean(got != want) < 0.02
            gm, wm = h.read_momentum(i), sim.read_momentum(i)
            if m_dtype:
                assert np.abs(gm - wm).max() <= 2 * bf16_ulp(np.abs(wm).max()), i
                assert np.mean(gm != wm) < 0.02
            else:
                assert np.abs(gm - wm).max() <= wl.grad_std * 1e-5 / (1.0 - wl.momentum), i


@pytest.mark.parametrize("m_dtype,rounding", MODES)
@pytest.mark.parametrize("n,P,k", [(4, 100_003, 2), (8, 33_333, 4), (5, 1, 3), (16, 9_999, 16)])
def test_fused_round_equals_separate_calls(oracle, n, P, k, m_dtype, rounding):
    wl = wl_of(n, P, m_dtype, rounding, k=k, rounds=5, sync_every=3)
    fused, plain = runtime.Arena(wl), runtime.Arena(wl)
    sim = make_sim(oracle, wl)
    for r in range(wl.rounds):
        sf, sp, so = fused.run_round_fused(r), plain.run_round(r), oracle_round(sim, wl, r)
        assert np.array_equal(sf, sp) and np.array_equal(sf, so), r
        n2, d2 = fused.h.stats_read()
        pn2, pd2 = plain.h.stats_read()
        assert np.allclose(n2, pn2, rtol=2e-6) and np.allclose(d2, pd2, rtol=2e-6, atol=1e-30), r
    for i in range(n):
        assert np.array_equal(fused.h.read_params(i), plain.h.read_params(i)), i
        assert np.array_equal(fused.h.read_momentum(i), plain.h.read_momentum(i)), i
        got, want = fused.h.read_params(i), sim.read_params(i)
        assert np.abs(got - want).max() <= 2 * bf16_ulp(np.abs(want).max()) and np.mean(got != want) < 0.02
    # the momentum arena holds what read_momentum returns, and the padding between rows stays zero
    mc = fused.m.float().cpu().numpy()
    assert not mc[:, P:].any() and np.array_equal(mc[1, :P], fused.h.read_momentum(1))
    fused.close()
    plain.close()


def test_fused_round_without_noise_is_bit_exact_against_the_oracle(oracle):
    wl = wl_of(6, 20_003, 1, 1, k=3, rounds=6, sync_every=2, grad_std=0.0, weight_decay=0.2)
    ar, sim = runtime.Arena(wl), make_sim(oracle, wl)
    rows = workloads.random_rows(6, wl.n_params, seed=11)
    load_rows(ar.h, sim, rows)
    for r in range(wl.rounds):
        assert np.array_equal(ar.run_round_fused(r), oracle_round(sim, wl, r))
        for i in range(6):
            assert np.array_equal(ar.h.read_params(i), sim.read_params(i)), (r, i)
            assert np.array_equal(ar.h.read_momentum(i), sim.read_momentum(i)), (r, i)
    ar.close()


def test_written_momentum_is_rounded_and_options_need_bf16_parameters(oracle):
    h = binding.Hadfl(1, 1027, dtype=1, m_dtype=1, seed=3)
    vals = np.linspace(-1, 1, 1027).astype(np.float32)
    h.write_momentum(0, vals)
    want = np.array([oracle.round_to_bf16(v) for v in vals], dtype=np.float32)
    assert np.array_equal(h.read_momentum(0), want)
    for kw in (dict(m_dtype=1), dict(rounding=1), dict(dtype=1, m_dtype=2), dict(dtype=1, rounding=2)):
        with pytest.raises(binding.HadflError) as e:
            binding.Hadfl(2, 64, **kw)
        assert e.value.code == binding.ERR_INVALID
