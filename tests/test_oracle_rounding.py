"""Pins for the oracle's reduced-precision state: bf16 momentum and stochastic rounding of the
bf16 stores of the local update (a workload variant outside the paper, which trains in fp32).

What fixes the expected values: the definition of stochastic rounding (neighbour of larger
magnitude with probability equal to the discarded fraction - counted exhaustively over the 2^16
random values), the already pinned generator, the already pinned fp32 local update (the value before
rounding), and the closed form of a weight-decay-only run (nearest-even storage stalls when the
update is below half a spacing; stochastic storage follows the closed form on average).
"""
import numpy as np
import pytest

from test_oracle_philox import M32, philox_generic

P = 1027


def f32_bits(v):
    return int(np.float32(v).view(np.uint32))


def bits_f32(b):
    return float(np.uint32(b).view(np.float32))


@pytest.mark.parametrize("v", [0.1, -0.1, 3.0e-5, -7.7e3, 1.0 + 2.0 ** -9, 0.3333333, 1.17e-38])
def test_stochastic_rounding_counts(oracle, v):
    """Over all 2^16 random values the upper neighbour is taken exactly (discarded bits) times."""
    b = f32_bits(v)
    low = b & 0xFFFF
    down = bits_f32(b & 0xFFFF0000)
    up = bits_f32((b & 0xFFFF0000) + 0x10000)
    got = np.array([oracle.round_to_bf16_stochastic(v, r) for r in range(1 << 16)])
    assert set(np.unique(got)) <= {down, up}
    assert int((got == up).sum()) == low
    assert abs(up) > abs(down)                       # "up" is away from zero, whatever the sign
    # expectation = the value itself (exact in rational arithmetic: down + (low / 2^16) * spacing)
    mean = down + (low / 65536.0) * (up - down)
    assert mean == pytest.approx(float(np.float32(v)), rel=0, abs=abs(up - down) * 2 ** -16)
    # the decision is monotone in r: r >= 2^16 - low rounds up
    assert np.all(got[: (1 << 16) - low] == down) and np.all(got[(1 << 16) - low:] == up)


def test_stochastic_rounding_special_values(oracle):
    for v in (0.0, 1.0, -2.5, 0.15625, float(np.float32(2.0 ** -100))):   # representable: unchanged
        for r in (0, 1, 0x7FFF, 0x8000, 0xFFFF):
            assert oracle.round_to_bf16_stochastic(v, r) == v
    assert oracle.round_to_bf16_stochastic(float("inf"), 0xFFFF) == float("inf")
    assert oracle.round_to_bf16_stochastic(float("-inf"), 0xFFFF) == float("-inf")
    assert np.isnan(oracle.round_to_bf16_stochastic(float("nan"), 0xFFFF))
    # only the low 16 bits of r are used
    assert oracle.round_to_bf16_stochastic(0.1, 0x12340001) == oracle.round_to_bf16_stochastic(0.1, 1)
    # antisymmetry
    for r in (3, 40000, 65535):
        assert oracle.round_to_bf16_stochastic(-0.7, r) == -oracle.round_to_bf16_stochastic(0.7, r)


def test_rounding_words_are_the_generator_on_the_stated_counter(oracle):
    seed = 0x0123456789ABCDEF
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for group, step, dev in [(0, 0, 0), (5, 17, 3), (2 ** 32 - 1, 2 ** 40 + 9, 31), (77, 2 ** 32 - 1, 1)]:
        ctr = [group, step & 0xFFFFFFFF, dev, 0x52000000 | (step >> 32)]
        want = philox_generic(ctr, key, 32, M32)
        assert [int(x) for x in oracle.rounding_words(seed, group, step, dev)] == want
        assert [int(x) for x in oracle.philox4x32_10(ctr, key)] == want
    # a stream of its own: not the gradient block of the same step
    grad_ctr = [5, 17, 3, 0x47000000]
    assert [int(x) for x in oracle.rounding_words(seed, 5, 17, 3)] != philox_generic(grad_ctr, key, 32, M32)


def _pair(oracle, **kw):
    """A bf16-storage simulation and an fp32-storage one in the same (bf16-representable) state."""
    args = dict(seed=77, grad_std=1e-2, momentum=0.9, weight_decay=5e-4)
    lo = oracle.Sim(2, P, dtype=1, **args, **kw)
    hi = oracle.Sim(2, P, dtype=0, **args)
    for i in range(2):
        hi.write_params(i, lo.read_params(i))
    return lo, hi


@pytest.mark.parametrize("m_dtype", [0, 1])
def test_stochastic_store_is_the_rounding_of_the_fp32_result(oracle, m_dtype):
    """One call: the stored value is the fp32 result of the (pinned) fp32 update, rounded with
    the call's rounding words - low half for the parameter, high half for the momentum."""
    lo, hi = _pair(oracle, m_dtype=m_dtype, rounding=1)
    start = np.array([2 ** 32 - 3, 9], dtype=np.uint64)       # also crosses a 2^32 step index
    lo.set_versions(step_counts=start)
    hi.set_versions(step_counts=start)
    steps = [5, 2]
    lo.local_step([0, 1], steps, 0.05)
    hi.local_step([0, 1], steps, 0.05)
    for dev in range(2):
        last = int(start[dev]) + steps[dev] - 1
        words = np.concatenate([oracle.rounding_words(77, g, last, dev) for g in range((P + 3) // 4)])[:P]
        w_hi, m_hi = hi.read_params(dev), hi.read_momentum(dev)
        want_w = [oracle.round_to_bf16_stochastic(v, int(x) & 0xFFFF) for v, x in zip(w_hi, words)]
        assert np.array_equal(lo.read_params(dev), np.array(want_w, dtype=np.float32))
        if m_dtype:
            want_m = [oracle.round_to_bf16_stochastic(v, int(x) >> 16) for v, x in zip(m_hi, words)]
            assert np.array_equal(lo.read_momentum(dev), np.array(want_m, dtype=np.float32))
        else:
            assert np.array_equal(lo.read_momentum(dev), m_hi)
    # both neighbours occur, and neither rarely: a store that always truncates or always rounds up
    # would be caught here
    w_hi = hi.read_params(0)
    went_up = np.abs(lo.read_params(0)) > np.abs(w_hi)
    assert 0.3 < went_up.mean() < 0.7


def test_bf16_momentum_nearest_even_is_one_rounding_per_call(oracle):
    lo, hi = _pair(oracle, m_dtype=1, rounding=0)
    lo.local_step([0, 1], [4, 1], 0.05)
    hi.local_step([0, 1], [4, 1], 0.05)
    for dev in range(2):
        want_m = np.array([oracle.round_to_bf16(v) for v in hi.read_momentum(dev)], dtype=np.float32)
        want_w = np.array([oracle.round_to_bf16(v) for v in hi.read_params(dev)], dtype=np.float32)
        assert np.array_equal(lo.read_momentum(dev), want_m)
        assert np.array_equal(lo.read_params(dev), want_w)
    # the second call starts from the rounded momentum: it now differs from the fp32-momentum run
    lo2, _ = _pair(oracle, m_dtype=0, rounding=0)
    lo2.local_step([0, 1], [4, 1], 0.05)
    assert np.array_equal(lo2.read_params(0), lo.read_params(0))
    lo.local_step([0], [1], 0.05)
    lo2.local_step([0], [1], 0.05)
    assert not np.array_equal(lo2.read_params(0), lo.read_params(0))


def test_written_momentum_is_rounded_when_stored_as_bf16(oracle):
    s = oracle.Sim(1, P, dtype=1, m_dtype=1, seed=3)
    vals = np.linspace(-1, 1, P).astype(np.float32)
    s.write_momentum(0, vals)
    want = np.array([oracle.round_to_bf16(v) for v in vals], dtype=np.float32)
    assert np.array_equal(s.read_momentum(0), want)


def test_a_device_without_steps_is_not_touched(oracle):
    s = oracle.Sim(2, P, dtype=1, m_dtype=1, rounding=1, seed=5)
    w0 = s.read_params(1).copy()
    s.local_step([0, 1], [3, 0], 0.05)
    assert np.array_equal(s.read_params(1), w0) and not s.read_momentum(1).any()


def test_options_need_bf16_parameters(oracle):
    for kw in (dict(m_dtype=1), dict(rounding=1), dict(dtype=1, m_dtype=2), dict(dtype=1, rounding=2)):
        with pytest.raises(oracle.OracleError):
            oracle.Sim(2, 64, **kw)


def test_nearest_even_stalls_where_stochastic_rounding_follows_the_closed_form(oracle):
    """Weight decay only (no noise, no momentum): w <- w (1 - lr wd) per step.  With lr wd = 1e-3
    the update is below half a bf16 spacing (2^-9 relative), so nearest-even storage never moves;
    stochastic storage is unbiased, so its mean over many columns follows (1 - lr wd)^T."""
    n, lr, wd, T = 4000, 0.1, 0.01, 150
    args = dict(seed=8, grad_std=0.0, momentum=0.0, weight_decay=wd)
    rne = oracle.Sim(1, n, dtype=1, **args)
    sr = oracle.Sim(1, n, dtype=1, rounding=1, **args)
    w0 = np.full(n, 0.4, dtype=np.float32)           # 0.4 is not at a binade edge
    rne.write_params(0, w0)
    sr.write_params(0, w0)
    start = rne.read_params(0).copy()
    for _ in range(T):
        rne.local_step([0], [1], lr)
        sr.local_step([0], [1], lr)
    assert np.array_equal(rne.read_params(0), start)
    shrink = (1.0 - float(np.float32(lr)) * float(np.float32(wd))) ** T
    got = sr.read_params(0).astype(np.float64)
    want = float(start[0]) * shrink
    # per column: a random walk of spacing 2^-9 * 0.25 .. steps; mean over n columns is tight
    sem = got.std() / np.sqrt(n)
    assert abs(got.mean() - want) < 5 * sem + 1e-6
    assert want < 0.9 * float(start[0]) and got.std() > 0     # it moved, and not in lockstep
