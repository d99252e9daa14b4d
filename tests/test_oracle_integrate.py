"""Pins for the oracle's "integration" of a received model (Section "Model aggregation and
fault-tolerant": an unselected device folds the received parameters into its own; the paper gives
no formula, the oracle offers a convex combination with weight beta beside Algorithm 1's overwrite).

What fixes the expected values: the end points (beta = 1 is the already pinned overwrite, beta = 0
the identity), the textbook midpoint, exact rational arithmetic on small integers, bounds every
convex combination obeys, and a correctly rounded evaluation in extended precision."""
from fractions import Fraction

import numpy as np
import pytest

from paper_2111_08274_b200 import workloads

P = 1027


def sim_with_rows(oracle, n, rows=None, **kw):
    s = oracle.Sim(n, P, seed=2, **kw)
    rows = workloads.random_rows(n, P, seed=78) if rows is None else rows
    for i in range(n):
        s.write_params(i, rows[i])
    return s, rows


def test_beta_one_is_the_overwrite_and_beta_zero_the_identity(oracle):
    a, rows = sim_with_rows(oracle, 5)
    b, _ = sim_with_rows(oracle, 5)
    for s in (a, b):
        s.set_versions([7, 2, 9, 4, 1])
    a.integrate(1, [0, 3, 4], 1.0)
    b.broadcast(1, [0, 3, 4])
    for i in range(5):
        assert np.array_equal(a.read_params(i), b.read_params(i))
    assert list(a.get_versions()[0]) == list(b.get_versions()[0]) == [2, 2, 9, 2, 2]
    a.integrate(2, [0, 1], 0.0)
    for i in (0, 1):
        assert np.array_equal(a.read_params(i), rows[1])
    assert list(a.get_versions()[0]) == [9, 9, 9, 2, 2]       # the larger version, also at beta = 0


def test_midpoint_is_the_textbook_average(oracle):
    s, rows = sim_with_rows(oracle, 3)
    s.integrate(0, [2], 0.5)
    want = ((rows[0].astype(np.float64) + rows[2].astype(np.float64)) * 0.5).astype(np.float32)
    assert np.array_equal(s.read_params(2), want)
    assert np.array_equal(s.read_params(0), rows[0]) and np.array_equal(s.read_params(1), rows[1])


def test_exact_on_small_integers(oracle):
    """Integers below 2^10 and beta = k/8: every product and the sum are exact in fp32, so the
    result must equal the rational value - a swapped operand or a dropped term shows at once."""
    rng = np.random.default_rng(5)
    rows = rng.integers(-1000, 1000, (2, P)).astype(np.float32)
    for k in range(9):
        s, _ = sim_with_rows(oracle, 2, rows)
        s.integrate(0, [1], k / 8.0)
        got = s.read_params(1)
        for p in range(0, P, 97):
            want = Fraction(k, 8) * int(rows[0, p]) + Fraction(8 - k, 8) * int(rows[1, p])
            assert Fraction(float(got[p])) == want


@pytest.mark.parametrize("beta", [0.1, 0.25, 0.3333333, 0.9])
def test_convex_combination_bounds_and_rounding(oracle, beta):
    s, rows = sim_with_rows(oracle, 4)
    s.integrate(3, [0, 1], beta)
    b32 = float(np.float32(beta))
    omb = float(np.float32(1.0) - np.float32(beta))
    for i in (0, 1):
        got = s.read_params(i).astype(np.float64)
        src, old = rows[3].astype(np.float64), rows[i].astype(np.float64)
        lo, hi = np.minimum(src, old), np.maximum(src, old)
        slack = 2 * np.spacing(np.maximum(np.abs(src), np.abs(old)).astype(np.float32))
        assert np.all(got >= lo - slack) and np.all(got <= hi + slack)
        # the stated evaluation: one rounding of (1 - beta) * old, then a fused multiply-add,
        # redone here in extended precision and rounded once
        t = (np.longdouble(omb) * old.astype(np.longdouble)).astype(np.float32)
        want = (np.longdouble(b32) * src.astype(np.longdouble) + t.astype(np.longdouble)).astype(np.float32)
        assert np.array_equal(s.read_params(i), want)
    assert np.array_equal(s.read_params(2), rows[2])


def test_each_receiver_mixes_with_its_own_row_and_momentum_is_untouched(oracle):
    s, rows = sim_with_rows(oracle, 4)
    s.local_step([0, 1, 2, 3], [1, 1, 1, 1], 0.01)
    before = [s.read_params(i).copy() for i in range(4)]
    m_before = [s.read_momentum(i).copy() for i in range(4)]
    s.integrate(0, [1, 2, 3], 0.25)
    after = [s.read_params(i) for i in range(4)]
    assert np.array_equal(after[0], before[0])
    for i in (1, 2, 3):
        assert not np.array_equal(after[i], before[i])
        assert np.allclose(after[i], 0.25 * before[0] + 0.75 * before[i], rtol=0, atol=1e-7)
        assert np.array_equal(s.read_momentum(i), m_before[i])
    assert not np.array_equal(after[1], after[2])


def test_bf16_storage_rounds_the_mix_to_nearest_even(oracle):
    s, _ = sim_with_rows(oracle, 2, dtype=1)
    hi, _ = sim_with_rows(oracle, 2)
    for i in range(2):
        hi.write_params(i, s.read_params(i))           # the same bf16-representable values in fp32
    s.integrate(0, [1], 0.3)
    hi.integrate(0, [1], 0.3)
    want = np.array([oracle.round_to_bf16(v) for v in hi.read_params(1)], dtype=np.float32)
    assert np.array_equal(s.read_params(1), want)


def test_bad_arguments_are_rejected(oracle):
    s, rows = sim_with_rows(oracle, 3)
    for args in ((0, [0], 0.5), (0, [1, 1], 0.5), (3, [1], 0.5), (0, [5], 0.5), (0, [1], -0.1),
                 (0, [1], 1.5), (0, [1], float("nan"))):
        with pytest.raises(oracle.OracleError):
            s.integrate(*args)
    s.integrate(0, [], 0.5)
    for i in range(3):
        assert np.array_equal(s.read_params(i), rows[i])
