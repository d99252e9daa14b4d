"""Pins for the oracle's probability-based selection (Eq. 8) and the version bookkeeping."""
import itertools
import os
from collections import Counter

import numpy as np
import pytest
from scipy import stats

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def read_rows(name):
    rows = []
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            rows.append([[float(t) for t in part.split()] for part in line.split("|")])
    return rows


def test_paper_vectors(oracle):
    for versions, (mu,), probs in read_rows("eq8_probabilities.txt"):
        assert oracle.third_quartile(versions) == mu
        assert np.allclose(oracle.select_probs(versions), probs, rtol=0, atol=5e-7)


def test_probabilities_are_the_normalised_gaussian_density(oracle):
    rng = np.random.default_rng(4)
    for _ in range(50):
        n = int(rng.integers(1, 33))
        v = rng.integers(0, 12, n).astype(np.float64)
        mu = np.quantile(v, 0.75)                      # library quartile (linear interpolation)
        assert np.isclose(oracle.third_quartile(v), mu, rtol=1e-15)
        f = stats.norm.pdf(v, loc=mu, scale=1.0)       # library Gaussian density
        P = oracle.select_probs(v)
        assert np.allclose(P, f / f.sum(), rtol=1e-12)
        assert abs(P.sum() - 1.0) < 1e-14
        assert np.allclose(oracle.select_probs(v + 1000.0), P, rtol=1e-12)     # shift invariance
        for a, b in itertools.combinations(range(n), 2):                        # symmetry
            if v[a] == v[b]:
                assert P[a] == P[b]


def test_qualitative_statements_of_the_paper(oracle):
    P = oracle.select_probs([4, 2, 2, 1])
    assert P[1] > P[0] and P[3] > 0       # medial beats latest; straggler keeps a chance
    P = oracle.select_probs([8, 7, 7, 6, 5, 2])
    assert P[5] < P[4] < P[3]             # older is less likely in the tail below mu
    assert P[5] > 0


def test_mask_renormalises_over_available_devices(oracle):
    v = [4.0, 2.0, 2.0, 1.0, 9.0]
    P = oracle.select_probs(v, avail=[1, 1, 1, 1, 0])
    assert P[4] == 0.0 and np.allclose(P[:4], oracle.select_probs(v[:4]), rtol=1e-15)
    for r in range(200):
        assert 4 not in oracle.select(v, 3, r, 5, avail=[1, 1, 1, 1, 0])
    with pytest.raises(ValueError):
        oracle.select(v, 5, 0, 5, avail=[1, 1, 1, 1, 0])
    with pytest.raises(ValueError):
        oracle.select(v, 0, 0, 5)


def tuple_probability(P, tup):
    p, rest = 1.0, 1.0
    for i in tup:
        p *= P[i] / rest
        rest -= P[i]
    return p


@pytest.mark.parametrize("versions,k", [([3, 3, 1, 1], 2), ([4, 2, 2, 1], 2), ([4, 2, 2, 1], 3),
                                        ([1, 2, 5], 2), ([2, 2], 1), ([4, 2, 2, 1], 4)])
def test_brute_force_enumeration(oracle, versions, k):
    """Every ordered k-tuple has probability prod_t P(i_t) / (1 - sum of earlier picks)."""
    n = len(versions)
    P = oracle.select_probs(versions)
    want = {t: tuple_probability(P, t) for t in itertools.permutations(range(n), k)}
    assert abs(sum(want.values()) - 1.0) < 1e-12
    rounds = 40000
    seen = Counter(tuple(int(i) for i in oracle.select(versions, k, r, 0xABCDEF)) for r in range(rounds))
    assert set(seen) <= set(want)
    for t, p in want.items():
        sigma = np.sqrt(p * (1 - p) / rounds)
        assert abs(seen.get(t, 0) / rounds - p) < 5 * sigma + 1e-9, (t, p, seen.get(t, 0) / rounds)
    # first-draw marginal is P(i) itself
    first = Counter(t[0] for t in seen.elements())
    for i in range(n):
        assert abs(first.get(i, 0) / rounds - P[i]) < 5 * np.sqrt(P[i] * (1 - P[i]) / rounds) + 1e-9
    # the paper's remark on the worst case for [3,3,1,1]: always picking the two slowest devices
    # is possible but unlikely
    if versions == [3, 3, 1, 1]:
        p_slowest = want[(2, 3)] + want[(3, 2)]
        assert 0 < p_slowest < 0.02


def test_full_selection_is_a_permutation_and_depends_on_round_and_seed(oracle):
    v = np.arange(16) % 5
    a = oracle.select(v, 16, 0, 1)
    assert sorted(a) == list(range(16))
    assert not np.array_equal(a, oracle.select(v, 16, 1, 1))
    assert not np.array_equal(a, oracle.select(v, 16, 0, 2))
    assert np.array_equal(a, oracle.select(v, 16, 0, 1))
    # prefixes: the first picks of a longer draw are the shorter draw
    assert np.array_equal(a[:4], oracle.select(v, 4, 0, 1))


def test_far_stragglers_are_not_discarded(oracle):
    """With a spread so wide that f underflows, devices are still drawn (uniformly)."""
    v = [1000.0, 1000.0, 1000.0, 0.0, 0.0, 0.0]
    P = oracle.select_probs(v)
    assert np.allclose(P[:3], 1 / 3) and np.all(P[3:] == 0.0)
    tails = Counter()
    for r in range(3000):
        s = oracle.select(v, 4, r, 77)
        assert sorted(s[:3]) == [0, 1, 2]
        tails[int(s[3])] += 1
    assert set(tails) == {3, 4, 5}
    assert all(abs(c / 3000 - 1 / 3) < 0.05 for c in tails.values())


def test_version_scale(oracle):
    s = oracle.Sim(4, 8, seed=1, version_scale=0.125)
    s.set_versions([32, 16, 16, 8])
    assert np.allclose(s.select_probs(), oracle.select_probs([4, 2, 2, 1]), rtol=1e-15)
    assert np.allclose(s.select_probs([8, 8, 24, 24]), oracle.select_probs([1, 1, 3, 3]), rtol=1e-15)


def test_version_trace(oracle):
    """Hand-computed counters (tests/golden/version_trace.txt)."""
    s = oracle.Sim(4, 16, seed=1)
    for (r,), sel, versions, steps in read_rows("version_trace.txt"):
        s.local_step([0, 1, 2, 3], [1, 2, 3, 4], 0.01)
        s.aggregate([int(i) for i in sel])
        v, sc = s.get_versions()
        assert list(v) == versions and list(sc) == steps, r


def test_predictor_closed_forms(oracle):
    """Eq. 7: a constant series predicts itself; a linear series is extrapolated exactly once the
    smoothing has forgotten its start."""
    assert oracle.predict_version([5.0] * 6, 0.5, 3) == 5.0
    t = np.arange(400, dtype=np.float64)
    series = 2.0 + 3.0 * t
    for alpha in (0.3, 0.5, 0.8):
        for m in (1, 4):
            assert np.isclose(oracle.predict_version(series, alpha, m), 2.0 + 3.0 * (399 + m), rtol=1e-9)
    # alpha close to 1 follows the latest value (the paper's remark on alpha)
    assert abs(oracle.predict_version([1.0, 2.0, 7.0], 0.999, 0) - 7.0) < 0.02
