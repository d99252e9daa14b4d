"""Pins for the oracle's partial aggregation (Eq. 5), its weights, the broadcast and the stats."""
import itertools

import numpy as np
import pytest
import torch

from paper_2111_08274_b200 import workloads

P = 1027


def sim_with_rows(oracle, n, rows=None, **kw):
    s = oracle.Sim(n, P, seed=2, **kw)
    rows = workloads.random_rows(n, P, seed=77) if rows is None else rows
    for i in range(n):
        s.write_params(i, rows[i])
    return s, rows


@pytest.mark.parametrize("k", range(1, 33))
def test_uniform_weights_sum_to_one(oracle, k):
    s = oracle.Sim(32, 8, seed=1)
    a = s.aggregation_weights(list(range(k)))
    assert np.all(a == np.float32(1.0 / k))
    total = np.float64(a.astype(np.float64).sum())
    assert abs(total - 1.0) <= k * 2.0 ** -25
    if k & (k - 1) == 0:
        assert total == 1.0


@pytest.mark.parametrize("k", [1, 2])
def test_identical_replicas_aggregate_to_themselves_exactly(oracle, k):
    row = workloads.random_rows(1, P, seed=5)[0]
    s, _ = sim_with_rows(oracle, 32, np.repeat(row[None], 32, 0))
    s.aggregate(list(range(k)))
    for i in range(32):
        assert np.array_equal(s.read_params(i), row)


@pytest.mark.parametrize("k", [3, 4, 5, 7, 8, 12, 16, 31, 32])
def test_identical_replicas_aggregate_to_themselves_within_rounding(oracle, k):
    """k-1 fused adds, each rounding a partial sum no larger than the row itself, plus the
    rounding of 1/k: at most (k+1)/2 ulp from the identity."""
    row = workloads.random_rows(1, P, seed=5)[0]
    s, _ = sim_with_rows(oracle, 32, np.repeat(row[None], 32, 0))
    s.aggregate(list(range(k)))
    err = np.abs(s.read_params(0).astype(np.float64) - row.astype(np.float64))
    assert np.all(err <= 0.5 * (k + 1) * np.spacing(np.abs(row)))
    assert err.max() <= 4 * np.spacing(np.abs(row)).max()      # in practice errors do not line up


def test_single_selected_device_is_a_no_op(oracle):
    s, rows = sim_with_rows(oracle, 4)
    s.set_versions([3, 1, 4, 1])
    s.aggregate([2])
    for i in range(4):
        assert np.array_equal(s.read_params(i), rows[i])
    assert list(s.get_versions()[0]) == [3, 1, 4, 1]


def test_two_rows_is_the_textbook_mean(oracle):
    s, rows = sim_with_rows(oracle, 4)
    s.aggregate([3, 1])
    want = np.float32(0.5) * (rows[3] + rows[1])         # exact in fp32 up to the single add rounding
    assert np.array_equal(s.read_params(3), want) and np.array_equal(s.read_params(1), want)
    assert np.array_equal(s.read_params(0), rows[0]) and np.array_equal(s.read_params(2), rows[2])


@pytest.mark.parametrize("k", [3, 4, 7, 16])
def test_mean_of_selected_rows_and_write_back(oracle, k):
    n = 16
    s, rows = sim_with_rows(oracle, n)
    m_before = [s.read_momentum(i).copy() for i in range(n)]
    sel = list(np.random.default_rng(k).permutation(n)[:k])
    s.aggregate(sel)
    want = rows[sel].astype(np.float64).mean(axis=0)      # Eq. 5 with K = number of selected devices
    for i in range(n):
        if i in sel:
            assert np.abs(s.read_params(i) - want).max() <= k * 2.0 ** -24 * np.abs(rows[sel]).max()
            assert np.array_equal(s.read_params(i), s.read_params(sel[0]))
        else:
            assert np.array_equal(s.read_params(i), rows[i])
        assert np.array_equal(s.read_momentum(i), m_before[i])   # momentum stays local


def test_order_changes_result_by_rounding_only(oracle):
    k = 5
    base = None
    for perm in itertools.islice(itertools.permutations(range(k)), 0, 120, 7):
        s, rows = sim_with_rows(oracle, k)
        s.aggregate(list(perm))
        out = s.read_params(0)
        if base is None:
            base = out
        # k-1 roundings, each of a partial sum no larger than the largest input of that column
        assert np.all(np.abs(out - base) <= (k - 1) * 2.0 ** -24 * np.abs(rows).max(axis=0))


def test_linearity_under_power_of_two_scaling(oracle):
    s1, rows = sim_with_rows(oracle, 6)
    s2, _ = sim_with_rows(oracle, 6, rows * np.float32(4.0))
    s1.aggregate([5, 0, 3])
    s2.aggregate([5, 0, 3])
    assert np.array_equal(s2.read_params(0), np.float32(4.0) * s1.read_params(0))


def test_argument_checks(oracle):
    s, _ = sim_with_rows(oracle, 4)
    for sel in ([], [0, 0], [4], [-1, 2], [0, 1, 2, 3, 0]):
        with pytest.raises(oracle.OracleError):
            s.aggregate(sel)


def test_version_weighted_mode_sums_to_one_and_prefers_mu(oracle):
    s = oracle.Sim(4, 8, seed=1, weight_mode=1)
    s.set_versions([4, 2, 2, 1])
    a = s.aggregation_weights([0, 1, 3])
    assert abs(np.float64(a.astype(np.float64).sum()) - 1.0) <= 2.0 ** -23
    f = np.exp(-0.5 * (np.array([4.0, 2.0, 1.0]) - 2.5) ** 2)     # mu = Q3 of all available = 2.5
    assert np.allclose(a, f / f.sum(), rtol=1e-6)
    assert a[1] > a[0] and np.isclose(a[0], a[2], rtol=1e-6)
    # equal versions -> uniform
    s.set_versions([7, 7, 7, 7])
    assert np.allclose(s.aggregation_weights([2, 0, 1]), 1.0 / 3.0, rtol=1e-6)


def test_bf16_storage_rounds_the_aggregate(oracle):
    rows = workloads.random_rows(4, P, seed=9)
    s, _ = sim_with_rows(oracle, 4, rows, dtype=1)
    rb = torch.from_numpy(rows).to(torch.bfloat16).float().numpy()
    for i in range(4):
        assert np.array_equal(s.read_params(i), rb[i])
    f, _ = sim_with_rows(oracle, 4, rb)
    s.aggregate([0, 2, 3])
    f.aggregate([0, 2, 3])
    assert np.array_equal(s.read_params(2), torch.from_numpy(f.read_params(2)).to(torch.bfloat16).float().numpy())


def test_broadcast_overwrites_receivers(oracle):
    s, rows = sim_with_rows(oracle, 5)
    s.set_versions([9, 1, 2, 3, 4])
    s.broadcast(0, [3, 1])
    assert np.array_equal(s.read_params(3), rows[0]) and np.array_equal(s.read_params(1), rows[0])
    assert np.array_equal(s.read_params(2), rows[2])
    assert list(s.get_versions()[0]) == [9, 9, 2, 9, 4]
    with pytest.raises(oracle.OracleError):
        s.broadcast(0, [0])


def test_stats_match_numpy(oracle):
    s, rows = sim_with_rows(oracle, 5)
    n2, d2 = s.stats(2)
    r = rows.astype(np.float64)
    assert np.allclose(n2, (r * r).sum(axis=1), rtol=1e-13)
    assert np.allclose(d2, ((r - r[2]) ** 2).sum(axis=1), rtol=1e-13)
    assert d2[2] == 0.0
    s.aggregate([0, 1])
    n2, d2 = s.stats(0)
    assert d2[0] == 0.0 and d2[1] == 0.0 and d2[2] > 0
