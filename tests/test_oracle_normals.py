"""Pins for the oracle's uniform -> normal transform (Box-Muller) and the initial model."""
import numpy as np
import pytest
from scipy import stats


def test_box_muller_identities(oracle):
    rng = np.random.default_rng(5)
    for _ in range(200):
        x = rng.integers(0, 2**32, 4, dtype=np.uint64).astype(np.uint32)
        z = oracle.words_to_normals(x)
        u = (x.astype(np.float64) + 0.5) / 2.0**32
        for pair in (0, 1):
            z0, z1 = z[2 * pair], z[2 * pair + 1]
            # radius and angle recover the two uniforms
            assert np.isclose(z0 * z0 + z1 * z1, -2.0 * np.log(u[2 * pair]), rtol=1e-12)
            ang = np.arctan2(z1, z0) % (2 * np.pi)
            assert np.isclose(ang, 2 * np.pi * u[2 * pair + 1], rtol=0, atol=1e-9)


def test_extreme_words_are_finite(oracle):
    z = oracle.words_to_normals(np.array([0, 0, 0xFFFFFFFF, 0xFFFFFFFF], dtype=np.uint32))
    assert np.all(np.isfinite(z))
    # u0 = 2^-33 gives the largest radius the generator can produce: sqrt(2*33*ln 2) = 6.7639
    assert np.isclose(np.hypot(z[0], z[1]), np.sqrt(66 * np.log(2.0)), rtol=1e-12)


def test_gradient_normals_are_standard_normal(oracle):
    n_groups = 50000
    z = np.concatenate([oracle.grad_normals(77, g, 3, 2) for g in range(n_groups)]).astype(np.float64)
    n = z.size
    assert abs(z.mean()) < 5.0 / np.sqrt(n)
    assert abs(z.var() - 1.0) < 5.0 * np.sqrt(2.0 / n)
    assert abs(stats.skew(z)) < 5.0 * np.sqrt(6.0 / n)
    assert abs(stats.kurtosis(z)) < 5.0 * np.sqrt(24.0 / n)
    assert stats.kstest(z, "norm").pvalue > 1e-4
    # the four lanes of a block are uncorrelated
    zz = z.reshape(-1, 4)
    c = np.corrcoef(zz.T)
    assert np.abs(c - np.eye(4)).max() < 5.0 / np.sqrt(n_groups)


def test_initial_model_is_shared_and_has_the_stated_std(oracle):
    P = 200_001
    s = oracle.Sim(3, P, seed=1234, init_std=0.05)
    w0 = s.read_params(0)
    for i in (1, 2):
        assert np.array_equal(s.read_params(i), w0)      # Algorithm 1: w^k_(0) = w_(0) for all k
        assert not s.read_momentum(i).any()
    assert abs(w0.std() / 0.05 - 1.0) < 5.0 / np.sqrt(2 * P)
    assert abs(w0.mean()) < 5 * 0.05 / np.sqrt(P)
    v, sc = s.get_versions()
    assert not v.any() and not sc.any()
    # lanes of the ragged last group beyond P are not part of the model
    assert s.n_cols == 4 * ((P + 3) // 4) and not s.read_cols(0)[P:].any()
    # a different seed is a different model
    assert not np.array_equal(oracle.Sim(1, 64, seed=1235).read_params(0), w0[:64])


def test_column_subset_reproduces_full_simulation(oracle):
    """Every operation is elementwise in the column index, so simulating a subset of the
    column groups gives exactly those columns of the full run (used to check large vectors)."""
    P = 4099
    groups = np.array([0, 1, 7, 500, 1023, 1024], dtype=np.uint32)   # 1024 is the ragged last group
    kw = dict(seed=42, grad_std=1e-2)
    full, part = oracle.Sim(4, P, **kw), oracle.Sim(4, P, groups=groups, **kw)
    for r in range(3):
        for s in (full, part):
            s.local_step([0, 1, 2, 3], [1, 2, 3, 4], 0.01)
            sel = s.select(r, 2, 99)
            s.aggregate(sel)
    cols = (4 * groups[:, None] + np.arange(4)[None, :]).reshape(-1)
    for i in range(4):
        f = np.zeros(4 * 1025, dtype=np.float32)
        f[:P] = full.read_params(i)
        assert np.array_equal(part.read_cols(i), f[cols])
    assert np.array_equal(full.get_versions()[0], part.get_versions()[0])


def test_bf16_rounding_is_nearest_even(oracle):
    import torch
    rng = np.random.default_rng(3)
    xs = np.concatenate([rng.standard_normal(2000).astype(np.float32) * 0.05,
                         np.array([0.0, 1.0, 1.00390625, 1.01171875, -1.00390625, 3.0e38, 1e-40], dtype=np.float32)])
    want = torch.from_numpy(xs).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([oracle.round_to_bf16(x) for x in xs], dtype=np.float32)
    assert np.array_equal(got, want)
