"""The -fopenmp build of the oracle (used only to time an all-cores CPU baseline) must give the
results of the plain single-threaded build bit for bit: its loops are split over column blocks, and
every operation of the round is elementwise in the column index."""
import numpy as np
import pytest

from oracle_driver import oracle_round
from paper_2111_08274_b200 import workloads
from paper_2111_08274_b200.workloads import Workload


@pytest.mark.parametrize("dtype,m_dtype,rounding", [(0, 0, 0), (1, 0, 0), (1, 1, 1)])
def test_openmp_build_equals_plain_build(oracle, dtype, m_dtype, rounding):
    wl = Workload("omp", 6, 20_003, 3, 5, "fixed", (1, 3, 2, 0, 4, 1), grad_std=1e-2, dtype=dtype,
                  m_dtype=m_dtype, rounding=rounding, seed=workloads.BASE_SEED + 61, sync_every=2,
                  sync_beta=0.5)
    kw = dict(dtype=wl.dtype, momentum=wl.momentum, weight_decay=wl.weight_decay, grad_std=wl.grad_std,
              init_std=wl.init_std, seed=wl.seed, version_scale=wl.version_scale,
              weight_mode=wl.weight_mode, m_dtype=wl.m_dtype, rounding=wl.rounding)
    plain = oracle.Sim(wl.n_devices, wl.n_params, **kw)
    omp = oracle.Sim(wl.n_devices, wl.n_params, openmp=True, **kw)
    assert oracle.threads() == 1 and oracle.threads(openmp=True) >= 1
    for r in range(wl.rounds):
        a, b = oracle_round(plain, wl, r), oracle_round(omp, wl, r)
        assert np.array_equal(a, b)
        sa, sb = plain.stats(int(a[0])), omp.stats(int(b[0]))
        assert np.array_equal(sa[0], sb[0]) and np.array_equal(sa[1], sb[1])
    for i in range(wl.n_devices):
        assert np.array_equal(plain.read_params(i), omp.read_params(i))
        assert np.array_equal(plain.read_momentum(i), omp.read_momentum(i))
    va, vb = plain.get_versions(), omp.get_versions()
    assert np.array_equal(va[0], vb[0]) and np.array_equal(va[1], vb[1])
