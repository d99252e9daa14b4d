"""End-to-end parity of the five workloads: the CUDA path against the CPU oracle, round by round.

Selections and version / step counters must agree exactly in every round.  Parameters are compared
within max|gpu - cpu| <= 2e-6 * max|x|: on the whole arena where the oracle finishes in seconds,
otherwise (the full-size vectors) on a column sample - the first and last groups of every row plus
random groups in between - which the oracle can follow on its own because every operation of the
round is elementwise in the column index.  bf16 storage: almost all elements equal, the others
within two bf16 steps (a last-bit difference of a gradient normal can move a rounding decision)."""
import numpy as np
import pytest
import torch

from gpu_common import compare_sample, require_gpu, run_and_compare
from oracle_driver import make_sim, oracle_round
from paper_2111_08274_b200 import runtime, workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def seams(wl):
    """Column groups where a one-wave grid of 3 or 4 blocks of 256 threads per SM (148 SMs, 8
    columns per thread) would start its next pass: a fault confined to the seam between passes, or
    to a partly filled last pass, would sit there."""
    return workloads.pass_boundaries(wl.n_params, [148 * 3 * 256, 148 * 4 * 256])


def test_c1_full_arena_every_round(oracle):
    wl = workloads.c1()
    run_and_compare(oracle, wl, None, check_rounds=range(wl.rounds), stats_rounds=range(wl.rounds))


def test_c1_ragged_tail_full_arena(oracle):
    """The same workload on a vector whose length is not a multiple of 4 and spans several blocks."""
    wl = workloads.shrink(workloads.c1(), 100_003)
    run_and_compare(oracle, wl, None, check_rounds=(0, 4))


def test_c2_full_size_sampled_columns(oracle):
    wl = workloads.c2()
    groups = workloads.sample_groups(wl.n_params, 30_000, 1024, seed=2)
    run_and_compare(oracle, wl, groups, check_rounds=(0, 9, 24))


def test_c2_full_size_fused_round_sampled_columns(oracle):
    """The launch configuration the benchmark times: the whole round of the full-size workload in
    one hadfl_round call per round."""
    wl = workloads.c2()
    # 2^20 random columns (2^18 groups) + the first and last 4096 columns of every row + the seams;
    # the oracle follows them on all host cores (its -fopenmp build: identical results)
    groups = workloads.sample_groups(wl.n_params, 262_144, 1024, seed=22, around=seams(wl))
    run_and_compare(oracle, wl, groups, check_rounds=(0, 9, 24), fused=True, openmp=True)


@pytest.mark.parametrize("name,rounds", [("c2", 8), ("c3", 11)])
def test_full_size_fused_round_whole_arena_against_the_oracle(oracle, name, rounds):
    """Every parameter and every momentum value of the full-size workload against the oracle (all
    host cores: its -fopenmp build, identical results), through the fused round, for the first
    rounds (c3: up to and including its first global synchronisation)."""
    from dataclasses import replace
    wl = replace(workloads.by_name(name), rounds=rounds)
    run_and_compare(oracle, wl, None, check_rounds=(0, rounds - 1), stats_rounds=(0,), fused=True, openmp=True)


def test_c3_full_size_fused_round_sampled_columns(oracle):
    wl = workloads.c3()
    groups = workloads.sample_groups(wl.n_params, 12_000, 1024, seed=33, around=seams(wl))
    run_and_compare(oracle, wl, groups, check_rounds=(0, 9, 10, 49), fused=True)


def test_c3_full_size_mixed_synchronisation_sampled_columns(oracle):
    """Config 3 with the staleness-bounding synchronisation read as a mix (every 10th round the
    unselected devices fold the aggregate into their own models with weight 1/2), through the
    fused round and through the separate calls."""
    from dataclasses import replace
    wl = replace(workloads.c3(), rounds=30, sync_beta=0.5)
    groups = workloads.sample_groups(wl.n_params, 4_000, 1024, seed=34)
    run_and_compare(oracle, wl, groups, check_rounds=(9, 19), fused=True)
    run_and_compare(oracle, wl, groups, check_rounds=(9, 19), fused=False)


def test_c2_shrunk_full_arena(oracle):
    wl = workloads.shrink(workloads.c2(), 50_002, rounds=8)
    run_and_compare(oracle, wl, None, check_rounds=range(8), stats_rounds=range(8))


def test_c3_full_size_sampled_columns(oracle):
    wl = workloads.c3()
    groups = workloads.sample_groups(wl.n_params, 6_000, 1024, seed=3)
    run_and_compare(oracle, wl, groups, check_rounds=(0, 9, 10, 49))


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("k", [2, 8, 16])
def test_c4_full_size_sampled_columns(oracle, k, fused):
    wl = workloads.c4(k)
    groups = workloads.sample_groups(wl.n_params, 6_000, 1024, seed=4 + k, around=seams(wl), halo=16)
    run_and_compare(oracle, wl, groups, check_rounds=(0, 9), fused=fused)


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("log2_p", range(16, 28))
def test_c5_bandwidth_sweep_sizes(oracle, log2_p, dtype, fused):
    for hetero in (False, True):
        wl = workloads.c5(log2_p, dtype=dtype, hetero=hetero)
        groups = workloads.sample_groups(wl.n_params, 256, 128, seed=log2_p, around=seams(wl), halo=4)
        run_and_compare(oracle, wl, groups, check_rounds=(0, 4, 99), fused=fused)


@pytest.mark.parametrize("dtype", [0, 1])
def test_c5_smallest_size_full_arena_first_rounds(oracle, dtype):
    wl = workloads.shrink(workloads.c5(16, dtype=dtype, hetero=True), 1 << 16, rounds=5)
    run_and_compare(oracle, wl, None, check_rounds=range(5), stats_rounds=range(5))


def test_rows_longer_than_two_to_the_31_elements(oracle):
    """Index arithmetic beyond 32 bits: two replicas of 2^31 + 6 parameters (row byte offsets and
    element indices above 2^32; column-group indices above 2^29), checked on sampled columns,
    through the separate calls and through the fused round."""
    from paper_2111_08274_b200.workloads import Workload
    P = 2**31 + 6
    wl = Workload("huge", 2, P, 2, 2, "fixed", (2, 1), grad_std=1e-2, seed=workloads.BASE_SEED + 99)
    groups = workloads.sample_groups(P, 512, 256, seed=7)
    run_and_compare(oracle, wl, groups, check_rounds=(0,))
    arena = runtime.Arena(wl)
    sim = make_sim(oracle, wl, groups)
    for r in range(wl.rounds):
        sel = arena.run_round_fused(r)
        assert np.array_equal(sel, oracle_round(sim, wl, r))
    compare_sample(arena, sim, groups, "huge fused")
    arena.close()
