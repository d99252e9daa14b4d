"""The fused round (hadfl_round) at the sizes and in the launch configurations the benchmark times,
against the separate calls over the WHOLE arena, bit for bit, and against the CPU oracle on sampled
columns.

Two arenas run the same rounds, one through hadfl_round, one through hadfl_local_step +
hadfl_aggregate (+ hadfl_broadcast on global-synchronisation rounds); afterwards the parameter and
momentum tensors (row padding included) must be equal bit for bit - a comparison on the GPU that
needs no oracle time and covers every column, whatever block, pass or tail it falls in.  Vector
lengths include those around 2^20 parameters, where a one-wave grid changes how many passes it
makes over the vector."""
import numpy as np
import pytest
import torch

from gpu_common import compare_sample, require_gpu
from oracle_driver import make_sim, oracle_round
from paper_2111_08274_b200 import runtime, workloads
from paper_2111_08274_b200.workloads import Workload

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def run_both(wl, rounds, oracle=None, groups=None):
    fused, plain = runtime.Arena(wl), runtime.Arena(wl)
    sim = make_sim(oracle, wl, groups) if oracle is not None else None
    for r in range(rounds):
        sf, sp = fused.run_round_fused(r), plain.run_round(r)
        assert np.array_equal(sf, sp), r
        if sim is not None:
            assert np.array_equal(sf, oracle_round(sim, wl, r)), r
            assert np.array_equal(fused.h.get_versions()[0], sim.get_versions()[0]), r
    fused.h.synchronize()
    plain.h.synchronize()
    assert torch.equal(fused.w, plain.w), "parameters differ between the fused round and the separate calls"
    assert torch.equal(fused.m, plain.m), "momentum differs between the fused round and the separate calls"
    vf, vp = fused.h.get_versions(), plain.h.get_versions()
    assert np.array_equal(vf[0], vp[0]) and np.array_equal(vf[1], vp[1])
    a, b = fused.h.stats_read(), plain.h.stats_read()
    assert np.allclose(a[0], b[0], rtol=2e-6) and np.allclose(a[1], b[1], rtol=2e-6, atol=1e-30)
    if sim is not None:
        compare_sample(fused, sim, groups, wl.name + " fused")
    fused.h.debug_check()
    plain.h.debug_check()
    fused.close()
    plain.close()


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("P", [1 << 20, 1_000_003, 909_313, 1_212_417, 1_212_418])
def test_vectors_of_about_a_million_parameters(oracle, P, dtype):
    """N = 16, k = 4, mixed step counts, a global-synchronisation round every third round."""
    wl = Workload("window", 16, P, 4, 7, "fixed", (1, 3, 2, 5, 1, 1, 4, 2) * 2, grad_std=1e-2,
                  dtype=dtype, seed=workloads.BASE_SEED + 41, sync_every=3)
    groups = workloads.sample_groups(P, 2_000, 512, seed=P & 0xFFFF,
                                     around=workloads.pass_boundaries(P, [148 * 3 * 256, 148 * 4 * 256]))
    run_both(wl, wl.rounds, oracle, groups)


@pytest.mark.parametrize("name,rounds", [("c2", 6), ("c3", 11), ("c4_k2", 3), ("c4_k8", 3), ("c4_k16", 3),
                                         ("c5_p27_fp32", 3), ("c5_p27_bf16_het", 3), ("c5_p24_bf16", 4),
                                         ("c5_p22_fp32_het", 4)])
def test_full_size_workloads_whole_arena_bit_for_bit(name, rounds):
    wl = workloads.by_name(name)
    run_both(wl, rounds)


def test_full_size_mixed_synchronisation_whole_arena_bit_for_bit():
    from dataclasses import replace
    wl = replace(workloads.c3(), sync_every=2, sync_beta=0.25)
    run_both(wl, 4)


@pytest.mark.parametrize("name,rounds", [("c5_p27_fp32", 9), ("c5_p26_bf16", 9), ("c5_p24_fp32", 10), ("c5_p22_bf16", 17)])
def test_full_size_batched_rounds_whole_arena_bit_for_bit(name, rounds):
    """One step per device: hadfl_rounds puts 8 rounds into each launch.  Against one launch per round, over
    the whole arena; from 2^26 parameters up the blocks stride over several chunks, each taken through the
    whole batch before the next."""
    from dataclasses import replace
    wl = replace(workloads.by_name(name), sync_every=4)
    batched, single = runtime.Arena(wl), runtime.Arena(wl)
    single.h.set_round_batch(1)
    before = batched.h.launch_count()
    sb = batched.run_rounds_fused(0, rounds)
    assert batched.h.launch_count() - before == (rounds + 7) // 8
    ss = single.run_rounds_fused(0, rounds)
    assert np.array_equal(sb, ss)
    batched.h.synchronize()
    single.h.synchronize()
    assert torch.equal(batched.w, single.w), "parameters differ between batched and single launches"
    assert torch.equal(batched.m, single.m), "momentum differs between batched and single launches"
    vb, vs = batched.h.get_versions(), single.h.get_versions()
    assert np.array_equal(vb[0], vs[0]) and np.array_equal(vb[1], vs[1])
    a, b = batched.h.stats_read(), single.h.stats_read()
    if wl.dtype == 0:  # fp32 batches of one-step rounds fold the statistics over chunks of half the width
        assert np.allclose(a[0], b[0], rtol=2e-6) and np.allclose(a[1], b[1], rtol=2e-6, atol=1e-30)
    else:
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    batched.h.debug_check()
    batched.close()
    single.close()


def test_full_size_batched_rounds_against_the_oracle(oracle):
    """The ResNet-18 size with one step per device, 8 devices: 11 rounds in two launches (8 + 3), sampled
    columns against the oracle."""
    from dataclasses import replace
    wl = replace(workloads.c2(), name="c2_steps1", steps_rule="fixed", steps_fixed=(1,) * 8, sync_every=5)
    groups = workloads.sample_groups(wl.n_params, 4_000, 1_024, seed=91)
    arena = runtime.Arena(wl)
    sim = make_sim(oracle, wl, groups)
    before = arena.h.launch_count()
    sel = arena.run_rounds_fused(0, 11)
    assert arena.h.launch_count() - before == 2
    for r in range(11):
        assert np.array_equal(sel[r], oracle_round(sim, wl, r)), r
    assert np.array_equal(arena.h.get_versions()[0], sim.get_versions()[0])
    compare_sample(arena, sim, groups, "c2_steps1 batched")
    arena.close()
