"""Device groups (Section "Heterogeneity-aware training strategy generation": with many devices,
partial synchronisation runs inside groups, and an inter-group synchronisation runs every few
intra-group periods).  Groups need no kernel of their own: the availability mask restricts Eq. 8 to
a group, aggregation and broadcast take any device lists.  Checked against the oracle driven the
same way."""
import numpy as np
import pytest

from gpu_common import assert_close_params, require_gpu
from oracle_driver import make_sim
from paper_2111_08274_b200 import runtime, workloads
from paper_2111_08274_b200.workloads import Workload

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def grouped_round(o, wl, r, groups, k_in_group, inter_every):
    """o: the library handle or the oracle simulation (same method names)."""
    n = wl.n_devices
    o.local_step(wl.device_ids(), wl.steps_for_round(r), wl.lr)
    picks = []
    for gi, members in enumerate(groups):           # intra-group partial synchronisation
        mask = np.zeros(n, dtype=np.uint8)
        mask[members] = 1
        o.set_available(mask)
        sel = o.select(r, k_in_group, wl.select_seed() + gi)
        o.aggregate(sel)
        picks.append(sel)
    if (r + 1) % inter_every == 0:                  # inter-group: one representative per group
        reps = np.array([int(p[0]) for p in picks], dtype=np.int32)
        o.set_available(None)
        o.aggregate(reps)
        for rep, members in zip(reps, groups):
            o.broadcast(int(rep), [int(d) for d in members if d != rep])
    o.set_available(None)
    return picks


def test_two_level_synchronisation_matches_oracle(oracle):
    n, P = 12, 30_003
    wl = Workload("groups", n, P, 2, 6, "fixed", tuple(1 + i % 3 for i in range(n)), grad_std=1e-2,
                  seed=workloads.BASE_SEED + 55)
    groups = [np.arange(0, 4), np.arange(4, 8), np.arange(8, 12)]
    arena = runtime.Arena(wl)
    sim = make_sim(oracle, wl)
    for r in range(wl.rounds):
        a = grouped_round(arena.h, wl, r, groups, 2, inter_every=3)
        b = grouped_round(sim, wl, r, groups, 2, inter_every=3)
        for x, y, members in zip(a, b, groups):
            assert np.array_equal(x, y) and set(int(i) for i in x) <= set(int(i) for i in members)
        assert np.array_equal(arena.h.get_versions()[0], sim.get_versions()[0])
    for i in range(n):
        assert_close_params(arena.h.read_params(i), sim.read_params(i), "w[%d]" % i)
    # after the inter-group round every device holds the same model
    ref = arena.h.read_params(0)
    assert all(np.array_equal(arena.h.read_params(i), ref) for i in range(n))
    arena.close()
