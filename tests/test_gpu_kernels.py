"""GPU parity, kernel by kernel: the CUDA path (through the C ABI) against the CPU oracle on the
same seeded inputs.  Integer work is compared bit for bit; fp32 parameters within
max|gpu - cpu| <= 2e-6 * max|x|; operations with a fixed fp32 order (aggregation, broadcast,
gradient-free updates) must agree exactly."""
import numpy as np
import pytest
import torch

from gpu_common import TOL_REL, assert_close_params, bf16_ulp, require_gpu
from oracle_driver import make_sim
from paper_2111_08274_b200 import binding, workloads
from paper_2111_08274_b200.workloads import Workload

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def small(n, P, **kw):
    args = dict(name="t", n_devices=n, n_params=P, k=min(2, n), rounds=1, steps_rule="fixed",
                steps_fixed=tuple(1 + i % 4 for i in range(n)), grad_std=1e-2, seed=0xC0FFEE + P)
    args.update(kw)
    return Workload(**args)


def gpu(wl, **kw):
    return binding.Hadfl.from_workload(wl, **kw)


def load_rows(h, sim, rows):
    for i in range(rows.shape[0]):
        h.write_params(i, rows[i])
        sim.write_params(i, rows[i])


# ---- generator --------------------------------------------------------------------------------
def test_philox_words_bit_exact(oracle):
    h = gpu(small(1, 8))
    rng = np.random.default_rng(1)
    n = 200_000
    ctr = rng.integers(0, 2**32, (n, 4), dtype=np.uint64).astype(np.uint32)
    ctr[0] = 0
    ctr[1] = 0xFFFFFFFF
    ctr[2:1000, 1:] = 0                   # the shape of real counters: group index, small fields
    ctr[2:1000, 3] = 0x47000000
    key = np.array([0x48414446, 0x9ABCDEF0], dtype=np.uint32)
    got = h.debug_philox(ctr, key)
    want = oracle.philox4x32_10_many(ctr, key)
    assert np.array_equal(got, want)
    for key in ([0, 0], [0xFFFFFFFF, 0xFFFFFFFF]):
        assert np.array_equal(h.debug_philox(ctr[:2000], key), oracle.philox4x32_10_many(ctr[:2000], key))


def test_normals_close_to_oracle(oracle):
    wl = small(4, 8, seed=0xABCDEF12345)
    h = gpu(wl)
    groups = np.concatenate([np.arange(50_000), [2**31, 2**32 - 1]]).astype(np.uint32)
    for step, dev in ((0, 0), (7, 3), (2**32 + 5, 1)):
        z = h.debug_normals(0, groups, step, dev)
        ref = np.stack([oracle.grad_normals(wl.seed, int(g), step, dev) for g in groups])
        err = np.abs(z.astype(np.float64) - ref.astype(np.float64)).max()
        print("max |z_gpu - z_cpu| (gradient normals, step %d): %.3e" % (step, err))
        # budget: lr * grad_std * err / (1 - momentum) must stay far below TOL_REL * max|x| ~ 5e-7
        assert err < 1e-5
        assert np.mean(np.abs(z - ref)) < 1e-6
    z = h.debug_normals(1, groups)
    ref = np.stack([oracle.init_normals(wl.seed, int(g)) for g in groups])
    err = np.abs(z.astype(np.float64) - ref.astype(np.float64)).max()
    print("max |z_gpu - z_cpu| (initial-model normals): %.3e" % err)
    assert err < 2e-6


# ---- K0 -----------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("P", [1, 2, 3, 4, 5, 31, 32, 33, 1000, 4099, 100_000])
def test_init_parity(oracle, P, dtype):
    wl = small(3, P, dtype=dtype)
    stride = (P + 31) // 32 * 32
    w = torch.full((3, stride), 7.0, dtype=torch.bfloat16 if dtype else torch.float32, device="cuda")
    m = torch.full((3, stride), 7.0, dtype=torch.float32, device="cuda")
    h = gpu(wl, w_ptr=w.data_ptr(), m_ptr=m.data_ptr(), row_stride_elems=stride)
    sim = make_sim(oracle, wl)
    h.synchronize()
    rows = [h.read_params(i) for i in range(3)]
    assert np.array_equal(rows[0], rows[1]) and np.array_equal(rows[0], rows[2])
    want = sim.read_params(0)
    if dtype == 0:
        assert_close_params(rows[0], want, "init")
        assert np.abs(rows[0] - want).max() <= 4e-8
    else:   # a last-bit difference of the fp32 normal can move the bf16 rounding by one step
        assert np.all(np.abs(rows[0] - want) <= bf16_ulp(want))
        assert np.mean(rows[0] != want) < 0.01
    assert not h.read_momentum(1).any()
    # padding between rows is zeroed, parameters are exactly what read_params returns
    wc = w.float().cpu().numpy()
    assert not wc[:, P:].any() and not m.cpu().numpy().any()
    assert np.array_equal(wc[2, :P], rows[2])
    v, s = h.get_versions()
    assert not v.any() and not s.any()


# ---- K1 -----------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("P", [1, 3, 4, 6, 1023, 1024, 4099, 70_001])
def test_local_step_parity(oracle, P, dtype):
    n = 5
    wl = small(n, P, dtype=dtype)
    h, sim = gpu(wl), make_sim(oracle, wl)
    rows = workloads.random_rows(n, P, seed=P)
    load_rows(h, sim, rows)
    # step counts of at most 2 take the one-row-per-block launch (fp32), larger ones the row walk
    calls = [([0, 1, 2, 3, 4], [1, 2, 3, 4, 8]), ([3, 1], [5, 0]), ([4], [1]), ([2, 0, 4, 1, 3], [2, 2, 1, 7, 3]),
             ([4, 2, 0, 1, 3], [1, 2, 1, 2, 2]), ([1, 3, 0], [2, 0, 1]), ([2, 4], [0, 0])]
    for ids, steps in calls:
        h.local_step(ids, steps, 0.01)
        sim.local_step(ids, steps, 0.01)
        for i in range(n):
            got, want = h.read_params(i), sim.read_params(i)
            if dtype == 0:
                assert_close_params(got, want, "w[%d]" % i)
            else:
                assert np.abs(got - want).max() <= 2 * bf16_ulp(np.abs(want).max()), i
                assert np.mean(got != want) < 0.02
            # momentum sees the generator's error directly: grad_std * max|dz| / (1 - mu), max|dz| < 1e-5
            m_tol = wl.grad_std * 1e-5 / (1.0 - wl.momentum)
            assert np.abs(h.read_momentum(i) - sim.read_momentum(i)).max() <= m_tol, i
        assert np.array_equal(h.get_versions()[0], sim.get_versions()[0])
        assert np.array_equal(h.get_versions()[1], sim.get_versions()[1])


def test_local_step_without_noise_is_bit_exact(oracle):
    """grad_std = 0: the update is pure fp32 fma arithmetic in a fixed order."""
    wl = small(4, 4099, grad_std=0.0, weight_decay=0.3, momentum=0.9)
    h, sim = gpu(wl), make_sim(oracle, wl)
    rows = workloads.random_rows(4, 4099, seed=3)
    load_rows(h, sim, rows)
    for _ in range(3):
        h.local_step([0, 1, 2, 3], [1, 2, 3, 4], 0.05)
        sim.local_step([0, 1, 2, 3], [1, 2, 3, 4], 0.05)
    for i in range(4):
        assert np.array_equal(h.read_params(i), sim.read_params(i))
        assert np.array_equal(h.read_momentum(i), sim.read_momentum(i))


def test_local_step_split_identity_and_determinism():
    wl = small(3, 20_003)
    a, b, c = gpu(wl), gpu(wl), gpu(wl)
    a.local_step([0, 1, 2], [3, 1, 0], 0.01)
    a.local_step([2, 0, 1], [6, 4, 2], 0.01)
    for h in (b, c):
        h.local_step([0, 1, 2], [7, 3, 6], 0.01)
    for i in range(3):
        assert np.array_equal(a.read_params(i), b.read_params(i))
        assert np.array_equal(a.read_momentum(i), b.read_momentum(i))
        assert np.array_equal(b.read_params(i), c.read_params(i))
    assert np.array_equal(a.get_versions()[1], b.get_versions()[1])


def test_local_step_high_step_counter(oracle):
    """Step counters beyond 2^32 index a different part of the gradient stream."""
    wl = small(2, 1001)
    h, sim = gpu(wl), make_sim(oracle, wl)
    start = np.array([2**32 - 2, 2**40 + 3], dtype=np.uint64)
    h.set_versions(step_counts=start)
    sim.set_versions(step_counts=start)
    h.local_step([0, 1], [4, 2], 0.01)
    sim.local_step([0, 1], [4, 2], 0.01)
    for i in range(2):
        assert_close_params(h.read_params(i), sim.read_params(i))
    assert np.array_equal(h.get_versions()[1], sim.get_versions()[1])


def test_local_step_untouched_rows_and_padding():
    P, n = 1001, 4
    stride = 1024
    w = torch.zeros((n, stride), device="cuda")
    m = torch.zeros((n, stride), device="cuda")
    h = gpu(small(n, P), w_ptr=w.data_ptr(), m_ptr=m.data_ptr(), row_stride_elems=stride)
    h.synchronize()
    w[:, P:] = 123.0        # canaries in the padding
    m[:, P:] = 321.0
    before = w.clone()
    h.local_step([1, 3], [2, 5], 0.01)
    h.aggregate([1, 3])
    h.broadcast(1, [0])
    h.stats(0)
    torch.cuda.synchronize()
    assert torch.all(w[:, P:] == 123.0) and torch.all(m[:, P:] == 321.0)
    assert torch.equal(w[2], before[2]) and not torch.equal(w[1], before[1])


# ---- K2 -----------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("P", [1, 5, 2048, 4099, 66_667])
def test_aggregate_bit_exact_for_every_k(oracle, P, dtype):
    n = 32
    wl = small(n, P, dtype=dtype)
    h, sim = gpu(wl), make_sim(oracle, wl)
    rows = workloads.random_rows(n, P, seed=17 + P)
    rng = np.random.default_rng(P)
    ks = range(1, n + 1) if P <= 4099 else (1, 2, 3, 4, 7, 8, 16, 17, 32)
    for k in ks:
        load_rows(h, sim, rows)
        sel = rng.permutation(n)[:k].astype(np.int32)
        h.aggregate(sel)
        sim.aggregate(sel)
        for i in set(int(s) for s in sel) | {int((sel[0] + 1) % n)}:
            assert np.array_equal(h.read_params(i), sim.read_params(i)), (k, i)
        assert np.array_equal(h.get_versions()[0], sim.get_versions()[0])
    assert not h.read_momentum(0).any()


def test_aggregate_version_weighted_mode(oracle):
    wl = small(8, 4099, weight_mode=1, version_scale=0.5)
    h, sim = gpu(wl), make_sim(oracle, wl)
    rows = workloads.random_rows(8, 4099, seed=4)
    load_rows(h, sim, rows)
    versions = [9, 1, 4, 4, 6, 2, 8, 3]
    for o in (h, sim):
        o.set_versions(versions)
    sel = [6, 1, 3, 0, 5]
    a = h.aggregation_weights(sel)
    assert np.array_equal(a, sim.aggregation_weights(sel))
    assert abs(float(a.astype(np.float64).sum()) - 1.0) < 2e-7 and a.std() > 0.01
    h.aggregate(sel)
    sim.aggregate(sel)
    for i in range(8):
        assert np.array_equal(h.read_params(i), sim.read_params(i))
    assert np.array_equal(h.get_versions()[0], sim.get_versions()[0])
    # caller-supplied (e.g. predicted) versions
    v2 = [3.0, 3.5, 1.0, 8.0, 2.0, 2.5, 9.0, 4.0]
    assert np.array_equal(h.aggregation_weights(sel, v2), sim.aggregation_weights(sel, v2))


@pytest.mark.parametrize("dtype", [0, 1])
def test_broadcast(oracle, dtype):
    wl = small(6, 4099, dtype=dtype)
    h, sim = gpu(wl), make_sim(oracle, wl)
    load_rows(h, sim, workloads.random_rows(6, 4099, seed=8))
    for o in (h, sim):
        o.set_versions([5, 1, 2, 3, 4, 9])
        o.broadcast(5, [0, 2, 3])
        o.broadcast(1, [])
    for i in range(6):
        assert np.array_equal(h.read_params(i), sim.read_params(i))
    assert list(h.get_versions()[0]) == [9, 1, 9, 9, 4, 9]


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("P", [1, 5, 1023, 4099, 600_011])
def test_integrate_bit_exact(oracle, P, dtype):
    """The mix of a received model into the receivers' own: fixed fp32 arithmetic (one rounded
    product, one fused multiply-add), so every stored bit equals the oracle's - for every number of
    receivers, on ragged rows, with fp32 and bf16 storage."""
    n = 32 if P <= 4099 else 6
    wl = small(n, P, dtype=dtype)
    h, sim = gpu(wl), make_sim(oracle, wl)
    load_rows(h, sim, workloads.random_rows(n, P, seed=P + 3))
    versions = np.arange(n, dtype=np.uint32)[::-1].copy()
    rng = np.random.default_rng(P)
    calls = [(0, [1], 0.5), (2, [0, 1, 3, 4, 5], 0.25), (1, [5, 0], 1.0), (3, [2], 0.0), (4, [], 0.7)]
    if n == 32:
        calls += [(7, [i for i in range(32) if i != 7], 0.1),
                  (31, list(rng.permutation(31)[:17]), 0.9)]
    for o in (h, sim):
        o.set_versions(versions)
        for src, dst, beta in calls:
            o.integrate(src, dst, beta)
    for i in range(n):
        assert np.array_equal(h.read_params(i), sim.read_params(i)), i
        assert not h.read_momentum(i).any()
    assert np.array_equal(h.get_versions()[0], sim.get_versions()[0])


def test_integrate_rejects_bad_arguments_and_leaves_the_arena_alone():
    wl = small(4, 1000)
    h = gpu(wl)
    before = [h.read_params(i).copy() for i in range(4)]
    for args in ((0, [0], 0.5), (0, [1, 1], 0.5), (4, [1], 0.5), (0, [7], 0.5), (0, [1], -0.1),
                 (0, [1], 1.01), (0, [1], float("nan"))):
        with pytest.raises(binding.HadflError) as e:
            h.integrate(*args)
        assert e.value.code == binding.ERR_INVALID
    for i in range(4):
        assert np.array_equal(h.read_params(i), before[i])


# ---- K3 -----------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("n,P", [(1, 1), (4, 1003), (32, 4099), (7, 300_001), (16, 2_000_003)])
def test_stats(oracle, n, P, dtype):
    wl = small(n, P, dtype=dtype)
    h, sim = gpu(wl), make_sim(oracle, wl)
    rows = workloads.random_rows(n, P, seed=n)
    load_rows(h, sim, rows)
    for ref in {0, n - 1, n // 2}:
        n2, d2 = h.stats(ref)
        wn2, wd2 = sim.stats(ref)
        assert np.allclose(n2, wn2, rtol=1e-5, atol=0)
        assert np.allclose(d2, wd2, rtol=1e-5, atol=0)
        assert d2[ref] == 0.0
        again = h.stats(ref)
        assert np.array_equal(again[0], n2) and np.array_equal(again[1], d2)     # reproducible


# ---- argument checks ----------------------------------------------------------------------------
def test_invalid_arguments_are_rejected_and_change_nothing():
    wl = small(4, 1000)
    h = gpu(wl)
    h.local_step([0, 1, 2, 3], [1, 1, 1, 1], 0.01)
    before = [h.read_params(i) for i in range(4)]
    vb = h.get_versions()
    E = binding.HadflError
    for ids, steps in (([0, 0], [1, 1]), ([4], [1]), ([-1], [1]), ([0], [-1]), ([], []), ([0, 1, 2, 3, 0], [1] * 5)):
        with pytest.raises(E):
            h.local_step(ids, steps, 0.01)
    for sel in ([], [1, 1], [4], [0, 1, 2, 3, 1]):
        with pytest.raises(E):
            h.aggregate(sel)
    for k in (0, 5, -2):
        with pytest.raises(E):
            h.select(0, k, 1)
    with pytest.raises(E):
        h.broadcast(0, [0])
    with pytest.raises(E):
        h.broadcast(4, [0])
    with pytest.raises(E):
        h.stats(4)
    with pytest.raises(E):
        h.read_params(0, count=1001)
    with pytest.raises(E):
        h.read_params(7)
    assert all(np.array_equal(h.read_params(i), before[i]) for i in range(4))
    assert np.array_equal(h.get_versions()[0], vb[0]) and np.array_equal(h.get_versions()[1], vb[1])
    for bad in (dict(n_devices=0), dict(n_devices=33), dict(n_params=0), dict(dtype=2), dict(weight_mode=5),
                dict(row_stride_elems=996), dict(row_stride_elems=1004), dict(version_scale=0.0)):
        args = dict(n_devices=4, n_params=1000)
        args.update(bad)
        with pytest.raises(E):
            binding.Hadfl(**args)
    h.set_available([1, 0, 0, 1])
    with pytest.raises(E):
        h.select(0, 3, 1)
    assert sorted(h.select(0, 2, 1)) == [0, 3]


def test_select_through_handle_matches_oracle(oracle):
    wl = small(16, 64, version_scale=0.125)
    h, sim = gpu(wl), make_sim(oracle, wl)
    rng = np.random.default_rng(0)
    for r in range(100):
        v = rng.integers(0, 200, 16).astype(np.uint32)
        mask = (rng.random(16) < 0.8).astype(np.uint8)
        mask[:4] = 1
        for o in (h, sim):
            o.set_versions(v)
            o.set_available(mask)
        assert np.array_equal(h.select_probs(), sim.select_probs())
        assert np.array_equal(h.select(r, 4, 0xFEED), sim.select(r, 4, 0xFEED))
        pv = rng.uniform(0, 30, 16)
        assert np.array_equal(h.select(r, 3, 5, pv), sim.select(r, 3, 5, pv))


def test_checkpoint_resume_is_exact():
    """Restoring parameters, momentum, versions and step counters continues the run bit for bit."""
    wl = small(3, 5003)
    a = gpu(wl)
    a.local_step([0, 1, 2], [2, 3, 1], 0.01)
    a.aggregate([0, 2])
    state = [(a.read_params(i), a.read_momentum(i)) for i in range(3)]
    v, s = a.get_versions()
    b = gpu(wl)
    for i, (w, m) in enumerate(state):
        b.write_params(i, w)
        b.write_momentum(i, m)
    b.set_versions(v, s)
    for h in (a, b):
        h.local_step([2, 0, 1], [4, 1, 2], 0.01)
        h.aggregate(h.select(1, 2, 9))
    for i in range(3):
        assert np.array_equal(a.read_params(i), b.read_params(i))
        assert np.array_equal(a.read_momentum(i), b.read_momentum(i))


def test_state_errors():
    """Calls that are not valid in the handle's state say so and change nothing."""
    wl = small(2, 1000)
    h = gpu(wl)
    with pytest.raises(binding.HadflError) as e:
        h.stats_read()                      # nothing enqueued yet
    assert e.value.code == binding.ERR_STATE
    h.set_versions(step_counts=np.array([2**56 - 3, 0], dtype=np.uint64))
    before = h.read_params(0)
    with pytest.raises(binding.HadflError) as e:
        h.local_step([0, 1], [4, 1], 0.01)  # device 0's gradient stream would run past 2^56 steps
    assert e.value.code == binding.ERR_STATE
    with pytest.raises(binding.HadflError) as e:
        h.round([0, 1], [4, 1], 0.01, 0, 1, 3)
    assert e.value.code == binding.ERR_STATE
    with pytest.raises(binding.HadflError):
        h.set_versions(step_counts=np.array([2**56, 0], dtype=np.uint64))
    assert np.array_equal(h.read_params(0), before)
    assert list(h.get_versions()[1]) == [2**56 - 3, 0]
    h.local_step([0, 1], [2, 1], 0.01)      # up to the limit is fine
    assert list(h.get_versions()[1]) == [2**56 - 1, 1]


@pytest.mark.parametrize("dtype", [0, 1])
def test_overlapped_backup_is_a_snapshot(dtype):
    """hadfl_backup_begin captures the row as it is at that point of the stream, even though later
    rounds (enqueued before the copy has finished) rewrite it."""
    wl = small(3, 3_000_003, dtype=dtype)
    h = gpu(wl)
    h.local_step([0, 1, 2], [1, 2, 1], 0.01)
    want = h.read_params(1)
    buf = torch.empty(wl.n_params, dtype=torch.float32).pin_memory()
    h.backup_begin(1, buf)
    for r in range(3):                      # keeps the GPU busy rewriting row 1 while the copy runs
        h.round([0, 1, 2], [2, 3, 1], 0.01, r, 2, 11)
    h.backup_wait()
    assert np.array_equal(buf.numpy(), want)
    assert not np.array_equal(h.read_params(1), want)
    h.backup_wait()                          # nothing in flight: no-op
    part = np.empty(1000, dtype=np.float32)
    h.backup_begin(1, part, count=1000)      # pageable memory works too
    h.backup_begin(2, buf)                   # a second begin first finishes the one in flight
    h.backup_wait()
    assert np.array_equal(part, h.read_params(1)[:1000]) and np.array_equal(buf.numpy(), h.read_params(2))
    with pytest.raises(binding.HadflError):
        h.backup_begin(3, buf)
