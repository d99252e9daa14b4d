"""Pins for the oracle's local update (Eq. 3, Algorithm 1; momentum / weight decay in the
PyTorch-SGD convention)."""
import numpy as np
import pytest
import torch

P = 2051  # ragged: 2051 mod 4 = 3


def noise(oracle, seed, P, step, device):
    n_groups = (P + 3) // 4
    z = np.concatenate([oracle.grad_normals(seed, g, step, device) for g in range(n_groups)])
    return z[:P]


def test_zero_gradient_leaves_the_model_unchanged(oracle):
    s = oracle.Sim(2, P, seed=1, grad_std=0.0, weight_decay=0.0)
    w0 = s.read_params(0).copy()
    s.local_step([0, 1], [5, 2], 0.01)
    assert np.array_equal(s.read_params(0), w0) and np.array_equal(s.read_params(1), w0)
    assert not s.read_momentum(0).any()
    v, sc = s.get_versions()
    assert list(v) == [5, 2] and list(sc) == [5, 2]


def test_plain_sgd_is_eq3(oracle):
    """momentum = 0, wd = 0: w_E = w_0 - lr * sum_e g_e (Eq. 3 applied E times)."""
    E, lr, gstd, seed = 6, 0.01, 1e-2, 21
    s = oracle.Sim(3, P, seed=seed, grad_std=gstd, momentum=0.0, weight_decay=0.0)
    w0 = s.read_params(2).astype(np.float64)
    s.local_step([2], [E], lr)
    g = sum(np.float64(np.float32(gstd) * noise(oracle, seed, P, e, 2)) for e in range(E))
    want = w0 - np.float64(np.float32(lr)) * g
    got = s.read_params(2).astype(np.float64)
    assert np.abs(got - want).max() <= E * np.spacing(np.float32(0.3))   # E roundings of w at most
    # the other devices did not move
    assert np.array_equal(s.read_params(0).astype(np.float64), w0)


def test_weight_decay_only_is_geometric(oracle):
    """grad_std = 0, momentum = 0: w_E = w_0 (1 - lr*wd)^E."""
    E, lr, wd = 8, 0.1, 0.25
    s = oracle.Sim(1, P, seed=3, grad_std=0.0, momentum=0.0, weight_decay=wd)
    w0 = s.read_params(0).astype(np.float64)
    s.local_step([0], [E], lr)
    want = w0 * (1.0 - np.float64(np.float32(lr)) * wd) ** E
    assert np.allclose(s.read_params(0), want, rtol=E * 1.2e-7, atol=0)


def test_momentum_weight_decay_recursion_closed_form(oracle):
    """grad_std = 0: (w, m) follows a linear 2x2 recursion; compare with its matrix power."""
    E, lr, mu, wd = 7, 0.05, 0.9, 0.3
    s = oracle.Sim(1, P, seed=4, grad_std=0.0, momentum=mu, weight_decay=wd)
    w0 = s.read_params(0).astype(np.float64)
    s.local_step([0], [E], lr)
    lr64, mu64, wd64 = (np.float64(np.float32(x)) for x in (lr, mu, wd))
    # m' = mu m + wd w ; w' = w - lr m'
    A = np.array([[1.0 - lr64 * wd64, -lr64 * mu64], [wd64, mu64]])
    M = np.linalg.matrix_power(A, E)
    assert np.allclose(s.read_params(0), M[0, 0] * w0, rtol=3e-6, atol=0)
    assert np.allclose(s.read_momentum(0), M[1, 0] * w0, rtol=3e-6, atol=1e-12)


@pytest.mark.parametrize("dtype64", [False, True])
def test_matches_torch_sgd(oracle, dtype64):
    """The update convention is torch.optim.SGD's (momentum, weight_decay, dampening 0)."""
    E, lr, mu, wd, gstd, seed, dev = 5, 0.01, 0.9, 5e-4, 1e-2, 31, 1
    s = oracle.Sim(2, P, seed=seed, grad_std=gstd, momentum=mu, weight_decay=wd)
    tdt = torch.float64 if dtype64 else torch.float32
    p = torch.nn.Parameter(torch.from_numpy(s.read_params(dev).copy()).to(tdt))
    opt = torch.optim.SGD([p], lr=float(np.float32(lr)), momentum=float(np.float32(mu)),
                          weight_decay=float(np.float32(wd)))
    for e in range(E):
        p.grad = torch.from_numpy(np.float32(gstd) * noise(oracle, seed, P, e, dev)).to(tdt)
        opt.step()
    s.local_step([dev], [E], lr)
    got = s.read_params(dev).astype(np.float64)
    want = p.detach().to(torch.float64).numpy()
    tol = E * 1.5e-8         # one rounding of w (half an ulp of 0.25..0.5) per step on either side
    assert np.abs(got - want).max() < tol
    buf = opt.state[p]["momentum_buffer"].to(torch.float64).numpy()
    assert np.abs(s.read_momentum(dev) - buf).max() < tol


def test_split_steps_equal_one_call(oracle):
    """Counter-based gradients: a then b steps is bit-identical to a+b steps in one call."""
    kw = dict(seed=8, grad_std=1e-2)
    a, b = oracle.Sim(2, P, **kw), oracle.Sim(2, P, **kw)
    a.local_step([0, 1], [3, 1], 0.01)
    a.local_step([1, 0], [2, 4], 0.01)
    b.local_step([0, 1], [7, 3], 0.01)
    for i in (0, 1):
        assert np.array_equal(a.read_params(i), b.read_params(i))
        assert np.array_equal(a.read_momentum(i), b.read_momentum(i))
    assert np.array_equal(a.get_versions()[1], b.get_versions()[1])


def test_devices_draw_different_gradients(oracle):
    s = oracle.Sim(2, P, seed=8, grad_std=1e-2)
    s.local_step([0, 1], [1, 1], 0.01)
    assert not np.array_equal(s.read_params(0), s.read_params(1))
    # the mean gradient over the vector is ~0 and its std is grad_std
    g = s.read_momentum(0).astype(np.float64) - 5e-4 * oracle.Sim(1, P, seed=8).read_params(0)
    assert abs(g.std() / 1e-2 - 1) < 0.1


def test_zero_steps_and_argument_checks(oracle):
    s = oracle.Sim(3, P, seed=8)
    w0 = s.read_params(1).copy()
    s.local_step([1], [0], 0.01)
    assert np.array_equal(s.read_params(1), w0)
    for ids, steps in (([0, 0], [1, 1]), ([3], [1]), ([-1], [1]), ([0], [-1]), ([], [])):
        with pytest.raises(oracle.OracleError):
            s.local_step(ids, steps, 0.01)


def test_bf16_storage_rounds_once_per_call(oracle):
    kw = dict(seed=8, grad_std=1e-2, dtype=1)
    s, f = oracle.Sim(1, P, **kw), oracle.Sim(1, P, seed=8, grad_std=1e-2)
    w0 = s.read_params(0)
    assert np.array_equal(w0, torch.from_numpy(f.read_params(0)).to(torch.bfloat16).float().numpy())
    # run the fp32 simulation from the bf16 start: bf16 result == rounding of its result
    f.write_params(0, w0)
    s.local_step([0], [3], 0.01)
    f.local_step([0], [3], 0.01)
    want = torch.from_numpy(f.read_params(0)).to(torch.bfloat16).float().numpy()
    assert np.array_equal(s.read_params(0), want)
    assert np.array_equal(s.read_momentum(0), f.read_momentum(0))
