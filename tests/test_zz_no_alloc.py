"""hadfl_stats_noalloc: the statistics kernel for callers that are not allowed to allocate device
memory (their memory belongs to another allocator, or an allocation's device-wide synchronisation
is unaffordable where they run).  It takes no handle, keeps its scratch in a fixed array inside the
library and works on raw device pointers.  Checked here against hadfl_stats on the same arena, on
two calls in a row (the second one finds the first one's leftovers in the shared scratch), and
against the CPU oracle's double-precision sums.

This file is collected last on purpose: if it fails under `pytest -x`, every other test has run."""
import numpy as np
import pytest
import torch

from gpu_common import require_gpu
from oracle_driver import make_sim
from paper_2111_08274_b200 import binding, runtime, workloads
from paper_2111_08274_b200.workloads import Workload

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def noalloc_stats(arena, ref, out):
    wl = arena.wl
    rc = binding.hadfl_stats_noalloc(arena.w.data_ptr(), wl.dtype, wl.n_devices, wl.n_params,
                                     arena.stride, ref, out.data_ptr(), arena.stream.cuda_stream)
    assert rc == binding.OK, rc
    torch.cuda.synchronize()
    res = out.cpu().numpy()
    return res[: wl.n_devices], res[wl.n_devices:]


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("n,P", [(4, 100_003), (16, 1_500_001), (32, 4099), (1, 7)])
def test_matches_hadfl_stats_on_two_calls_in_a_row(oracle, n, P, dtype):
    wl = Workload("na", n, P, min(2, n), 1, "fixed", tuple(1 + i % 3 for i in range(n)),
                  grad_std=1e-2, dtype=dtype, seed=workloads.BASE_SEED + 77)
    arena = runtime.Arena(wl)
    sim = make_sim(oracle, wl)          # its replicas are overwritten with the arena's values below
    out = torch.full((2 * n,), -1.0, dtype=torch.float32, device=arena.device)   # caller's buffer
    arena.h.local_step(wl.device_ids(), wl.steps_for_round(0), wl.lr)
    for call, ref in enumerate((0, n - 1)):
        want_n2, want_d2 = arena.h.stats(ref)
        got_n2, got_d2 = noalloc_stats(arena, ref, out)
        assert np.allclose(got_n2, want_n2, rtol=1e-5, atol=0), (call, got_n2, want_n2)
        assert np.allclose(got_d2, want_d2, rtol=1e-5, atol=0), (call, got_d2, want_d2)
        assert got_d2[ref] == 0.0
        # the oracle sums, in double, the very values the arena holds (read back bit for bit)
        for i in range(n):
            sim.write_params(i, arena.h.read_params(i))
        on2, od2 = sim.stats(ref)
        assert np.allclose(got_n2, on2, rtol=1e-5, atol=0), (call, got_n2, on2)
        assert np.allclose(got_d2, od2, rtol=1e-5, atol=1e-30), (call, got_d2, od2)
        # the arena moves on between the two calls, so stale scratch could not go unnoticed
        arena.h.local_step(wl.device_ids(), wl.steps_for_round(1), wl.lr)
    arena.close()


def test_limits_and_bad_arguments_are_refused_without_touching_the_output():
    wl = Workload("na", 4, 4099, 2, 1, "fixed", (1, 1, 1, 1), seed=workloads.BASE_SEED + 78)
    arena = runtime.Arena(wl)
    out = torch.full((8,), -1.0, dtype=torch.float32, device=arena.device)
    w, s, st = arena.w.data_ptr(), arena.stream.cuda_stream, arena.stride
    f = binding.hadfl_stats_noalloc
    assert f(w, 0, 33, 4099, st, 0, out.data_ptr(), s) == binding.ERR_TOO_LARGE
    assert f(w, 0, 4, 2**31, 2**31 + 8, 0, out.data_ptr(), s) == binding.ERR_TOO_LARGE
    assert f(w, 0, 4, 4099, st, 4, out.data_ptr(), s) == binding.ERR_INVALID
    assert f(w, 0, 4, 4099, 4100, 0, out.data_ptr(), s) == binding.ERR_INVALID
    assert f(w, 2, 4, 4099, st, 0, out.data_ptr(), s) == binding.ERR_INVALID
    assert f(None, 0, 4, 4099, st, 0, out.data_ptr(), s) == binding.ERR_INVALID
    assert f(w + 4, 0, 4, 4099, st, 0, out.data_ptr(), s) == binding.ERR_INVALID
    assert f(w, 0, 4, 4099, st, 0, None, s) == binding.ERR_INVALID
    # buffers that are not device memory of the current GPU are refused on the host, not in the kernel
    host_w = np.zeros(4 * st, dtype=np.float32)
    host_out = np.zeros(8, dtype=np.float32)
    aligned = host_w.ctypes.data + (-host_w.ctypes.data) % 16
    assert f(aligned, 0, 1, 7, 8, 0, out.data_ptr(), s) == binding.ERR_INVALID
    assert f(w, 0, 4, 4099, st, 0, host_out.ctypes.data, s) == binding.ERR_INVALID
    pinned = torch.zeros(8, dtype=torch.float32).pin_memory()
    assert f(w, 0, 4, 4099, st, 0, pinned.data_ptr(), s) == binding.ERR_INVALID
    assert f(w, 0, 4, 4099, st, 0, out.data_ptr(), s) == binding.OK      # and a later good call still works
    torch.cuda.synchronize()
    assert torch.all(out != -1.0)
    out.fill_(-1.0)
    torch.cuda.synchronize()
    assert torch.all(out == -1.0)
    arena.close()
