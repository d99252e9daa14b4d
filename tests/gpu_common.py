"""Shared helpers of the GPU parity tests."""
import numpy as np
import pytest
import torch

TOL_REL = 2e-6      # max|gpu - cpu| <= TOL_REL * max|x| for fp32 parameters


def require_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2111_08274_b200 import runtime
    runtime.ensure_built()


def assert_close_params(got, want, what=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    scale = np.abs(want).max()
    err = np.abs(got - want).max() if got.size else 0.0
    assert err <= TOL_REL * scale, "%s: max err %.3e > %.1e * %.3e" % (what, err, TOL_REL, scale)
    return err / scale if scale > 0 else 0.0


def bf16_ulp(x):
    """Spacing of bf16 numbers at |x| (fp32 array in, fp64 array out)."""
    bits = np.abs(np.asarray(x, dtype=np.float32)).view(np.uint32) & np.uint32(0x7F800000)
    e = (bits >> 23).astype(np.int32) - 127
    return np.ldexp(1.0, np.maximum(e, -126) - 7)
