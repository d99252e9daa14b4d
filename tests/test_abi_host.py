"""The C-ABI library loads without a GPU, exports what include/hadfl.h declares, and its host-only
planning functions (Eq. 8 selection, Eq. 7 prediction) agree with the oracle."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2111_08274_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2111_08274_b200 import build
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hadfl.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hadfl_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert "hadfl_init" in names and "hadfl_aggregate" in names and len(names) >= 25
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.SYMBOLS) == names


def test_config_struct_layout_matches_the_header():
    c = binding.hadfl_config
    offs = {n: getattr(c, n).offset for n, _ in c._fields_}
    assert offs == {"n_devices": 0, "n_params": 8, "dtype": 16, "momentum": 20, "weight_decay": 24,
                    "grad_std": 28, "init_std": 32, "seed": 40, "version_scale": 48, "weight_mode": 56,
                    "w_ptr": 64, "m_ptr": 72, "row_stride_elems": 80, "cuda_stream": 88,
                    "m_dtype": 96, "rounding": 100}
    assert C.sizeof(c) == 104


def test_host_selection_matches_oracle_bit_for_bit(lib, oracle):
    rng = np.random.default_rng(99)
    for case in range(300):
        n = int(rng.integers(1, 33))
        scale = [1.0, 0.125, 3.0][case % 3]
        x = rng.integers(0, 40, n).astype(np.float64) * scale
        avail = None
        if case % 4 == 0 and n > 1:
            avail = (rng.random(n) < 0.7).astype(np.uint8)
            avail[int(rng.integers(n))] = 1
        n_avl = n if avail is None else int(avail.sum())
        assert np.array_equal(binding.hadfl_selection_probs(x, avail), oracle.select_probs(x, avail))
        k = int(rng.integers(1, n_avl + 1))
        r, seed = int(rng.integers(0, 2**40)), int(rng.integers(0, 2**63))
        got = binding.hadfl_selection_draw(x, k, r, seed, avail)
        assert np.array_equal(got, oracle.select(x, k, r, seed, avail)), case


def test_host_selection_underflow_fallback_matches_oracle(lib, oracle):
    x = [1000.0] * 3 + [0.0] * 5
    for r in range(200):
        assert np.array_equal(binding.hadfl_selection_draw(x, 6, r, 3), oracle.select(x, 6, r, 3))


def test_host_selection_rejects_bad_arguments(lib):
    for k in (0, 5, -1):
        with pytest.raises(binding.HadflError):
            binding.hadfl_selection_draw([1.0, 2.0, 3.0, 4.0], k, 0, 1)
    with pytest.raises(binding.HadflError):
        binding.hadfl_selection_draw([1.0, 2.0], 2, 0, 1, avail=[1, 0])
    with pytest.raises(binding.HadflError):
        binding.hadfl_selection_probs([1.0, 2.0], avail=[0, 0])
    with pytest.raises(binding.HadflError):
        binding.hadfl_selection_probs(np.zeros(33))


def test_predictor_matches_oracle(lib, oracle):
    rng = np.random.default_rng(5)
    for _ in range(50):
        series = np.cumsum(rng.integers(1, 9, int(rng.integers(1, 30)))).astype(np.float64)
        alpha, m = float(rng.uniform(0.05, 0.95)), float(rng.integers(0, 5))
        assert binding.hadfl_predict_version(series, alpha, m) == oracle.predict_version(series, alpha, m)
    with pytest.raises(binding.HadflError):
        binding.hadfl_predict_version([1.0], 1.0)


def test_no_handle_is_rejected_not_crashed(lib):
    assert lib.hadfl_synchronize(None) == binding.ERR_INVALID
    assert lib.hadfl_destroy(None) == binding.OK
    assert lib.hadfl_init(None, None) == binding.ERR_INVALID


def test_statistics_grid_rule_and_its_cap(lib):
    """The grid rule of the statistics kernel as a host function: one wave of 8 blocks per SM split
    over the rows, at most one block per 16 KB chunk of a row, and the block cap that bounds the
    scratch of hadfl_stats_noalloc (which a 148-SM GPU never reaches, a larger one would)."""
    from paper_2111_08274_b200 import binding
    f = binding.hadfl_stats_grid_lanes
    big = 1 << 30
    assert f(148, 8, big) == 148                       # 1184 resident blocks over 8 rows
    assert f(148, 32, big) == 37
    assert f(148, 32, big, 0, 2048) == 37              # the cap does not bind on 148 SMs
    assert f(148, 1, big, 0, 2048) == 1184
    assert f(148, 8, 4096) == 1 and f(148, 8, 4097) == 2 and f(148, 8, 1) == 1   # one block per 4096 fp32 values
    assert f(148, 8, 8192, 1) == 1 and f(148, 8, 8193, 1) == 2                   # ... or 8192 bf16 values
    for sms, n in ((300, 8), (300, 32), (1024, 3), (257, 1)):                    # beyond 256 SMs the cap binds
        lanes = f(sms, n, big, 0, 2048)
        assert lanes * n <= 2048 < (lanes + 1) * n, (sms, n, lanes)
        assert f(sms, n, big) * n >= 8 * sms
    assert f(0, 8, big) == 0 and f(148, 33, big) == 0 and f(148, 8, 0) == 0 and f(148, 8, big, 2) == 0


def test_debug_build_range_predicate(lib):
    """[addr, addr + nbytes) inside [lo, hi): the predicate the debug build's kernels apply to every
    access, including its corner cases near the ends of the range and of the address space."""
    from paper_2111_08274_b200 import binding
    f = binding.hadfl_debug_range_holds
    lo, hi = 0x7F0000001000, 0x7F0000002000
    assert f(lo, hi, lo, 16) and f(lo, hi, hi - 16, 16) and f(lo, hi, lo, hi - lo) and f(lo, hi, hi, 0)
    assert not f(lo, hi, lo - 1, 16) and not f(lo, hi, hi - 15, 16) and not f(lo, hi, hi, 1)
    assert not f(lo, hi, lo, hi - lo + 1) and not f(lo, hi, 0, 16) and not f(lo, hi, hi + 4096, 4)
    top = 2**64 - 1
    assert not f(lo, hi, top - 3, 16) and not f(lo, hi, lo, top)          # no wrap-around
    assert f(top - 64, top, top - 16, 16) and not f(top - 64, top, top - 8, 16)
    assert not f(hi, lo, lo, 0)                                           # an empty / inverted range holds nothing
    assert not binding.hadfl_debug_build()                                # the library under test is the normal build
