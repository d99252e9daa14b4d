"""The debug build (libhadfl_debug.so, -DHADFL_DEBUG): kernels check every arena access and every
scratch store against the address ranges the handle registered, skip what falls outside and record
it; synchronising calls then fail with HADFL_ERR_STATE.  This test runs GPU parity tests of the
other files in a child process that loads the debug build instead of the normal one: they must pass
unchanged (same results, and no access out of range anywhere - every one of them ends in calls that
synchronise).  No test provokes an out-of-range access on the GPU; the range predicate itself is
unit-tested on the host (tests/test_abi_host.py).

HADFL_DEBUG_SUITE=full runs every GPU test file in the child instead of the selection below (the
whole suite passes on the debug build, in about the time the normal build takes)."""
import os
import subprocess
import sys

import pytest

from gpu_common import require_gpu

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))
SELECTION = ["test_gpu_round.py", "test_gpu_kernels.py", "test_gpu_rounding.py", "test_gpu_groups.py",
             "test_gpu_run.py", "test_zz_no_alloc.py",
             "test_gpu_configs.py::test_c1_full_arena_every_round",
             "test_gpu_configs.py::test_c1_ragged_tail_full_arena",
             "test_gpu_configs.py::test_c2_shrunk_full_arena",
             "test_gpu_configs.py::test_c5_smallest_size_full_arena_first_rounds",
             "test_gpu_configs.py::test_c2_full_size_fused_round_sampled_columns",
             "test_gpu_configs.py::test_rows_longer_than_two_to_the_31_elements",
             "test_gpu_fused_full_size.py"]


def test_gpu_tests_pass_on_the_debug_build_with_no_access_out_of_range():
    require_gpu()
    if os.environ.get("HADFL_LIBRARY"):
        pytest.skip("already running inside the debug-build child process")
    from paper_2111_08274_b200 import build
    lib = build.build(debug=True)
    env = dict(os.environ, HADFL_LIBRARY=lib)
    probe = subprocess.run([sys.executable, "-c",
                            "from paper_2111_08274_b200 import binding; print(int(binding.hadfl_debug_build()))"],
                           cwd=os.path.dirname(HERE), env=env, capture_output=True, text=True)
    assert probe.returncode == 0 and probe.stdout.strip() == "1", probe.stderr[-2000:]
    if os.environ.get("HADFL_DEBUG_SUITE") == "full":
        targets = [os.path.join(HERE, f) for f in sorted(os.listdir(HERE))
                   if f.startswith("test_") and f.endswith(".py") and f != os.path.basename(__file__)]
    else:
        targets = [os.path.join(HERE, t) for t in SELECTION]
    run = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider"] + targets,
                         cwd=os.path.dirname(HERE), env=env, capture_output=True, text=True)
    assert run.returncode == 0, run.stdout[-4000:] + run.stderr[-2000:]
