"""The round-by-round runner (python -m paper_2111_08274_b200.run): its log must describe the same
run whether a round is one fused call or four separate ones, and the planned versions it feeds to
the selection must be the oracle's Eq. 7 predictions of the logged version history."""
import json

import numpy as np
import pytest

from gpu_common import require_gpu
from paper_2111_08274_b200 import run

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def log_of(tmp_path, name, *args):
    path = tmp_path / name
    run.main(["--workload", "c1", "--n-params", "20003", "--rounds", "8", "--jsonl", str(path), *args])
    return [json.loads(line) for line in path.read_text().splitlines()]


def test_fused_and_separate_runs_log_the_same_rounds(tmp_path):
    fused = log_of(tmp_path, "fused.jsonl")
    plain = log_of(tmp_path, "plain.jsonl", "--separate")
    assert len(fused) == len(plain) == 8
    for f, p in zip(fused, plain):
        for key in ("round", "selected", "steps", "versions", "step_counters", "global_sync"):
            assert f[key] == p[key], key
        assert np.allclose(f["selection_probabilities"], p["selection_probabilities"], rtol=0, atol=0)
        assert abs(sum(f["selection_probabilities"]) - 1.0) < 1e-12
        assert np.allclose(f["norm2"], p["norm2"], rtol=2e-6)
        assert np.allclose(f["divergence2"], p["divergence2"], rtol=2e-6, atol=1e-30)
        assert all(f["divergence2"][s] == 0.0 for s in f["selected"])
        assert f["gpu_ms"] > 0.0


def test_planned_versions_are_the_oracles_predictions(tmp_path, oracle):
    alpha = 0.6
    rows = log_of(tmp_path, "planned.jsonl", "--predict", str(alpha))
    assert rows[0]["planned_versions"] is None and rows[1]["planned_versions"] is None
    history = [[] for _ in range(4)]
    for r, row in enumerate(rows):
        if r >= 2:
            want = [oracle.predict_version(history[i], alpha, 1.0) for i in range(4)]
            assert row["planned_versions"] == want
            # the probabilities logged are Eq. 8 on those planned versions
            assert np.array_equal(row["selection_probabilities"], oracle.select_probs(np.array(want)))
        for i in range(4):
            history[i].append(float(row["versions"][i]))
