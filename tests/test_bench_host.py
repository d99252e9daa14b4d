"""Host-side logic of bench.py that needs no GPU: how many timed regions are run, which workloads
the sweep covers, how per-kernel figures are formed, and that the table printer reads a line back."""
import importlib.util
import json
import os

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_timed_region_is_repeated_until_enough_time_has_been_sampled(bench):
    assert bench.repeats_for(0.0087, 0.5) == 58          # 20 rounds of 0.43 ms: 58 regions reach half a second
    assert bench.repeats_for(0.8, 0.5) == 1 and bench.repeats_for(0.5, 0.5) == 1
    assert bench.repeats_for(0.2, 0.5) == 3
    assert bench.repeats_for(1e-6, 0.5) == 400           # capped
    assert bench.repeats_for(0.0, 0.5) == 1 and bench.repeats_for(0.01, 0.0) == 1


def test_sweep_sets(bench):
    default = [w.name for w in bench.sweep_cases("default")]
    assert default[:2] == ["c3", "c4_k8"]
    for lp in (20, 22, 24, 26, 27):
        for tag in ("fp32", "bf16", "fp32_het", "bf16_het"):
            assert "c5_p%d_%s" % (lp, tag) in default
    assert len(default) == 22
    full = [w.name for w in bench.sweep_cases("full")]
    assert set(default) <= set(full) and "c1" in full and "c4_k16" in full and "c5_p16_fp32" in full
    assert "c5_p25_bf16_m16_sr" in full and len(full) == len(set(full))
    from paper_2111_08274_b200 import workloads
    for name in default:                                   # every default point can be named on the command line
        assert workloads.by_name(name).name == name


def test_kernel_entries_and_traffic(bench):
    e = bench.gbs_entry(1_430_267_136, 0.385, 6464.3, "frac_of_measured_hbm")
    assert abs(e["achieved_gbs"] - 3715.0) < 1.0 and abs(e["frac_of_measured_hbm"] - 0.5747) < 1e-3
    assert abs(e["frac_of_8TBs"] - e["achieved_gbs"] / 8000.0) < 1e-12
    t = bench.traffic_entry("aggregate", 4 * 11_173_962)
    assert t["traffic"] == t["traffic_read"] + t["traffic_write_lower_bound"]
    assert abs(t["traffic_read"] - 4.0 * 4 * 11_173_962) < 1.0 and "lower bound" in t["traffic_is"]
    busiest = max(bench.PIPE_CYCLES_PER_ELEM_STEP, key=bench.PIPE_CYCLES_PER_ELEM_STEP.get)
    peak = bench.SM_COUNT * bench.SUBPARTITIONS_PER_SM * 1965e6 / bench.PIPE_CYCLES_PER_ELEM_STEP[busiest] / 1e9
    assert busiest == "fmaheavy" and 2060 < peak < 2075   # G element-steps/s at the maximum SM clock


def test_table_printer_reads_a_saved_line(bench, tmp_path, capsys):
    k = bench.gbs_entry(1e9, 0.2, 6464.3, "frac_of_measured_hbm")
    k["gelem_steps_per_s"] = 400.0
    point = {"workload": "c5_p24_fp32", "N": 16, "P": 1 << 24, "k": 4, "storage": "fp32",
             "mean_steps_per_device": 1.0, "rounds_per_s": 1500.0, "separate_calls_rounds_per_s": 1100.0,
             "rounds_per_launch": 8.0, "rounds_per_s_one_round_per_launch": 1400.0,
             "kernels": {"round": k, "local_step": k, "aggregate": k, "stats": k}}
    line = {"sweep": {"peak_gbs": 6464.3, "peak_kind": "measured", "points": [point]}}
    path = tmp_path / "line.json"
    path.write_text(json.dumps(line) + "\n")
    bench.print_tables(str(path))
    out = capsys.readouterr().out
    assert "| c5_p24_fp32 | 16 | 16777216 | 4 | fp32 | 1.00 |" in out and "5000 (77 / 62)" in out
    assert "| 1400 | 1500 (8) |" in out
