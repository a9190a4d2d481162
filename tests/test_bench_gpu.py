"""bench.py as the driver runs it: the JSON line's contract on a short run, and the mode that cuts
one search into rank windows (world size 1 here: the cut, the search through the library and the
comparison with the stored expected values)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args):
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], cwd=ROOT, capture_output=True, text=True, timeout=1200)
    assert r.returncode == 0, r.stderr[-2000:]
    return json.loads(r.stdout.strip().splitlines()[-1])


def test_bench_line_of_one_workload():
    d = _run("--workload", "config2", "--steps", "3", "--warmup", "3", "--no-cpu-baseline")
    assert d["metric"] == "candidate_point_evals_per_s" and d["n_gpus"] == 1 and d["steps"] == 3 and d["higher_is_better"]
    assert d["config"]["workload"].startswith("config2") and d["value"] > 0 and d["ms_per_step"] > 0
    assert d["gpu_launches"] >= 3 * 4
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0 and e["value"] < d["value"]
    r = d["roofline"]
    assert r["bound"] == "alu" and 0 < r["frac"] < 1.5 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert r["division_cost"]["int64_general_form"] > r["division_cost"]["int32_by_constant_reciprocal_form"] > 1
    assert d["clocks"]["sm_mhz"] is None or d["clocks"]["sm_mhz"] > 0
    assert d["config"]["filter_tests"] + d["config"]["candidates_skipped"] <= d["config"]["candidates_per_step"]


def test_bench_sharded_search_equals_the_stored_expected_values():
    d = _run("--shard", "--steps", "1", "--warmup", "3")
    assert d["scaling"] == "strong" and d["config"]["merged_equals_expected"] is True and d["value"] > 0
