"""bench.py on the GPU: the JSON line carries every key the benchmark contract names, the per-regime split adds up,
both roofline denominators are there, and a run whose levels are forced reports that regime only."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench(*flags):
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *flags], capture_output=True, text=True,
                         timeout=900)
    assert res.returncode == 0, res.stderr[-3000:]
    lines = [l for l in res.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1, "rank 0 prints exactly one JSON line"
    return json.loads(lines[0])


def test_bench_line_config1_with_regimes_and_both_denominators():
    d = _bench("--config", "1", "--steps", "12", "--warmup", "3", "--e2e-steps", "2", "--no-cpu-baseline")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline",
                "step_ms_by_regime", "kernels"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 12 and d["warmup"] == 3 and d["value"] > 0 and d["gpu_launches"] > 0
    assert d["dtype"] == "f32" and d["data"] == "synthetic" and d["vs_baseline"] is None and d["scaling"] == "weak"
    assert "workload" in d["config"] and "model" not in d["config"]
    # config 1 checks every 5 steps: steps 3..14 of the run are low until the check after step 9, then high
    reg = d["step_ms_by_regime"]
    assert sum(v["steps"] for v in reg.values()) == 12 and set(reg) <= {"low", "high", "mixed"}
    assert reg["low"]["steps"] == 7 and reg["high"]["steps"] == 5
    for v in reg.values():
        assert v["min_ms"] <= v["median_ms"] <= v["max_ms"]
        assert set(v["frac_of_12B"]) == {"of_measured_copy_peak", "of_nominal_8TBs"}
        assert v["frac_of_12B"]["of_nominal_8TBs"] <= v["frac_of_12B"]["of_measured_copy_peak"]
    r = d["roofline"]
    for key in ("bound", "achieved", "peak", "unit", "frac", "traffic", "peak_nominal", "frac_of_nominal",
                "step_frac_of_12B", "step_frac_of_12B_nominal"):
        assert key in r, key
    assert r["bound"] == "hbm" and r["peak_nominal"] == 8000.0 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3
    e = d["e2e"]
    assert e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0 and 0 < e["value"] < d["value"]
    assert "regime_of_value" in d["config"] and "7 of 12" in d["config"]["regime_of_value"]


@pytest.mark.parametrize("level", ["low", "high"])
def test_bench_forced_level_reports_one_regime(level):
    d = _bench("--config", "1", "--steps", "11", "--warmup", "3", "--e2e-steps", "1", "--no-cpu-baseline",
               "--force-level", level)
    assert list(d["step_ms_by_regime"]) == [level] and d["step_ms_by_regime"][level]["steps"] == 11
    assert level in d["config"]["levels"]
