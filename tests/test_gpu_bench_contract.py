"""bench.py prints one JSON line with the agreed keys, for the library and for the reference arm (the oracle)."""
import json
import os
import subprocess
import sys

import pytest

from conftest import ROOT

pytestmark = pytest.mark.gpu


def _run(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                         cwd=ROOT, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, lines
    return json.loads(lines[0])


def test_library_arm_line():
    d = _run("--workload", "c2", "--steps", "5", "--warmup", "3")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 5 and d["warmup"] == 3 and d["higher_is_better"] is True
    assert d["dtype"] == "int64" and d["data"] == "synthetic" and d["vs_baseline"] is None and d["scaling"] == "weak"
    assert "workload" in d["config"] and "model" not in d["config"] and d["result"]["all_status_ok"] is True
    # result keys live beside the config, so that both arms print the same config
    assert set(d["config"]) == {"workload", "n", "R", "B", "objective", "input_bytes_per_step_per_gpu", "l2", "parallelism"}
    t = d["timing"]
    assert t["samples"] == 5 and t["inner_repeats"] >= 1 and t["timed_region_ms"] >= 90.0
    assert t["ms_per_step_min"] <= t["ms_per_step_median"] <= t["ms_per_step_max"]
    for key in ("examined_bytes", "all_input_bytes"):
        w = d["roofline"]["whole_call"][key]
        assert 0 < w["frac_of_nominal_8000"] < w["frac_of_measured"] < 1.5
    assert d["value"] > 0 and d["gpu_launches"] > 0
    for key in ("bound", "achieved", "peak", "unit", "frac", "traffic"):
        assert key in d["roofline"], key
    assert d["roofline"]["bound"] == "hbm" and abs(d["roofline"]["frac"] - d["roofline"]["achieved"] / d["roofline"]["peak"]) < 1e-9
    for key in ("value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step"):
        assert key in d["e2e"], key
    assert d["e2e"]["h2d_bytes_per_step"] == 16 * 64 * 4096 * 8 and 0 < d["e2e"]["value"] < d["value"]
    cpu = d["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["cores"] >= 1 and cpu["value"] > 0 and cpu["sample"]
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}


def test_reference_arm_line():
    d = _run("--impl", "reference", "--workload", "c2", "--steps", "2", "--warmup", "1")
    assert d["impl"] == "reference" and d["value"] > 0 and d["unit"] == "timestamps/s"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"].startswith("c2")
    lib = _run("--workload", "c2", "--steps", "3", "--warmup", "3", "--no-cpu-baseline", "--no-probe")
    assert lib["config"] == d["config"]
    assert "not extrapolated" in d["timing"]["what"] and d["ms_per_step"] == d["timing"]["ms_per_step_median"]
