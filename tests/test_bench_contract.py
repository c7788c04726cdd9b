"""The one JSON line `bench.py` prints: the keys its readers rely on, for the reference arm (the oracle on the host
cores, runs anywhere) and for the library's own arm (needs a GPU)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

BASE_KEYS = ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config", "e2e", "gpu_launches", "cpu_baseline")


def _run(args, timeout):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, cwd=ROOT, capture_output=True,
                         text=True, timeout=timeout)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1, lines          # exactly one line on stdout
    return json.loads(lines[0])


def test_reference_arm_line():
    d = _run(["--impl", "reference", "--steps", "1", "--warmup", "1"], 300)
    for k in BASE_KEYS:
        assert k in d, k
    assert d["impl"] == "reference" and d["metric"] == "verified_draft_positions_per_sec" and d["unit"] == "positions/s"
    assert d["value"] > 0 and d["higher_is_better"] is True and d["vs_baseline"] is None and d["gpu_launches"] == 0
    assert d["config"]["workload"].startswith("cfg3_") and "model" not in d["config"]
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == d["value"] and cb["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


@pytest.mark.gpu
def test_own_arm_line():
    d = _run(["--steps", "20", "--warmup", "3"], 900)
    for k in BASE_KEYS + ("roofline", "clocks", "largest_config"):
        assert k in d, k
    assert "impl" not in d or d["impl"] != "reference"
    assert d["n_gpus"] == 1 and d["steps"] == 20 and d["warmup"] >= 3 and d["dtype"] == "f32" and d["data"] == "synthetic"
    assert d["config"]["workload"].startswith("cfg3_") and "exceed L2" in d["config"]["l2"]
    assert d["gpu_launches"] > 0 and d["value"] > 1e5
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert 0.3 < r["frac"] < 1.3                       # far above 1 would mean the timed kernel is not doing the work
    assert r["traffic"] is None or r["traffic"] >= r["algorithmic_bytes_per_launch"]
    e = d["e2e"]
    assert e["h2d_bytes_per_step"] > 2e9 and e["d2h_bytes_per_step"] > 0 and 0 < e["value"] < d["value"]
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["value"] > 0 and cb["cores"] >= 1
    assert set(("sm_mhz", "sm_max_mhz", "reasons")) <= set(d["clocks"])
    big = d["largest_config"]
    assert big["workload"].startswith("cfg4_") and big["all_outputs"]["frac_of_nominal_8TBs"] > 0.5
    assert big["algorithm1_only"]["same_accept_len_as_all_outputs"] is True
