"""bench.py prints ONE JSON line with the keys its contract names; a short run of the real command is parsed here."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(args):
    r = subprocess.run([sys.executable, "bench.py"] + args, cwd=ROOT, capture_output=True, text=True, timeout=1200)
    assert r.returncode == 0, r.stderr[-3000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1, "exactly one line on stdout, got %d" % len(lines)
    return json.loads(lines[0])


def test_the_json_line_of_a_short_run():
    d = run_bench(["--layers", "16", "--steps", "4", "--warmup", "3", "--quick", "--no-cpu-baseline"])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
                "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline"):
        assert key in d, key
    assert d["metric"] == "mxq_linear_hbm_gbs" and d["unit"] == "GB/s" and d["n_gpus"] == 1 and d["steps"] == 4 and d["warmup"] == 3
    assert d["higher_is_better"] is True and d["scaling"] == "weak" and d["vs_baseline"] is None and d["data"] == "synthetic"
    assert "workload" in d["config"] and "model" not in d["config"] and d["config"]["streams"] == 2
    # two calls of eight layer sets per step, four timed steps
    assert d["config"]["calls_per_step"] == 2 and d["gpu_launches"] == 8
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 1000 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert 0.3 < r["frac"] < 1.2, "the persistent kernel far from its usual rate (or timing something else): %r" % r
    assert abs(r["achieved"] - d["value"]) / d["value"] < 0.02
    assert r["traffic"] is not None and 0.98 < r["traffic"] / r["bytes_per_launch"] < 1.1
    e = d["e2e"]
    assert e["unit"] == "GB/s" and 0 < e["value"] <= d["value"] * 1.05 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    c = d["clocks"]
    assert c["sm_max_mhz"] >= c["sm_mhz"] > 0 and isinstance(c["reasons"], list)
    assert d["value"] > 0 and d["ms_per_step"] > 0


def test_the_separate_calls_route_and_a_single_stream():
    d = run_bench(["--layers", "8", "--steps", "3", "--warmup", "3", "--quick", "--no-cpu-baseline", "--route", "separate"])
    assert d["config"]["calls_per_step"] == 56 and d["gpu_launches"] == 3 * 56 and d["roofline"]["kernel"].startswith("linear_fp4_kernel")
    d = run_bench(["--layers", "8", "--steps", "3", "--warmup", "3", "--quick", "--no-cpu-baseline", "--streams", "1", "--layers-per-call", "4"])
    assert d["config"]["calls_per_step"] == 2 and d["config"]["streams"] == 1 and d["gpu_launches"] == 6
