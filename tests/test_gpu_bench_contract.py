"""bench.py prints one JSON line with the keys the measurement contract asks for."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_has_the_contract_keys():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "4", "--warmup", "3", "--e2e-steps", "1",
                          "--no-cpu-baseline", "--no-legs", "--sustain-s", "0.3"], capture_output=True, text=True, timeout=600,
                         cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "gpu_launches", "clocks", "roofline", "e2e"):
        assert key in d, key
    assert d["steps"] == 4 and d["warmup"] == 3 and d["n_gpus"] == 1 and d["vs_baseline"] is None
    assert d["gpu_launches"] == 4 * 4 and "workload" in d["config"] and "model" not in d["config"]
    assert d["config"]["workload"].startswith("7B-shaped") and d["config"]["plan_matches_thresholds"] is True
    assert d["sustained"]["seconds"] >= 0.3 and d["sustained"]["clocks"]["samples"] >= 3
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert 0.3 < r["frac"] < 1.2 and r["traffic"] is not None
    e = d["e2e"]
    assert e["h2d_bytes_per_step"] > 2e10 and e["d2h_bytes_per_step"] > 0 and 0 < e["value"] < d["value"]
    assert d["value"] == pytest.approx(d["config"]["bytes_per_step"] / d["ms_per_step"] / 1e6, rel=1e-6)
