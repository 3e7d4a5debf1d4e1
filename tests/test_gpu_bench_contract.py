"""The benchmark's output line: one JSON object with the keys its readers rely on, produced by a run that really
launched the library's kernels.  A small batch keeps the run to a few seconds."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*flags):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--batch", "2", "--steps", "2", "--warmup", "3",
                          "--no-cpu", *flags], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    return json.loads(lines[0])


@pytest.mark.parametrize("flags", [(), ("--no-graph", "--no-overlap")], ids=["graph", "plain"])
def test_bench_line(flags):
    d = _run(*flags)
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "e2e", "gpu_launches", "clocks", "layers"):
        assert key in d, key
    assert d["unit"] == "images/s" and d["n_gpus"] == 1 and d["steps"] == 2 and d["higher_is_better"] is True
    assert d["scaling"] == "weak" and d["data"] == "synthetic" and d["vs_baseline"] is None
    assert "workload" in d["config"] and d["config"]["batch_per_gpu"] == 2
    assert d["value"] > 0 and abs(d["value"] - 2 * 1000.0 / d["ms_per_step"]) <= 1e-3 * d["value"] + 0.02
    r = d["roofline"]
    for key in ("bound", "achieved", "peak", "unit", "frac", "traffic"):
        assert key in r, key
    assert r["bound"] == "alu" and 0 < r["frac"] < 1.2 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < d["value"]                      # copies inside the timed region can only cost time
    assert d["gpu_launches"] >= 2 * 13                  # at least one kernel per layer and step
    assert len(d["layers"]) == 13 and all(l["conv_us"] > 0 for l in d["layers"])
