"""The benchmark's own output line on a GPU: every key of its contract, and sane values."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_on_the_small_profiling_case():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "p18k4",
                          "--steps", "3", "--warmup", "3", "--pool", "1", "--no-cpu-baseline"],
                         capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step",
                "higher_is_better", "scaling", "vs_baseline", "dtype", "data", "config",
                "roofline", "e2e", "gpu_launches", "clocks"):
        assert key in line, key
    assert line["n_gpus"] == 1 and line["steps"] == 3 and line["scaling"] == "weak"
    assert line["dtype"] == "f32" and line["data"] == "synthetic" and line["vs_baseline"] is None
    r = line["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 1000
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3
    assert 0.5 < r["frac"] < 1.3                       # far outside: the timed kernel did not do the work
    assert r["algorithmic_bytes_per_launch"] == 32 * 4 * 11_689_512
    # one period: exchange riding on the first step, 2 plain steps, a distance round with its
    # finalize kernel, the weighting rule
    assert line["gpu_launches"] >= 3 * 6
    e = line["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < line["value"]                  # copies from the host are inside its timing
    assert line["clocks"]["sm_max_mhz"] is None or line["clocks"]["sm_max_mhz"] > 1000
