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
                "roofline", "e2e", "gpu_launches", "clocks", "reps", "timed_seconds", "ms_per_step_reps"):
        assert key in line, key
    # the value is the median of at least five repetitions that kept the device busy for seconds
    assert line["reps"] >= 5 and line["timed_seconds"] >= 1.5
    spread = line["ms_per_step_reps"]
    assert spread["min"] <= spread["median"] <= spread["max"]
    assert abs(spread["median"] - line["ms_per_step"]) < 1e-3 * line["ms_per_step"] + 1e-4
    assert len(spread["in_run_order"]) >= 5
    assert line["n_gpus"] == 1 and line["steps"] == 3 and line["scaling"] == "weak"
    assert line["dtype"] == "f32" and line["data"] == "synthetic" and line["vs_baseline"] is None
    r = line["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 1000
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3
    assert 0.5 < r["frac"] < 1.3                       # far outside: the timed kernel did not do the work
    assert r["algorithmic_bytes_per_launch"] == 32 * 4 * 11_689_512
    assert r["launches_bracketed"] >= 10 and r["ms_per_launch"] > 0
    # one period is four launches: the exchange riding on the first step, two plain steps and a
    # distance round that stores its tile sums (the riding exchange of the next period assembles
    # the distances and runs the weighting rule at its head)
    assert line["gpu_launches"] == 4 * line["steps"] * line["reps"]
    e = line["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < line["value"]                  # copies from the host are inside its timing
    c = line["clocks"]
    assert c["sm_max_mhz"] is None or c["sm_max_mhz"] > 1000
    if c["sm_mhz"] is not None:                        # nvidia-smi is there: samples inside the region
        assert c["window"] == "timed region" and c["samples"] >= 10
        assert abs(c["ms_per_step_x_mhz"] - line["ms_per_step"] * c["sm_mhz"]) < 1.0
