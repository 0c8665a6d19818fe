"""bench.py end to end on the smallest workload (needs a B200): every leg runs -- timed region, kernel
pass, early-exit comparison, end-to-end from host buffers, CPU baseline -- and the line has the agreed keys."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
        "vs_baseline", "dtype", "data", "config", "roofline", "e2e", "cpu_baseline", "clocks", "gpu_launches"}


def _bench(*flags):
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "tiny_ucb", "--steps", "6", "--warmup", "3",
           "--cpu-seconds", "0.5", "--no-others", *flags]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    return json.loads(res.stdout.strip().splitlines()[-1])


@pytest.mark.parametrize("flags", [(), ("--walk",), ("--drafted", "--bandit-step"), ("--no-graph",)])
def test_bench_line_on_the_tiny_workload(flags):
    d = _bench(*flags)
    assert KEYS <= set(d), KEYS - set(d)
    assert d["value"] > 0 and d["ms_per_step"] > 0 and d["gpu_launches"] >= 3 * d["steps"]
    assert d["config"]["workload"] == "tiny_ucb" and d["n_gpus"] == 1
    r = d["roofline"]
    assert r["bound"] == "hbm" and 0 < r["frac"] < 1.2 and r["achieved"] > 0 and r["peak"] > 0
    assert d["e2e"]["value"] > 0 and d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] > 0


def test_bench_line_on_the_tiny_tree_workload():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "tiny_tree", "--steps", "6", "--warmup", "3",
           "--cpu-seconds", "0.5", "--no-others"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    d = json.loads(res.stdout.strip().splitlines()[-1])
    assert KEYS <= set(d), KEYS - set(d)
    assert d["value"] > 0 and d["config"]["workload"] == "tiny_tree" and 1.0 <= d["mean_accepted_len"] <= 4.0
    assert d["roofline"]["bound"] == "hbm" and d["roofline"]["achieved"] > 0
    assert d["e2e"]["value"] > 0 and d["cpu_baseline"]["value"] > 0
