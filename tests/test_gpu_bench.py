"""bench.py end to end on the smallest workload: one JSON line with every key of the contract."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*extra):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "cfg1_tiny_f32",
                          "--steps", "5", "--warmup", "3", *extra],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    return json.loads(lines[0])


def test_bench_line_has_the_whole_contract():
    d = _run()
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
              "scaling", "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches",
              "roofline", "cpu_baseline", "device_status", "roofline_hbm_steps", "other_workloads",
              "host_enqueue_ms_per_step"):
        assert k in d, k
    assert d["other_workloads"] is None                # only the default workload's line carries them
    steps = {r["step"]: r for r in d["roofline_hbm_steps"]}
    assert set(steps) == {"route", "aux_stats", "dispatch", "combine", "combine_bwd", "dispatch_bwd", "route_bwd"}
    assert all(r["ms"] > 0 and r["bytes"] > 0 and r["unit"] == "GB/s" for r in steps.values())
    assert d["config"]["count_ratio"] is None or d["config"]["count_ratio"] >= 1.0
    assert d["unit"] == "tokens/s" and d["n_gpus"] == 1 and d["steps"] == 5 and d["warmup"] == 3
    assert d["value"] > 0 and abs(d["value"] - 256 / (d["ms_per_step"] * 1e-3)) <= 1e-6 * d["value"]
    assert d["config"]["workload"] == "cfg1_tiny_f32" and d["dtype"] == "f32" and d["data"] == "synthetic"
    assert d["gpu_launches"] > 0 and d["gpu_launches"] % 5 == 0 and d["device_status"] == 0
    assert d["e2e"]["value"] > 0 and d["e2e"]["h2d_bytes_per_step"] == 2 * 256 * 128 * 4
    assert d["e2e"]["d2h_bytes_per_step"] > d["e2e"]["h2d_bytes_per_step"]
    assert set(("bound", "achieved", "peak", "unit", "frac", "traffic")) <= set(d["roofline"])
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] > 0 and "256 tokens" in d["cpu_baseline"]["sample"]
    assert set(("sm_mhz", "sm_max_mhz", "reasons")) <= set(d["clocks"])


def test_bench_graph_replay_line():
    d = _run("--graph", "--no-cpu-baseline", "--no-e2e")
    assert d["config"]["launch"] == "CUDA graph replay"
    assert d["value"] > 0 and d["gpu_launches"] > 0 and d["device_status"] == 0
