"""The GPU arm of the benchmark prints one JSON line with the keys its readers rely on (short run)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_gpu_arm_prints_one_line_with_rooflines_end_to_end_and_launch_count():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "1", "--steps", "4", "--warmup", "3",
                          "--replays", "3", "--no-cpu-baseline", "--no-other-configs", "--no-rollout-extras"],
                         cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
              "vs_baseline", "dtype", "data", "config", "clocks", "gpu_launches", "roofline", "roofline_env", "e2e",
              "replays", "sustained"):
        assert k in d, k
    assert d["steps"] == 4 and d["warmup"] == 3 and d["n_gpus"] == 1 and d["scaling"] == "weak"
    assert d["unit"] == "env-steps/s" and d["value"] > 1e6 and d["dtype"] == "bf16"
    assert d["config"]["workload"] == "cfg4_65536_smpl24"
    assert d["gpu_launches"] == 4 * 5            # three hidden GEMMs, the Gaussian head and the env step per step
    r = d["roofline"]
    assert r["bound"] == "tensor" and r["unit"] == "TFLOP/s" and 0.05 < r["frac"] < 1.2
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and r["traffic"] > 0
    e = d["roofline_env"]
    assert e["bound"] == "hbm" and e["unit"] == "GB/s" and 0.02 < e["frac"] < 1.2 and e["traffic"] > 0
    assert d["e2e"]["value"] > 0 and d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > 0
    assert d["e2e"]["value"] < d["value"]        # host buffers cross PCIe every step
    assert d["clocks"]["sm_max_mhz"] >= d["clocks"]["sm_mhz"] > 0
