"""The benchmark's output contract, as far as it can be checked without a GPU.

`bench.py --impl reference` times the CPU oracle on a bounded sample of the benchmark workload and prints one
JSON line with the same metric, unit and workload as the GPU arm; under a multi-rank launch only rank 0 runs and
prints, the other ranks leave with exit code 0 and no output.  The GPU arm's line is checked by the GPU tests'
box (its keys are listed here so that both arms stay in step).
"""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

COMMON_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
               "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"}


def _run(extra_env=None):
    env = dict(os.environ)
    env.update(extra_env or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "1",
                           "--steps", "1", "--warmup", "0"], cwd=ROOT, env=env, capture_output=True, text=True,
                          timeout=600)


def test_reference_arm_prints_one_line_with_the_contract_keys():
    out = _run()
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert COMMON_KEYS <= set(d), sorted(COMMON_KEYS - set(d))
    assert d["impl"] == "reference"
    assert d["unit"] == "env-steps/s" and d["metric"].startswith("env-steps/s")
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["data"] == "synthetic"
    assert d["value"] > 0 and d["ms_per_step"] > 0
    assert d["config"]["workload"] == "cfg4_65536_smpl24"
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == d["value"] and "2048 envs" in cb["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_other_ranks_of_a_multi_rank_reference_run_leave_quietly():
    out = _run({"RANK": "1", "LOCAL_RANK": "1", "WORLD_SIZE": "2", "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": "29571"})
    assert out.returncode == 0, out.stderr[-2000:]
    assert out.stdout.strip() == ""
