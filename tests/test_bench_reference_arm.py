"""The benchmark's reference arm (the CPU oracle timed on the host cores) needs no GPU, so its
line can be checked here: the keys the benchmark contract asks for, and that under two ranks
only rank 0 works and prints."""

import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BENCH = os.path.join(ROOT, "bench.py")


def run_bench(*extra):
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    res = subprocess.run([sys.executable, BENCH, "--impl", "reference", "--steps", "1", "--warmup", "3",
                          "--ref-seconds", "4", *extra], capture_output=True, text=True, timeout=600, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1, lines                      # exactly one line, from rank 0
    return json.loads(lines[0])


def check_line(line, gpus):
    assert line["impl"] == "reference"
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e", "gpu_launches"):
        assert key in line, key
    assert line["n_gpus"] == gpus and line["steps"] == 1 and line["warmup"] == 3
    assert line["higher_is_better"] is True and line["vs_baseline"] is None and line["gpu_launches"] == 0
    assert line["value"] > 0 and line["ms_per_step"] > 0
    assert "config 4" in line["config"]["workload"]
    cb = line["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == line["value"] and "columns" in cb["sample"]
    e2e = line["e2e"]
    assert e2e["value"] == line["value"] and e2e["unit"] == line["unit"]
    assert e2e["h2d_bytes_per_step"] == 0 and e2e["d2h_bytes_per_step"] == 0


def test_reference_arm_line_has_the_contract_keys():
    check_line(run_bench(), 1)


def test_reference_arm_under_two_ranks_prints_once():
    check_line(run_bench("--gpus", "2"), 2)
