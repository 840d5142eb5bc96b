"""The benchmark's own line on a GPU, on the smallest paper-shaped workload (20 GB) and few
steps: the keys of the contract, launches counted, the roofline arithmetic reproducible from the
line's own numbers."""

import json
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_contract_on_the_125M_workload():
    if torch.cuda.mem_get_info()[0] < 30e9:
        pytest.skip("needs 30 GB of free device memory")
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "config 2", "--steps", "4",
                          "--warmup", "3", "--no-configs", "--no-cpu-baseline", "--e2e-cols", str(1 << 22)],
                         capture_output=True, text=True, timeout=900, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 4 and d["warmup"] == 3 and d["scaling"] == "weak"
    assert "config 2" in d["config"]["workload"] and d["data"] == "synthetic" and d["dtype"] == "f32"
    W, P = d["config"]["W"], d["config"]["P"]
    # whole-job throughput = units / time
    assert d["value"] == pytest.approx(W * P / (d["ms_per_step"] * 1e-3), rel=1e-6)
    # two draws, the fused kernel and the routing copy per step
    assert d["gpu_launches"] == 4 * d["steps"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["launches_timed"] == d["steps"]
    assert r["bytes_per_launch"] == 20 * W * P
    assert r["achieved"] == pytest.approx(r["bytes_per_launch"] / (r["ms_per_launch"] * 1e-3) / 1e9, rel=1e-6)
    assert r["frac"] == pytest.approx(r["achieved"] / r["peak"], rel=1e-9)
    assert 0.5 < r["frac_of_same_run_copy"] < 1.1
    assert r["traffic"] is None or 0.9 < r["traffic"] / r["bytes_per_launch"] < 1.1
    assert r["ms_per_launch"] < d["ms_per_step"]
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < d["value"]                       # host copies are inside its timed region
    c = d["clocks"]
    assert c["sm_max_mhz"] is None or c["sm_mhz"] <= c["sm_max_mhz"]
    assert not {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"} & set(c["reasons"])
