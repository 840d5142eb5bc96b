"""The N > 1 path is N independent replicas; only the timing is combined
(max of the ranks' times, sum of their work).  Exercised with two gloo ranks
on CPU."""

import json
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def worker(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    from paper_2506_10911_b200 import replicas
    assert replicas.env_rank() == (rank, rank, world)
    assert replicas.init("gloo")
    replicas.barrier()
    ms, units = replicas.job_time_and_units(10.0 + 5.0 * rank, 1000.0 * (rank + 1))
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"ms": ms, "units": units, "tp": replicas.throughput(units, ms)}, f)
    replicas.barrier()
    import torch.distributed as dist
    dist.destroy_process_group()


def test_two_ranks_max_time_sum_units(tmp_path):
    mp.spawn(worker, args=(2, free_port(), str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        got = json.load(open(tmp_path / f"r{r}.json"))
        assert got["ms"] == 15.0                 # slowest rank
        assert got["units"] == 3000.0            # all ranks' work
        assert abs(got["tp"] - 3000.0 / 0.015) < 1e-6


def test_single_process_is_passthrough():
    sys.path.insert(0, ROOT)
    from paper_2506_10911_b200 import replicas
    assert replicas.job_time_and_units(3.0, 7.0) == (3.0, 7.0)
    assert replicas.throughput(10.0, 1000.0) == 10.0


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""


def test_launcher_starts_every_rank_and_only_rank0_reports(tmp_path):
    """What `bench.py --gpus N` does when it is not already under a launcher: start N rank
    processes itself.  Two gloo ranks join, one JSON line comes back, with n_gpus 2."""
    sys.path.insert(0, ROOT)
    from paper_2506_10911_b200 import replicas
    out = tmp_path / "out.txt"
    env_before = dict(os.environ)
    with open(out, "w") as f:
        rc = replicas.launch(2, [sys.executable, "-m", "paper_2506_10911_b200.replicas", "--selftest", "gloo"],
                             stdout=f, timeout=120)
    assert rc == 0
    assert dict(os.environ) == env_before                      # the launcher's own environment is untouched
    lines = [ln for ln in out.read_text().splitlines() if ln.strip()]
    assert len(lines) == 1
    got = json.loads(lines[0])
    assert got["n_gpus"] == 2 and got["ranks_joined"] == 2
    assert got["ms"] == 11.0 and got["units"] == 200.0


def test_launcher_reports_a_failing_rank(tmp_path):
    sys.path.insert(0, ROOT)
    from paper_2506_10911_b200 import replicas
    code = "import os, sys, time; r = int(os.environ['RANK']); sys.exit(7) if r == 1 else time.sleep(30)"
    assert replicas.launch(2, [sys.executable, "-c", code], timeout=60) == 7


def test_bench_spawns_ranks_when_not_under_a_launcher(monkeypatch):
    """bench.py --gpus 2 outside a launcher hands its own command line to replicas.launch."""
    sys.path.insert(0, ROOT)
    import importlib
    bench = importlib.import_module("bench")
    from paper_2506_10911_b200 import replicas
    seen = {}
    monkeypatch.setattr(replicas, "launch", lambda n, argv, **kw: seen.update(n=n, argv=argv) or 0)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        monkeypatch.delenv(k, raising=False)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2", "--steps", "3"])
    assert bench.main() == 0
    assert seen["n"] == 2 and seen["argv"][1].endswith("bench.py") and seen["argv"][2:] == ["--gpus", "2", "--steps", "3"]
