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
