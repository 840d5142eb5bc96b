"""Multi-GPU plumbing: the outer step of this library runs on one GPU, so N
GPUs run N independent replicas of the workload (one process per GPU, no
data-path collective).  Only the timing is combined across ranks: the job's
time is the slowest rank's, its work the sum over ranks."""

from __future__ import annotations

import os
import socket
import subprocess
import sys
import time

import torch
import torch.distributed as dist


def env_rank() -> tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, device: torch.device | None = None) -> bool:
    """Join the process group if launched with more than one rank."""
    _, _, world = env_rank()
    if world <= 1:
        return False
    if not dist.is_initialized():
        kw = {}
        if device is not None and device.type == "cuda":
            kw["device_id"] = device
        dist.init_process_group(backend=backend, **kw)
    return True


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def job_time_and_units(local_ms: float, local_units: float, device="cpu") -> tuple[float, float]:
    """Max of the ranks' times and sum of the ranks' units of work."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(local_ms), float(local_units)
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def throughput(units: float, ms: float) -> float:
    return units / (ms * 1e-3)


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch(n: int, argv: list[str], stdout=None, timeout: float | None = None) -> int:
    """Start ``argv`` as n rank processes on this node (rank r gets RANK = LOCAL_RANK = r,
    WORLD_SIZE = n and a rendezvous on 127.0.0.1) and wait for them.  ``stdout`` goes to
    rank 0 only (the rank that reports); the other ranks' standard output is discarded.
    Returns 0 if every rank exited 0; otherwise stops the remaining ranks and returns the
    first non-zero exit code (124 if ``timeout`` seconds ran out)."""
    port = free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen(argv, env=env, stdout=stdout if r == 0 else subprocess.DEVNULL))
    deadline = None if timeout is None else time.monotonic() + timeout
    rc = 0
    pending = list(procs)
    while pending and rc == 0:
        for p in list(pending):
            code = p.poll()
            if code is not None:
                pending.remove(p)
                if code != 0:
                    rc = code
        if deadline is not None and time.monotonic() > deadline:
            rc = 124
        if pending and rc == 0:
            time.sleep(0.05)
    for p in pending:            # a rank failed or time ran out: stop exactly the processes started here
        p.terminate()
    for p in pending:
        try:
            p.wait(timeout=10)
        except subprocess.TimeoutExpired:
            p.kill()
    return rc


def _selftest(backend: str) -> int:
    """Rank-side half of the launcher check: join, combine a made-up timing, rank 0 reports."""
    import json
    rank, _, world = env_rank()
    init(backend)
    barrier()
    ms, units = job_time_and_units(10.0 + rank, 100.0)
    barrier()
    if rank == 0:
        print(json.dumps({"n_gpus": world, "ranks_joined": dist.get_world_size() if dist.is_initialized() else 1,
                          "ms": ms, "units": units}), flush=True)
    else:
        print(f"rank {rank} has nothing to report", flush=True)      # must not reach the job's output
    if dist.is_initialized():
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    if len(sys.argv) >= 2 and sys.argv[1] == "--selftest":
        raise SystemExit(_selftest(sys.argv[2] if len(sys.argv) > 2 else "gloo"))
    raise SystemExit("usage: python -m paper_2506_10911_b200.replicas --selftest [backend]")
