"""Multi-GPU plumbing: the outer step of this library runs on one GPU, so N
GPUs run N independent replicas of the workload (one process per GPU, no
data-path collective).  Only the timing is combined across ranks: the job's
time is the slowest rank's, its work the sum over ranks."""

from __future__ import annotations

import os

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
