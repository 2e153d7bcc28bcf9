"""Multi-process plumbing of the benchmark: the layer has no collective (the ranks are independent
replicas of one workload, weak scaling), so all that crosses ranks is a barrier and the maximum of
the per-rank device times.  Works with NCCL (one GPU per rank) and with gloo (CPU tests)."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(rank, local_rank, world_size) from the launcher's environment (1 process if unset)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, device=None) -> int:
    """Join the process group named by MASTER_ADDR / MASTER_PORT; returns the world size."""
    _, _, world = env_world()
    if world > 1 and not dist.is_initialized():
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, **kw)
    return world


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a per-rank scalar (the job's time is its slowest rank's)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, ms_per_step: float, world: int) -> float:
    """Whole-job rate: every rank processes `units_per_rank` per step, the step takes the slowest
    rank's time."""
    return world * units_per_rank / (ms_per_step * 1e-3)
