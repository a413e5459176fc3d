"""Replica bookkeeping for runs on more than one GPU.

Every (sequence, KV head) of the path is independent, so N GPUs run N independent replicas of the same
workload; the only exchange is a barrier around the timed region and the maximum of the per-rank
device times.  No tensor of the path ever crosses ranks.
"""
from __future__ import annotations

import os
from typing import Optional

import torch


def env_rank_world() -> tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment; (0, 1, 0) for a plain run."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, world: int):
    """Joins the process group when there is more than one rank (rendezvous from MASTER_ADDR / MASTER_PORT)."""
    if world <= 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        dist.init_process_group(backend)
    return dist


def barrier(dist, device: Optional[str] = None) -> None:
    """Device sync, process barrier, device sync: brackets a timed region on every rank."""
    if device is not None and str(device).startswith("cuda"):
        torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
        if device is not None and str(device).startswith("cuda"):
            torch.cuda.synchronize()


def max_over_ranks(dist, ms: float, device: str = "cpu") -> float:
    """The slowest rank's time: the job is as slow as its slowest replica."""
    if dist is None:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(world: int, units_per_rank: float, ms: float) -> float:
    """Units per second of the whole job: every rank processed ``units_per_rank`` within ``ms``."""
    return world * units_per_rank / (ms * 1e-3)
