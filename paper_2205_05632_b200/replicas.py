"""Host-side plumbing for running independent replicas of the optimizer, one process per GPU.

The COMP-AMS step keeps all n workers on one GPU and has no exchange between GPUs, so several
GPUs only ever run independent replicas. What the ranks share is the clock: a barrier before and
after the timed region and the maximum over ranks of the device time.
"""
from __future__ import annotations

import os
from typing import Optional, Tuple

import torch


def rank_world_local() -> Tuple[int, int, int]:
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device: Optional[torch.device] = None):
    """Joins the process group when WORLD_SIZE > 1 (rendezvous from MASTER_ADDR / MASTER_PORT);
    returns torch.distributed or None for a single process."""
    _, world, _ = rank_world_local()
    if world <= 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        kwargs = {}
        if backend == "nccl" and device is not None:
            kwargs["device_id"] = device
        dist.init_process_group(backend, **kwargs)
    return dist


def barrier(dist) -> None:
    if dist is not None:
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(value: float, dist, device="cpu") -> float:
    """The slowest rank's figure: what a job that waits for all replicas observes."""
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def aggregate_throughput(units_per_rank_step: float, world: int, ms_per_step_max: float) -> float:
    """Whole-job throughput of `world` replicas each processing units_per_rank_step per step."""
    return world * units_per_rank_step / (ms_per_step_max * 1e-3)
