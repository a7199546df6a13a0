"""Multi-GPU plumbing of the benchmark: independent replicas, one process per GPU.

The path has no exchange step (units are independent), so ranks share nothing but the clock:
a barrier on both sides of the timed region and the maximum of the per-rank device times.
`backend` is "nccl" on GPUs; the CPU tests run the same code over "gloo".
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def rank_env() -> Tuple[int, int, int]:
    """(rank, world size, local rank) from the launcher's environment; (0, 1, 0) without one."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None) -> None:
    """Joins the process group when there is more than one rank (rendezvous from MASTER_ADDR/PORT)."""
    _, world, _ = rank_env()
    if world > 1 and not dist.is_initialized():
        if backend == "nccl":
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)


def barrier(sync_cuda: bool = True) -> None:
    if dist.is_initialized():
        dist.barrier()
    if sync_cuda and torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: what the whole job took."""
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_step: int, world: int, ms_per_step: float) -> float:
    """Aggregate units per second of `world` replicas that each process `units_per_rank_step` per step."""
    return units_per_rank_step * world / (ms_per_step * 1e-3)


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
