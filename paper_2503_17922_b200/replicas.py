"""Multi-GPU plumbing of the benchmark: independent replicas, one process per GPU.

The path has no exchange step (units are independent), so ranks share nothing but the clock:
a barrier on both sides of the timed region and the maximum of the per-rank device times.
`backend` is "nccl" on GPUs; the CPU tests run the same code over "gloo".
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys
from typing import Callable, List, Tuple

import torch
import torch.distributed as dist


def rank_env() -> Tuple[int, int, int]:
    """(rank, world size, local rank) from the launcher's environment; (0, 1, 0) without one."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def launcher_present() -> bool:
    """True when a launcher (torch.distributed.run) has set this process's rank environment."""
    return "RANK" in os.environ and "WORLD_SIZE" in os.environ


def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def launcher_command(n: int, script: str, argv: List[str], port: int) -> List[str]:
    """The command that runs `script argv` as n ranks of one node, one process per GPU."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), script] + list(argv)


def relaunch_under_launcher(n: int, script: str, argv: List[str]) -> int:
    """Runs `script argv` again as n ranks (used when a multi-replica run was asked for as a plain
    command, without a launcher); returns the launcher's exit code.  The ranks print the result."""
    env = dict(os.environ)
    env.setdefault("OMP_NUM_THREADS", "4")
    return subprocess.call(launcher_command(n, script, argv, free_port()), env=env)


def timed_region(step: Callable[[int], None], steps: int, warmup: int, start: Callable[[], None],
                 stop_ms: Callable[[], float], device="cpu", sync_cuda: bool = True) -> float:
    """`warmup` untimed steps, a barrier, `steps` steps between start() and stop_ms() (which returns
    this rank's milliseconds), a barrier, and the maximum over the ranks: milliseconds the whole job
    took for the timed steps."""
    for i in range(warmup):
        step(i)
    barrier(sync_cuda)
    start()
    for i in range(steps):
        step(i)
    ms = stop_ms()
    barrier(sync_cuda)
    return max_over_ranks(ms, device)


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
