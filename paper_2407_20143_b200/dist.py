"""Process-group plumbing for the benchmark: one process per GPU, no data-path collective.

The resharding path has no exchange step on one node (every rank reshards its own replica
of the state), so the only collectives are the barrier around the timed region and the
max over ranks of the measured time.
"""
from __future__ import annotations

import os
from typing import Optional

import torch
import torch.distributed as dist


def world() -> tuple:
    """(rank, local_rank, world_size) from the launcher's environment."""
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def init(backend: Optional[str] = None) -> bool:
    """Join the process group if the launcher started more than one rank."""
    rank, _, ws = world()
    if ws <= 1:
        return False
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29531")
        backend = backend or ("nccl" if torch.cuda.is_available() else "gloo")
        dist.init_process_group(backend=backend, rank=rank, world_size=ws)
    return True


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(x: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def aggregate_throughput(units_local: float, ms_local: float, device="cpu") -> dict:
    """Whole-job throughput: units of all ranks over the slowest rank's time."""
    ms = max_over_ranks(ms_local, device)
    units = sum_over_ranks(units_local, device)
    return {"ms": ms, "units": units, "per_second": units / (ms * 1e-3) if ms > 0 else 0.0}


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
