"""Multi-GPU plumbing for the benchmark: the path does not shard (one video stream and its store
live on one GPU), so N GPUs run N independent replicas and only the timing is combined."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def init_from_env(backend: str | None = None) -> tuple[int, int, int]:
    """(rank, world_size, local_rank); initialises torch.distributed when WORLD_SIZE > 1."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend or ("nccl" if torch.cuda.is_available() else "gloo"),
                                rank=rank, world_size=world)
    return rank, world, local


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def combine(local_ms: float, local_units: float, device="cpu") -> tuple[float, float]:
    """(max over ranks of the time, sum over ranks of the units processed)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(local_ms), float(local_units)
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([float(local_units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def throughput(local_ms: float, local_units: float, device="cpu") -> float:
    """Whole-job units per second: all ranks' units divided by the slowest rank's time."""
    ms, units = combine(local_ms, local_units, device)
    return units / (ms * 1e-3) if ms > 0 else 0.0
