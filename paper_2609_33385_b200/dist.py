"""Multi-process plumbing for replica runs: each rank drives an independent context on its own
GPU (the path has per-layer mutable cache state and does not shard; there is no collective on
the data path).  Only the timing aggregation crosses ranks."""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def aggregate(units_local: float, elapsed_ms_local: float, device="cpu") -> Tuple[float, float]:
    """Whole-job units (sum over ranks) and elapsed time (max over ranks)."""
    if not dist.is_initialized():
        return float(units_local), float(elapsed_ms_local)
    u = torch.tensor([float(units_local)], dtype=torch.float64, device=device)
    t = torch.tensor([float(elapsed_ms_local)], dtype=torch.float64, device=device)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(u.item()), float(t.item())


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
