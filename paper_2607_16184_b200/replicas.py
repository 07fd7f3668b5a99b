"""Multi-GPU launch plumbing.  The layer call does not shard (one GPU, no collectives), so N GPUs
run N independent replicas; the only cross-rank traffic is the timing barrier and a max-reduce of
the per-rank elapsed time."""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when not launched by it."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier(device: torch.device):
    if dist.is_initialized():
        t = torch.zeros(1, device=device)
        dist.all_reduce(t)
        if device.type == "cuda":
            torch.cuda.synchronize(device)


def aggregate(elapsed_ms: float, units: float, device: torch.device) -> Tuple[float, float]:
    """(max elapsed ms over ranks, units summed over ranks): whole-job throughput = units / time."""
    if not dist.is_initialized():
        return elapsed_ms, units
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()
