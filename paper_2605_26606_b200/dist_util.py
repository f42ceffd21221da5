"""Rank plumbing for multi-GPU runs: prompt groups are independent, so every rank generates its own
sampling batch with replicated weights and nothing is exchanged on the data path.  Only the benchmark's
bookkeeping crosses ranks: a barrier around the timed region and a reduction of (max time, total units)."""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def init(backend: str) -> Tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def aggregate(elapsed_ms: float, units: float, device="cpu") -> Tuple[float, float]:
    """(max over ranks of elapsed_ms, sum over ranks of units)."""
    if not dist.is_initialized():
        return float(elapsed_ms), float(units)
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def rank_data_seed(base_seed: int, rank: int) -> int:
    """Every rank draws a different sampling batch (weak scaling: per-GPU work is fixed)."""
    return base_seed + 1000 * rank
