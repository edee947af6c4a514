"""Multi-GPU plumbing of the benchmark: independent replicas, one per rank.

The path has no exchange step (one sequence, one GPU), so N GPUs run N independent sequences: each rank owns
its own inputs (seeds offset by the rank) and the only collective traffic is the barrier and the max-over-ranks of
the measured device time.  torch.distributed is used for exactly that; nothing here touches the data path.
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_ranks() -> Tuple[int, int, int]:
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None) -> Tuple[int, int, int]:
    """Joins the process group when launched with WORLD_SIZE > 1 (rendezvous through MASTER_ADDR/MASTER_PORT)."""
    rank, world, local = env_ranks()
    if world > 1 and not dist.is_initialized():
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, rank=rank, world_size=world, **kw)
    return rank, world, local


def replica_seed(base_seed: int, rank: int) -> int:
    """Seed of a replica's inputs: replicas see different data (independent sequences)."""
    return base_seed + 1000 * rank


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: what a job of N replicas takes."""
    if not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()
