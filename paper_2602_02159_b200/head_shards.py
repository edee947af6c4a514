"""A layer whose heads are spread over several GPUs (one process per GPU).

Every stage of the path works head by head (KV group by KV group) except one: the attention-sink scores S_j of Eq. 6
are a mean over ALL heads.  With the KV heads of a layer dealt out in equal contiguous runs, a rank computes S over
its own heads, the ranks average their S (one all-reduce of L floats per denoising step: the only exchange of the
step), and every rank takes the same Top-N_sink from the average.  Block scores, block lists, sink keep flags and
attention outputs stay per KV group and never leave the rank that owns the group.  torch.distributed carries the
all-reduce (NCCL on GPUs; gloo in the CPU test of this module); nothing else of the data path goes through it.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch
import torch.distributed as dist


def local_heads(n_q_heads: int, n_kv_heads: int, rank: int, world: int) -> Tuple[slice, slice]:
    """(query heads, KV heads) owned by `rank`: equal contiguous runs of whole KV groups."""
    if n_kv_heads % world != 0 or n_q_heads % n_kv_heads != 0:
        raise ValueError(f"{n_kv_heads} KV heads cannot be dealt out evenly to {world} ranks")
    per_kv = n_kv_heads // world
    hpg = n_q_heads // n_kv_heads
    return slice(rank * per_kv * hpg, (rank + 1) * per_kv * hpg), slice(rank * per_kv, (rank + 1) * per_kv)


def mean_over_ranks(scores: torch.Tensor, group: Optional[dist.ProcessGroup] = None) -> torch.Tensor:
    """In place: scores <- mean over the ranks of `group` of their scores (equal head counts per rank, so the mean of
    the ranks' means over heads is the mean over all heads).  Without a process group: unchanged."""
    if not dist.is_initialized():
        return scores
    world = dist.get_world_size(group)
    if world == 1:
        return scores
    dist.all_reduce(scores, op=dist.ReduceOp.SUM, group=group)
    scores.mul_(1.0 / world)
    return scores
