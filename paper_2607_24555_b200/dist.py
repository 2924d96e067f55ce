"""Host-side plumbing for running the decode path on several GPUs.

The path shards with no exchange: every (request, KV head) problem owns its pages, summaries,
selection and output heads, so each rank simply runs its own slice of the batch (weak scaling
when every rank gets a full batch).  The only collective is the timing reduction of the benchmark
(max over ranks), done with torch.distributed on whichever backend the job was launched with.
"""
from __future__ import annotations

import os
from typing import List, Tuple

import torch
import torch.distributed as dist


def env_rank_world() -> Tuple[int, int, int]:
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def shard_requests(n_requests: int, rank: int, world: int) -> List[int]:
    """Contiguous, balanced split of request indices; the first (n % world) ranks get one more."""
    base, extra = divmod(n_requests, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return list(range(lo, hi))


def max_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()
