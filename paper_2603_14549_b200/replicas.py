"""Process-group plumbing for running the prune step as independent replicas.

Every sequence of a batch is pruned on its own (all sums of Eq. 1-5 stay inside one sequence),
so several GPUs never exchange data: each rank owns whole sequences and runs the single-GPU
library on them.  What the ranks do share is bookkeeping -- a barrier before and after a timed
region, the slowest rank's time, the total number of tokens processed -- and that is all this
module does.  It works with any torch.distributed backend (nccl on GPUs, gloo on CPUs).
"""
from __future__ import annotations

import os
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def world() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment; (0, 1, 0) without one."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str) -> Tuple[int, int, int]:
    """Joins the process group when launched with more than one rank."""
    rank, size, local = world()
    if size > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=size)
    return rank, size, local


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def _reduce(value: float, op, device) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.MAX, device)


def sum_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.SUM, device)


def shard_sequences(n_sequences: int, world_size: int, rank: int) -> List[int]:
    """Strong-scaling split of one batch: whole sequences, contiguous, sizes differing by at
    most one, every sequence owned by exactly one rank."""
    base, extra = divmod(n_sequences, world_size)
    lo = rank * base + min(rank, extra)
    return list(range(lo, lo + base + (1 if rank < extra else 0)))


def replica_seed(base_seed: int, rank: int) -> int:
    """Weak scaling: every rank draws its own batch of the same shape."""
    return base_seed + 100003 * rank


def aggregate_throughput(units_per_rank: Sequence[float], seconds_per_rank: Sequence[float]) -> float:
    """Whole-job throughput: all units over the slowest rank's time."""
    return float(sum(units_per_rank)) / max(seconds_per_rank)
