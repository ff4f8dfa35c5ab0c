"""Process-group plumbing for running the SpMM workload on several GPUs of one node.

The hot path has no exchange step: each rank holds its own weight matrices and activation
blocks (independent problems), so ranks share nothing but the launch and the timing -- a barrier
on both sides of the timed region and a max-reduction of the per-rank device time.
"""
from __future__ import annotations

import os
from typing import List, Sequence, TypeVar

T = TypeVar("T")


def env_world():
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init_process_group(backend: str):
    """Join the process group the launcher described (MASTER_ADDR / MASTER_PORT in the env)."""
    import torch.distributed as dist
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: what a multi-GPU number is quoted on."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def rank_seed_offset(rank: int) -> int:
    """Every rank draws its own matrices: same shapes and recipe, seeds shifted by 100000*rank."""
    return 100000 * rank


def shard_round_robin(items: Sequence[T], rank: int, world: int) -> List[T]:
    """Independent problems dealt out to ranks in turn (used when the total work is fixed)."""
    return [x for i, x in enumerate(items) if i % world == rank]
