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


# ------------------------------------------------------------------------------------------------
# One weight matrix split by rows over the ranks (the paper runs OPT-66B on two GPUs, Sec. 5.3)
def row_shard(M: int, rank: int, world: int, tile: int = 128):
    """Rows [r0, r1) of an M-row matrix that rank `rank` of `world` holds: whole row-tiles (a tile of
    the format is never cut), dealt out contiguously and as evenly as the tile count allows."""
    tiles = (M + tile - 1) // tile
    t0, t1 = tiles * rank // world, tiles * (rank + 1) // world
    return min(M, t0 * tile), min(M, t1 * tile)


class RowShardedMatrix:
    """`Y = W X` with W split by rows over the ranks of the default process group: every rank
    encodes and keeps only its slab of W, X is the same on all ranks (an activation block is a few
    hundred KB), each rank's kernel writes its slab of Y, and one all-gather after the kernel gives
    every rank the whole Y -- an ordinary collective on the result, nothing fused into the kernel and
    no peer memory handed to it.

    `local_product(W_slab) -> f(X) -> Y_slab` builds the per-rank product.  The default encodes the
    slab with the library and multiplies on the current CUDA device (no fallback); tests pass a
    CPU stand-in to exercise the partitioning and the collective over gloo."""

    def __init__(self, W, local_product=None, tile: int = 128):
        import numpy as np
        rank, _, world = env_world()
        self.M, self.K = W.shape
        self.rank, self.world = rank, world
        self.ranges = [row_shard(self.M, r, world, tile) for r in range(world)]
        r0, r1 = self.ranges[rank]
        self.max_rows = max(b - a for a, b in self.ranges)
        slab = np.ascontiguousarray(W[r0:r1])
        self._product = (local_product or _gpu_product)(slab) if r1 > r0 else None

    def matmul(self, X):
        """X: K x N (torch tensor on this rank's device, the same values on every rank).  Returns
        the whole M x N product on every rank."""
        import torch
        import torch.distributed as dist
        N = X.shape[1]
        r0, r1 = self.ranges[self.rank]
        mine = torch.zeros((self.max_rows, N), dtype=torch.float16, device=X.device)   # slabs are padded to one size
        if self._product is not None:
            mine[: r1 - r0] = self._product(X)
        if self.world == 1 or not (dist.is_available() and dist.is_initialized()):
            return mine[: r1 - r0]
        parts = [torch.empty_like(mine) for _ in range(self.world)]
        dist.all_gather(parts, mine)
        return torch.cat([p[: b - a] for p, (a, b) in zip(parts, self.ranges)], dim=0)


def _gpu_product(W_slab):
    from . import tl3
    m = tl3.encode(W_slab)
    m.upload()
    return lambda X: m.spmm(X)
