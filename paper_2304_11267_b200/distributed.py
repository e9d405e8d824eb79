"""Multi-GPU plumbing: one process per GPU, no data-path collective.

Attention has no exchange step between (batch, head) pairs (Eq. 3 is evaluated per pair), so a
multi-GPU job is a partition of the flattened (batch, head) index: every rank runs the same
single-GPU library on its contiguous slice and the result is the concatenation of the slices.
The only collectives here are control-plane ones (a barrier, a max and a sum of scalars).
"""
from __future__ import annotations

import os
from typing import Tuple

from .workloads import shard_units


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init_process_group(backend: str):
    """Join the job described by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT (no-op for one rank)."""
    import torch.distributed as dist
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def shard_bh(x, rank: int, world: int):
    """Slice a [B, H, N, d] array/tensor to this rank's (batch, head) units -> [1, units, N, d]."""
    B, H = x.shape[0], x.shape[1]
    begin, end = shard_units(B * H, rank, world)
    flat = x.reshape((B * H,) + tuple(x.shape[2:]))
    return flat[begin:end].reshape((1, end - begin) + tuple(x.shape[2:]))


def barrier(world: int) -> None:
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """The slowest rank's time: the only honest duration of a multi-GPU step."""
    if world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, world: int, device="cpu") -> float:
    if world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
