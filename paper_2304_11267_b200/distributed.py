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


def _free_port() -> int:
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, target, args):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    rc = target(*args)
    if rc not in (None, 0):
        raise SystemExit(int(rc))


def launched_by_a_launcher() -> bool:
    """True when RANK / WORLD_SIZE come from torchrun (or another launcher): the ranks exist already."""
    return "WORLD_SIZE" in os.environ and "RANK" in os.environ


def spawn_ranks(world: int, target, args=()) -> None:
    """Start `world` ranks of `target(*args)` on this node, one process each, with RANK / LOCAL_RANK / WORLD_SIZE /
    MASTER_ADDR (127.0.0.1) / MASTER_PORT (a free port) set as a launcher would set them, and wait for them.
    Raises if any rank fails or returns a non-zero code: a job that ends with fewer ranks than asked must not pass.
    `target` must be importable (a module-level function)."""
    if world < 1:
        raise ValueError("world size must be positive")
    import torch.multiprocessing as mp
    ctx = mp.spawn(_rank_main, args=(world, _free_port(), target, tuple(args)), nprocs=world, join=False)
    while not ctx.join():       # raises ProcessRaisedException / ProcessExitedException on the first failure
        pass
    codes = [p.exitcode for p in ctx.processes]
    if len(codes) != world or any(c != 0 for c in codes):
        raise RuntimeError("asked for %d ranks, exit codes %s" % (world, codes))


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
