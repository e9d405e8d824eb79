"""world_size-2 CPU test (gloo) of the multi-GPU host logic: the (batch, head) partition, the
concatenation of per-rank results, and the max/sum reductions the benchmark uses for timing.
The per-rank compute stands in for the GPU library with the CPU oracle (test code may use it)."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import oracle
    from paper_2304_11267_b200 import distributed as D
    from paper_2304_11267_b200 import workloads
    r, lr, w = D.init_process_group("gloo")
    assert (r, w) == (rank, world)
    call = workloads.Call("t", 1, 5, 40, 77, 16, 3, padded_text=True)     # 5 units over 2 ranks: 3 + 2
    q, k, v = workloads.make_inputs(call)
    qs, ks, vs = (D.shard_bh(x, rank, world) for x in (q, k, v))
    mine, _, _ = oracle.forward(qs, ks, vs, call.scale())
    begin, end = workloads.shard_units(call.B * call.H, rank, world)
    assert mine.shape == (1, end - begin, 40, 16)
    # gather the slices on every rank (control-plane only: the data path itself has no collective)
    pieces = [None] * world
    dist.all_gather_object(pieces, (begin, end, mine))
    full = np.concatenate([p[2][0] for p in sorted(pieces, key=lambda p: p[0])], axis=0)
    ref, _, _ = oracle.forward(q, k, v, call.scale())
    assert np.array_equal(full, ref.reshape(5, 40, 16))
    D.barrier(world)
    slow = D.max_over_ranks(10.0 + rank, world)
    total = D.sum_over_ranks(float(end - begin), world)
    assert slow == 10.0 + world - 1 and total == 5.0
    open(os.path.join(out_dir, "ok%d" % rank), "w").write("ok")
    dist.destroy_process_group()


def test_two_ranks_partition_and_reduce(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert sorted(os.listdir(tmp_path)) == ["ok0", "ok1"]


def test_single_rank_helpers_are_identity():
    from paper_2304_11267_b200 import distributed as D
    assert D.max_over_ranks(3.5, 1) == 3.5 and D.sum_over_ranks(2.0, 1) == 2.0
    x = np.arange(2 * 3 * 4 * 5).reshape(2, 3, 4, 5)
    assert np.array_equal(D.shard_bh(x, 0, 1).reshape(2, 3, 4, 5), x)
    a = D.shard_bh(x, 1, 4)            # 6 units over 4 ranks: 2, 2, 1, 1
    assert a.shape == (1, 2, 4, 5) and np.array_equal(a[0], x.reshape(6, 4, 5)[2:4])


def _spawned_rank(out_dir, fail_rank):
    """What bench.py's ranks do with the environment spawn_ranks gives them (gloo instead of nccl)."""
    sys.path.insert(0, ROOT)
    from paper_2304_11267_b200 import distributed as D
    rank, local_rank, world = D.init_process_group("gloo")
    assert D.launched_by_a_launcher() and local_rank == rank and os.environ["MASTER_ADDR"] == "127.0.0.1"
    D.barrier(world)
    slowest = D.max_over_ranks(1.0 + rank, world)
    open(os.path.join(out_dir, "rank%d_of_%d" % (rank, world)), "w").write("%g" % slowest)
    dist.destroy_process_group()
    return 3 if rank == fail_rank else 0


def test_spawn_ranks_starts_every_rank_and_fails_loudly(tmp_path):
    """`bench.py --gpus N` without a launcher starts its N ranks through spawn_ranks: every rank must come up with a
    launcher's environment, and a rank that fails must fail the whole job."""
    from paper_2304_11267_b200 import distributed as D
    good = tmp_path / "good"
    good.mkdir()
    D.spawn_ranks(2, _spawned_rank, (str(good), -1))
    assert sorted(os.listdir(good)) == ["rank0_of_2", "rank1_of_2"]
    assert open(good / "rank0_of_2").read() == "2"            # the max over ranks reached rank 0
    bad = tmp_path / "bad"
    bad.mkdir()
    with pytest.raises(Exception):
        D.spawn_ranks(2, _spawned_rank, (str(bad), 1))
    with pytest.raises(ValueError):
        D.spawn_ranks(0, _spawned_rank, (str(bad), -1))
