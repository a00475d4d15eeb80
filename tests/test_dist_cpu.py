"""The multi-rank plumbing of the benchmark on CPU: two gloo ranks."""

import os
import socket

import pytest
import torch
import torch.multiprocessing as mp

from paper_2609_32518_b200 import dist as D


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r, lr, w = D.init("gloo")
    assert (r, lr, w) == (rank, rank, world)
    D.barrier()
    slowest = D.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow one
    streams = list(D.shard_streams(5, rank, world))
    D.barrier()
    D.finalize()
    out.put((rank, slowest, streams))


def test_two_gloo_ranks_barrier_max_and_stream_split():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for pr in procs:
        pr.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for pr in procs:
        pr.join(timeout=60)
        assert pr.exitcode == 0
    assert [g[1] for g in got] == [15.0, 15.0]              # every rank sees the slowest time
    assert got[0][2] + got[1][2] == [0, 1, 2, 3, 4]         # streams covered once, none split
    assert abs(len(got[0][2]) - len(got[1][2])) <= 1


def test_single_process_is_a_no_op():
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert D.env_ranks() == (0, 0, 1)
    assert D.max_over_ranks(3.5) == 3.5
    D.barrier()
    assert list(D.shard_streams(4, 0, 1)) == [0, 1, 2, 3]


@pytest.mark.parametrize("n,world", [(4, 8), (12, 8), (1, 2), (37, 4)])
def test_stream_split_is_a_partition(n, world):
    seen = []
    for r in range(world):
        seen += list(D.shard_streams(n, r, world))
    assert seen == list(range(n))
