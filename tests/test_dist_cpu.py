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


def _head_worker(rank, world, port, out):
    """One rank of a head-sharded layer on CPU: it owns its heads' cache slices, runs the oracle's
    append and attention on them alone, and the ranks' outputs are gathered along the head axis."""
    import numpy as np
    import torch.distributed as dist
    import oracle as O
    import workloads as W
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    D.init("gloo")
    sh = W.Shape(batch=2, heads=5, chunk_frames=2, grid_h=4, grid_w=6, ring_frames=4)
    wl = W.Workload("heads", sh, seed=41, history_starts=((0, 2), (0,)), measured_starts=(4, 2), window_frames=(4,))
    mine = list(D.shard_heads(sh.heads, rank, world))
    ring = O.RingState(sh.batch, sh.ring_frames, sh.tokens_per_frame, len(mine))
    tabs = {}

    def append(starts):
        q, k, v = W.batch_qkv(wl, starts)                      # all heads' inputs, then this rank's slice
        for st in starts:
            tabs.setdefault(st, O.rope_table(st, sh.chunk_frames, sh.grid_h, sh.grid_w))
        cos = np.stack([tabs[st][0] for st in starts])
        sin = np.stack([tabs[st][1] for st in starts])
        return O.rope_kv_append(ring, starts, q[:, :, mine], k[:, :, mine], v[:, :, mine], cos, sin)

    append([0, 0])
    append([2, 0])
    q_rot = append([4, 2])
    part = O.window_attn(ring, [4, 2], 4, q_rot, sh.chunk_frames)      # [B, L, my heads, 128]
    parts = [None] * world
    dist.all_gather_object(parts, (mine, part))
    D.finalize()
    if rank == 0:
        out.put(parts)


def test_head_shards_reassemble_the_unsharded_result():
    import numpy as np
    import oracle as O
    import workloads as W
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_head_worker, args=(r, world, port, out)) for r in range(world)]
    for pr in procs:
        pr.start()
    parts = out.get(timeout=180)
    for pr in procs:
        pr.join(timeout=60)
        assert pr.exitcode == 0
    # the same layer unsharded
    sh = W.Shape(batch=2, heads=5, chunk_frames=2, grid_h=4, grid_w=6, ring_frames=4)
    wl = W.Workload("heads", sh, seed=41, history_starts=((0, 2), (0,)), measured_starts=(4, 2), window_frames=(4,))
    ring = O.RingState(sh.batch, sh.ring_frames, sh.tokens_per_frame, sh.heads)
    q_rot = None
    for starts in ([0, 0], [2, 0], [4, 2]):
        q, k, v = W.batch_qkv(wl, starts)
        tabs = [O.rope_table(st, sh.chunk_frames, sh.grid_h, sh.grid_w) for st in starts]
        q_rot = O.rope_kv_append(ring, starts, q, k, v, np.stack([t[0] for t in tabs]), np.stack([t[1] for t in tabs]))
    whole = O.window_attn(ring, [4, 2], 4, q_rot, sh.chunk_frames)
    heads = [h for mine, _ in parts for h in mine]
    assert heads == list(range(sh.heads))                      # every head once, in order
    glued = np.concatenate([p for _, p in parts], axis=2)
    assert np.array_equal(glued, whole)                        # heads are independent: identical, not just close


@pytest.mark.parametrize("n,world", [(12, 2), (12, 3), (12, 4), (12, 6), (40, 8), (12, 8), (5, 2)])
def test_head_split_is_a_balanced_partition(n, world):
    sizes, seen = [], []
    for r in range(world):
        part = list(D.shard_heads(n, r, world))
        sizes.append(len(part))
        seen += part
    assert seen == list(range(n)) and max(sizes) - min(sizes) <= 1


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    import importlib.util
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(root, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    cmd = bench.relaunch_command(8, 29555, ["--gpus", "8", "--steps", "20"])
    assert cmd[0] == sys.executable and cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--nproc-per-node=8" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29555"
    assert cmd[-4:] == ["--gpus", "8", "--steps", "20"] and cmd[-5].endswith("bench.py")
