"""The work split of the attention kernel, replayed on the host (no GPU).

The kernel's roles all walk the same integer schedule; `unstep_window_attn_plan` lists it with the
same code compiled for the host.  Whatever the shape, window and worker count, every (item, key
tile) step must be covered exactly once, a split item's parts must be counted correctly (a part
that waits for more parts than exist would never merge, and its rows would never be written), and
no two parts of one worker may share a scratch slot."""

import itertools

import pytest

import paper_2609_32518_b200 as U


def check_plan(shape, starts, window, workers, sink=0, sink_attend=0):
    segs = U.window_attn_plan(shape, starts, window, workers, sink, sink_attend)
    T = shape.grid_h * shape.grid_w
    q_tiles = -(-shape.chunk_frames * T // 128)
    q_pairs = (q_tiles + 1) // 2
    covered = {}
    parts_seen = {}
    slots_of_worker = {}
    for (w, b, h, qp, nq, t0, t1, tiles, parts, slot) in segs:
        assert 0 <= w < workers and 0 <= b < shape.batch and 0 <= h < shape.heads and 0 <= qp < q_pairs
        assert nq == (2 if 2 * qp + 1 < q_tiles else 1)
        assert 0 <= t0 < t1 <= tiles
        item = (b, h, qp)
        for t in range(t0, t1):
            assert (item, t) not in covered, f"step {(item, t)} given to two workers"
            covered[(item, t)] = w
        whole = t0 == 0 and t1 == tiles
        assert (parts == 1 and slot == -1) if whole else (parts >= 2 and slot in (0, 1))
        if not whole:
            parts_seen.setdefault(item, []).append((w, parts))
            assert slot not in slots_of_worker.setdefault(w, set()), f"worker {w} reuses scratch slot {slot}"
            slots_of_worker[w].add(slot)
    # every step of every item exactly once
    n_items = shape.batch * shape.heads * q_pairs
    items = {k[0] for k in covered}
    assert len(items) == n_items
    by_item = {}
    for (item, t) in covered:
        by_item.setdefault(item, set()).add(t)
    tiles_of = {}
    for (w, b, h, qp, nq, t0, t1, tiles, parts, slot) in segs:
        tiles_of[(b, h, qp)] = tiles
    for item, ts in by_item.items():
        assert ts == set(range(tiles_of[item])), f"item {item}: steps missing"
    # a split item: as many parts as each of its parts expects, on consecutive workers
    for item, lst in parts_seen.items():
        ws = sorted(w for w, _ in lst)
        assert all(n == len(lst) for _, n in lst), f"item {item}: {len(lst)} parts, expected {[n for _, n in lst]}"
        assert ws == list(range(ws[0], ws[0] + len(ws)))
    return segs


def test_shapes_whose_remainder_is_smaller_than_the_grid():
    # 10 heads x 15 query pairs = 150 items on 148 workers: one whole round, then 2 items x 30
    # tiles = 60 steps for 148 workers
    sh = U.Shape.make(batch=1, heads=10, chunk_frames=3, grid_h=32, grid_w=40, ring_frames=3)
    segs = check_plan(sh, [0], 3, 148)
    assert max(s[0] for s in segs) == 147
    # 11 heads of one query tile, 2 key tiles in all: the launch shrinks to very few workers
    sh = U.Shape.make(batch=1, heads=11, chunk_frames=2, grid_h=8, grid_w=8, ring_frames=2)
    check_plan(sh, [0], 2, 148)


def test_the_1p3b_and_14b_shapes_on_148_and_74_workers():
    sh = U.Shape.make(batch=1, heads=12, chunk_frames=3, grid_h=30, grid_w=52, ring_frames=21)
    for workers in (148, 74):
        segs = check_plan(sh, [18], 21, workers)
        assert sum(s[6] - s[5] for s in segs) == 12 * 19 * 256
    sh5 = U.Shape.make(batch=1, heads=40, chunk_frames=3, grid_h=45, grid_w=80, ring_frames=12)
    check_plan(sh5, [9], 12, 148)
    sh4 = U.Shape.make(batch=4, heads=12, chunk_frames=3, grid_h=30, grid_w=52, ring_frames=21)
    check_plan(sh4, [0, 6, 12, 18], 21, 148)


@pytest.mark.parametrize("workers", [1, 2, 5, 31, 74, 148])
def test_sweep_of_small_shapes(workers):
    for heads, (gh, gw), fc, win in itertools.product((1, 2, 3, 10, 11), ((8, 8), (8, 25), (3, 5), (16, 20)),
                                                      (1, 2, 3), (0, 1, 4)):
        ring = fc + win
        sh = U.Shape.make(batch=2, heads=heads, chunk_frames=fc, grid_h=gh, grid_w=gw, ring_frames=ring)
        check_plan(sh, [ring + 1, 0], ring, workers)


def test_sink_prefix_and_bad_arguments():
    sh = U.Shape.make(batch=1, heads=12, chunk_frames=3, grid_h=30, grid_w=52, ring_frames=6)
    segs = check_plan(sh, [18], 6, 148, sink=3, sink_attend=3)
    # frames 0..2 sit in slots 0..2 and frames 15..20 in slots 3..8: one run of 14040 keys
    assert segs[0][7] == -(-9 * 1560 // 128)
    # a chunk later the ring has wrapped: frames 18..20 in slots 6..8, 21..23 in slots 3..5 -> runs 0..2 | 6..8 | 3..5
    segs = check_plan(sh, [21], 6, 148, sink=3, sink_attend=3)
    assert segs[0][7] == 3 * -(-3 * 1560 // 128)
    with pytest.raises(U.UnstepError):
        U.window_attn_plan(sh, [18], 7, 148)          # window longer than the ring
    with pytest.raises(U.UnstepError):
        U.window_attn_plan(sh, [18], 6, 0)            # no workers
