"""Head-sharded execution on the GPU: a rank that owns heads [lo, hi) keeps the cache slices of
those heads and runs append and attention on them alone.  Here the two shards of a 5-head layer run
one after the other on one GPU (nothing waits on anything), each on its own head slice of the
inputs; the caches must equal the oracle's head slices bit for bit and the outputs must match the
oracle's slices within the attention tolerances."""

import numpy as np
import pytest

import workloads as W
from harness import DevicePath, OraclePath, attn_errors, to_bits
from paper_2609_32518_b200 import dist as D

pytestmark = pytest.mark.gpu


def test_two_head_shards_reproduce_the_unsharded_layer():
    sh = W.Shape(batch=2, heads=5, chunk_frames=3, grid_h=8, grid_w=25, ring_frames=7)
    wl = W.Workload("shards", sh, seed=51, history_starts=((), ()), measured_starts=(9, 3), window_frames=(7, 4),
                    k_scale=4.0)
    ora = OraclePath(sh)
    schedule = [[0, 0], [3, 0], [6, 0], [9, 3]]
    for starts in schedule[:-1]:
        ora.append(starts, *W.batch_qkv(wl, starts))
    q, k, v = W.batch_qkv(wl, schedule[-1])
    q_ref = ora.append(schedule[-1], q, k, v)
    refs = {wf: ora.attend(schedule[-1], wf, q_ref) for wf in wl.window_frames}

    world = 2
    seen = []
    for rank in range(world):
        mine = list(D.shard_heads(sh.heads, rank, world))
        seen += mine
        shard = W.with_heads(wl, len(mine))
        dev = DevicePath(shard.shape)
        for starts in schedule[:-1]:
            hq, hk, hv = W.batch_qkv(wl, starts)
            dev.append(starts, hq[:, :, mine], hk[:, :, mine], hv[:, :, mine])
        q_dev = dev.append(schedule[-1], q[:, :, mine], k[:, :, mine], v[:, :, mine])
        assert np.array_equal(to_bits(q_dev), q_ref[:, :, mine])
        assert np.array_equal(to_bits(dev.ring_k), ora.ring.ring_k[:, :, :, mine])
        assert np.array_equal(to_bits(dev.ring_v), ora.ring.ring_v[:, :, :, mine])
        for wf in wl.window_frames:
            out = to_bits(dev.attend(schedule[-1], wf, q_dev))
            got = out.astype(np.uint16)
            ref = refs[wf][:, :, mine]
            mx, mean, rel = attn_errors(got, ref)
            err_ok = np.abs(W.bf16_bits_to_f32(got).astype(np.float64) - ref) <= np.maximum(2e-2, 1.5 * 2.0 ** -8 * np.abs(ref))
            assert err_ok.all() and mean <= 2e-3 and rel <= 1.5e-2, (rank, wf, mx, mean, rel)
    assert seen == list(range(sh.heads))
