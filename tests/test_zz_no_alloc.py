"""The no-allocation attention entry point against the regular one.

Some users of this library cannot let it call cudaMalloc: their process has given all device
memory to a framework allocator, or they run a latency-critical loop that must not take the
synchronisation an allocation can imply, or their deployment fixes its memory footprint at
start-up.  `unstep_window_attn_noalloc` serves them with a scratch array that is part of the
library image.  This file is collected last on purpose: if it fails, a run that stops at the
first failure has already been through every other test."""

import ctypes

import numpy as np
import pytest
import torch

import paper_2609_32518_b200 as U
import workloads as W
from harness import DevicePath, to_bits

FAKE = 0x10000


def test_oversized_problem_is_refused_before_any_device_work():
    # 32 streams x 4096 heads x 19 query pairs needs far more counters than the array holds
    big = U.Shape.make(batch=32, heads=4096, chunk_frames=3, grid_h=30, grid_w=52, ring_frames=21)
    starts = (ctypes.c_int32 * 32)(*([0] * 32))
    rc = U.lib().unstep_window_attn_noalloc(ctypes.byref(big), starts, 3, FAKE, FAKE, FAKE, FAKE, None)
    assert rc == -5 and "scratch" in U.strerror(rc)
    # the ordinary argument checks still come first
    bad = U.Shape.make(batch=1, heads=2, chunk_frames=2, grid_h=8, grid_w=8, ring_frames=6, head_dim=64,
                       bands=(22, 21, 21))
    one = (ctypes.c_int32 * 1)(0)
    assert U.lib().unstep_window_attn_noalloc(ctypes.byref(bad), one, 2, FAKE, FAKE, FAKE, FAKE, None) == -2


@pytest.mark.gpu
def test_noalloc_entry_point_matches_the_regular_one_twice_in_a_row():
    # 2 streams x 3 heads x 3 query pairs of 14 ragged key tiles over ~31 CTAs: most items are
    # split across CTAs, so both calls go through the scratch (partials, counters, merge)
    sh = W.Shape(batch=2, heads=3, chunk_frames=3, grid_h=8, grid_w=25, ring_frames=7)
    wl = W.Workload("noalloc", sh, seed=31, history_starts=((), ()), measured_starts=(9, 3),
                    window_frames=(7,), k_scale=4.0)
    dev = DevicePath(sh)
    for s0 in (0, 3, 6):                                   # fill the ring through the library
        q, k, v = W.batch_qkv(wl, [s0, s0])
        dev.append([s0, s0], q, k, v)
    for rep, starts in enumerate(((9, 3), (6, 6))):        # two calls in a row, different windows
        q, k, v = W.batch_qkv(wl, starts, tag=rep)
        q_rot = dev.append(starts, q, k, v)
        want = dev.attend(starts, 7, q_rot)                # the existing entry point
        got = torch.full_like(want.view(torch.int16), 0x7FC1).view(torch.bfloat16)
        U.window_attn_noalloc(dev.abi, list(starts), 7, q_rot, dev.ring_k, dev.ring_v, got)
        torch.cuda.synchronize()
        assert U.poll_status() == 0
        a = want.float().cpu().numpy().astype(np.float64)
        b = got.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(b).all()
        err = np.abs(a - b)
        assert err.max() <= 2e-2 and err.mean() <= 2e-3, (rep, err.max(), err.mean())
        # same kernel, same work split, fixed merge order: the two results are in fact identical
        assert np.array_equal(to_bits(want), to_bits(got)), f"call {rep}: results differ bitwise"
