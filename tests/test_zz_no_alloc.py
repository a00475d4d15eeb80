"""The no-allocation attention entry point against the oracle and against the regular entry point.

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

import oracle as O
import paper_2609_32518_b200 as U
import workloads as W
from harness import DevicePath, OraclePath, to_bits

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


def _check_against_oracle(got_bits, ref, what):
    # the tolerances of the other attention tests
    got = O.bf16_bits_to_f32(got_bits).astype(np.float64)
    assert np.isfinite(got).all(), what
    err = np.abs(got - ref)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3 and rel <= 1.5e-2, (what, err.max(), err.mean(), rel)


@pytest.mark.gpu
def test_noalloc_entry_point_matches_the_oracle_and_the_regular_one_twice_in_a_row():
    # 2 streams x 3 heads x 3 query pairs of 14 ragged key tiles over ~31 CTAs: most items are
    # split across CTAs, so both calls go through the scratch (partials, counters, merge)
    sh = W.Shape(batch=2, heads=3, chunk_frames=3, grid_h=8, grid_w=25, ring_frames=7)
    wl = W.Workload("noalloc", sh, seed=31, history_starts=((), ()), measured_starts=(9, 3),
                    window_frames=(7,), k_scale=4.0)
    dev, ora = DevicePath(sh), OraclePath(sh)
    for s0 in (0, 3, 6):                                   # fill the ring through the library
        q, k, v = W.batch_qkv(wl, [s0, s0])
        dev.append([s0, s0], q, k, v)
        ora.append([s0, s0], q, k, v)
    for rep, starts in enumerate(((9, 3), (6, 6))):        # two calls in a row, different windows
        q, k, v = W.batch_qkv(wl, starts, tag=rep)
        q_rot = dev.append(starts, q, k, v)
        q_ref = ora.append(starts, q, k, v)
        assert np.array_equal(to_bits(q_rot), q_ref)
        want = dev.attend(starts, 7, q_rot)                # the existing entry point
        got = torch.full_like(want.view(torch.int16), 0x7FC1).view(torch.bfloat16)
        U.window_attn_noalloc(dev.abi, list(starts), 7, q_rot, dev.ring_k, dev.ring_v, got)
        torch.cuda.synchronize()
        assert U.poll_status() == 0
        _check_against_oracle(to_bits(got), ora.attend(starts, 7, q_ref), f"call {rep}")
        # same kernel, same work split, fixed merge order: the two entry points agree bit for bit
        assert np.array_equal(to_bits(want), to_bits(got)), f"call {rep}: results differ bitwise"


@pytest.mark.gpu
def test_noalloc_with_more_streams_than_one_launch_carries():
    # 33 streams: two kernel launches of one call, back to back on one stream, share the array
    # (the second clears and reuses the counters the first has just used)
    sh = W.Shape(batch=33, heads=2, chunk_frames=1, grid_h=8, grid_w=20, ring_frames=3)
    starts = tuple(2 + (b % 3) for b in range(33))
    wl = W.Workload("noalloc33", sh, seed=32, history_starts=((),) * 33, measured_starts=starts,
                    window_frames=(3,), k_scale=4.0)
    dev, ora = DevicePath(sh), OraclePath(sh)
    for back in (2, 1):
        prev = [s - back for s in starts]
        q, k, v = W.batch_qkv(wl, prev)
        dev.append(prev, q, k, v)
        ora.append(prev, q, k, v)
    q, k, v = W.batch_qkv(wl, starts)
    q_rot = dev.append(starts, q, k, v)
    q_ref = ora.append(starts, q, k, v)
    ref = ora.attend(starts, 3, q_ref)
    for rep in range(2):
        got = torch.full_like(q_rot.view(torch.int16), 0x7FC1).view(torch.bfloat16)
        U.window_attn_noalloc(dev.abi, list(starts), 3, q_rot, dev.ring_k, dev.ring_v, got)
        torch.cuda.synchronize()
        assert U.poll_status() == 0
        _check_against_oracle(to_bits(got), ref, f"33 streams, call {rep}")
        assert np.array_equal(to_bits(dev.attend(starts, 3, q_rot)), to_bits(got))
