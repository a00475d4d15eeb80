"""GPU parity of the windowed attention against the float64 oracle (through the C ABI).

Tolerances are the ones the task fixes for bf16 operands with float32 accumulation:
max |err| <= 2e-2 and mean |err| <= 2e-3; a relative L2 bound is added because the
absolute bounds are loose when thousands of keys average the output towards zero."""

import os

import numpy as np
import pytest
import torch

import oracle as O
import paper_2609_32518_b200 as U
import workloads as W
from harness import (DevicePath, OraclePath, assert_ring_equal, attn_errors, stream_history, to_bits)

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS, REL_L2 = 2e-2, 2e-3, 1.5e-2


# Workloads whose keys are scaled have outputs of magnitude 4 and more (a peaked softmax returns
# single value rows).  There the rounding of the bf16 RESULT alone is up to half a unit in the last
# place = 2^-8 |o| = 1.56e-2 at |o| = 4, which leaves an ideal bf16-P / bf16-out pipeline no room
# under an absolute 2e-2 on every one of millions of elements.  The named configurations keep the
# absolute bound on every element; the extra stress shapes bound each element by
# max(2e-2, 1.5 * 2^-8 |reference|): one rounding of the result plus half as much for the rounding
# of P, whose relative error is 2^-9 per weight.
STRICT = {"cfg1", "cfg1_wrapped", "cfg2", "cfg3", "cfg3_s51", "cfg4", "cfg5"}


def check(got_bits, ref, what="", strict=True):
    mx, mean, rel = attn_errors(got_bits, ref)
    got = O.bf16_bits_to_f32(got_bits).astype(np.float64)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    if strict:
        ok_max = mx <= MAX_ABS
    else:
        ok_max = bool((np.abs(got - ref) <= np.maximum(MAX_ABS, 1.5 * 2.0 ** -8 * np.abs(ref))).all())
    assert ok_max and mean <= MEAN_ABS and rel <= REL_L2, f"{what}: max {mx:.3e} mean {mean:.3e} relL2 {rel:.3e}"
    return mx, mean, rel


@pytest.fixture(autouse=True)
def _full_compare(request):
    """--full (or UNSTEP_FULL_COMPARE=1): the sampled comparisons below become full ones."""
    global FULL
    FULL = bool(request.config.getoption("--full")) or os.environ.get("UNSTEP_FULL_COMPARE", "") == "1"
    yield


FULL = False
ERRORS = {}   # (workload, window, pass) -> (max abs, mean abs, relative L2, "full" or "sampled"), for reports


@pytest.fixture(scope="module", autouse=True)
def _error_report():
    """UNSTEP_ERRORS_JSON=<path>: write the measured errors of this module's comparisons there."""
    yield
    path = os.environ.get("UNSTEP_ERRORS_JSON")
    if path and ERRORS:
        import json
        with open(path, "w") as fh:
            json.dump({f"{k[0]} Wf={k[1]} pass={k[2]}": v for k, v in ERRORS.items()}, fh, indent=1)


def run(wl, rows_fn=None, heads=None, tag=0, dev=None, ora=None):
    """Stream the history, append the measured chunk, attend with every window length.
    `rows_fn`/`heads` restrict the comparison to a stratified sample unless a full comparison
    was asked for."""
    if FULL:
        rows_fn, heads = None, None
    if dev is None:
        dev, ora = DevicePath(wl.shape), OraclePath(wl.shape)
        stream_history(wl, dev, ora)
    s = wl.measured_starts
    q, k, v = W.batch_qkv(wl, s, tag)
    q_dev = dev.append(s, q, k, v)
    q_ref = ora.append(s, q, k, v)
    assert np.array_equal(to_bits(q_dev), q_ref)
    assert_ring_equal(dev, ora)
    L = wl.shape.chunk_tokens
    rows = None if rows_fn is None else rows_fn(L)
    for wf in wl.window_frames:
        out = to_bits(dev.attend(s, wf, q_dev))
        ref = ora.attend(s, wf, q_ref, rows=rows, heads=heads)
        got = out if rows is None else out[:, rows]
        if heads is not None:
            got = got[:, :, heads]
        ERRORS[(wl.name, wf, tag)] = check(got, ref, f"{wl.name} Wf={wf}", strict=wl.name in STRICT) + ("full" if rows is None and heads is None else "sampled",)
    assert U.poll_status() == 0
    return dev, ora


def test_cfg1_all_rows():
    run(W.WORKLOADS["cfg1"])


def test_cfg1_wrapped_windows():
    run(W.WORKLOADS["cfg1_wrapped"])


def test_startup_window_is_clamped_at_frame_zero():
    sh = W.WORKLOADS["cfg1"].shape
    wl = W.Workload("startup", sh, seed=21, history_starts=((),), measured_starts=(0,),
                    window_frames=(6, 2))
    dev, ora = DevicePath(sh), OraclePath(sh)
    run(wl, dev=dev, ora=ora)


def test_ragged_tiles_scaled_keys_two_streams():
    # T = 8*25 = 200 keys per frame (one full tile + 72), L = 600 queries (4 tiles + 88),
    # K x4 so that the running maximum moves, two streams at different fill levels
    sh = W.Shape(batch=2, heads=3, chunk_frames=3, grid_h=8, grid_w=25, ring_frames=7)
    wl = W.Workload("ragged", sh, seed=22, history_starts=((0, 3, 6, 9), (0,)),
                    measured_starts=(12, 3), window_frames=(7, 5, 3), k_scale=4.0)
    run(wl)


def test_zero_keys_mean_of_frames_through_the_kernel():
    # K = 0 and V[frame p] = p: the output is the mean of the attended frame indices
    sh = W.Shape(batch=1, heads=1, chunk_frames=3, grid_h=4, grid_w=40, ring_frames=9)
    dev = DevicePath(sh)
    T = sh.tokens_per_frame
    for p in range(21):
        dev.ring_k[0, p % 9] = 0
        dev.ring_v[0, p % 9] = float(p)
    q = torch.randn((1, sh.chunk_tokens, 1, 128), device="cuda").to(torch.bfloat16)
    for wf, want in ((9, 16.0), (6, 17.5), (4, 18.5), (3, 19.0)):
        out = dev.attend([18], wf, q).float()
        assert torch.allclose(out, torch.full_like(out, want), atol=0.07), (wf, out.mean().item())


def test_unused_ring_slots_may_hold_nan():
    # slots outside the window (and the ragged end of a frame) never reach the output
    wl = W.WORKLOADS["cfg1"]
    dev, ora = DevicePath(wl.shape), OraclePath(wl.shape)   # rings start as NaN sentinels
    wl2 = W.Workload("nan", wl.shape, seed=23, history_starts=((),), measured_starts=(2,),
                     window_frames=(2,))
    run(wl2, dev=dev, ora=ora)


def test_cfg2_every_row_and_head():
    # the shape the metric is quoted on is always compared in full
    run(W.WORKLOADS["cfg2"])


def test_cfg3_window_sweep_sampled_rows():
    run(W.WORKLOADS["cfg3"], rows_fn=lambda L: W.sample_rows(L, per_tile=3), heads=[0, 5, 11])


def test_cfg3_second_point_where_only_the_longest_window_wraps():
    run(W.WORKLOADS["cfg3_s51"], rows_fn=lambda L: W.sample_rows(L, per_tile=3), heads=[1, 6, 10])


def test_cfg3_tight_ring_capacity_equals_window():
    run(W.WORKLOADS["cfg3_tight"], rows_fn=lambda L: W.sample_rows(L, per_tile=3), heads=[2, 7, 11])


def test_cfg4_clean_cache_pattern():
    wl = W.WORKLOADS["cfg4"]
    rows_fn = lambda L: W.sample_rows(L, per_tile=2)   # noqa: E731
    dev, ora = run(wl, rows_fn=rows_fn, heads=[0, 7], tag=0)
    # clean pass: fresh K/V for the same chunk at the same positions, then re-query
    run(wl, rows_fn=rows_fn, heads=[3, 11], tag=1, dev=dev, ora=ora)


def test_cfg5_sampled_rows():
    run(W.WORKLOADS["cfg5"], rows_fn=lambda L: W.sample_rows(L, per_tile=2), heads=[0, 13, 39])


def test_more_streams_than_one_launch_carries():
    # 35 streams (the per-launch parameter block holds 32), one short frame per chunk, own positions
    sh = W.Shape(batch=35, heads=1, chunk_frames=1, grid_h=4, grid_w=10, ring_frames=4)
    starts = tuple(3 + (b % 5) for b in range(35))
    wl = W.Workload("many", sh, seed=24, history_starts=((),) * 35, measured_starts=starts,
                    window_frames=(4, 2, 1))
    dev, ora = DevicePath(sh), OraclePath(sh)
    for back in (3, 2, 1):                       # frames start-3 .. start-1 of every stream
        prev = [s - back for s in starts]
        q, k, v = W.batch_qkv(wl, prev)
        dev.append(prev, q, k, v)
        ora.append(prev, q, k, v)
    run(wl, dev=dev, ora=ora)


def test_queries_shorter_than_a_tile_and_single_head():
    # L = 2*3*5 = 30 queries, T = 15 keys per frame: one ragged query tile, per-frame key tiles
    sh = W.Shape(batch=2, heads=1, chunk_frames=2, grid_h=3, grid_w=5, ring_frames=6)
    wl = W.Workload("short", sh, seed=25, history_starts=((0, 2, 4), (0,)), measured_starts=(6, 2),
                    window_frames=(6, 3, 2), k_scale=4.0)
    run(wl)


def test_split_items_merge_in_a_fixed_order_bitwise_repeatable():
    # The 1.3B shape leaves 80 of its 228 work items to be split along the keys between CTAs;
    # whichever part finishes last merges them, in part order, so repeated launches must agree
    # bit for bit although the finishing order varies.  A large K scale forces rescales of O.
    wl = W.WORKLOADS["cfg3"]
    sh = wl.shape
    gen = torch.Generator(device="cuda").manual_seed(5)
    dims = (sh.batch, sh.ring_frames, sh.tokens_per_frame, sh.heads, sh.head_dim)
    ring_k = (4.0 * torch.randn(dims, generator=gen, device="cuda")).to(torch.bfloat16)
    ring_v = torch.randn(dims, generator=gen, device="cuda").to(torch.bfloat16)
    q = torch.randn((sh.batch, sh.chunk_tokens, sh.heads, sh.head_dim), generator=gen,
                    device="cuda").to(torch.bfloat16)
    abi = U.Shape.make(sh.batch, sh.heads, sh.chunk_frames, sh.grid_h, sh.grid_w, sh.ring_frames)
    for wf in (21, 6):
        outs = []
        for _ in range(4):
            out = torch.empty_like(q)
            U.window_attn(abi, [42], wf, q, ring_k, ring_v, out)
            outs.append(out.view(torch.int16).clone())
        torch.cuda.synchronize()
        assert all(torch.equal(outs[0], o) for o in outs[1:]), f"Wf={wf}: launches differ"
        assert torch.isfinite(out.float()).all()
    assert U.poll_status() == 0


def test_scores_far_above_the_first_tiles_maximum_take_the_redo_path():
    # Later key tiles are exponentiated against the first tile's row maximum and only checked
    # afterwards; scores more than 64 (log2 units) above it make the kernel find the true
    # maximum, rescale and redo the tile.  History with ordinary keys, then a chunk whose keys are
    # 64 times larger: its scores have a standard deviation of ~90 log2 units.
    base = W.WORKLOADS["cfg1"]
    dev, ora = DevicePath(base.shape), OraclePath(base.shape)
    stream_history(base, dev, ora)
    big = W.Workload("huge_keys", base.shape, seed=26, history_starts=base.history_starts,
                     measured_starts=base.measured_starts, window_frames=(6, 4), k_scale=64.0)
    run(big, dev=dev, ora=ora)
    # and back to ordinary keys on top of the huge ones (the reference maximum is now far too high
    # for most rows of the newest keys: their weights underflow, as in the exact softmax)
    after = W.Workload("after_huge", base.shape, seed=27, history_starts=base.history_starts,
                       measured_starts=(6,), window_frames=(6, 2))
    run(after, dev=dev, ora=ora)


def test_single_huge_key_in_a_late_tile_is_caught():
    # One key of a late tile scores hundreds of log2 units above everything else for about half of
    # the rows (its exponential against the first tile's maximum overflows to inf): those rows
    # must be redone against the true maximum.
    wl = W.WORKLOADS["cfg1"]
    dev, ora = DevicePath(wl.shape), OraclePath(wl.shape)
    stream_history(wl, dev, ora)             # 4 frames of 64 tokens = two full key tiles
    s = wl.measured_starts
    q, k, v = W.batch_qkv(wl, s, 3)
    k = k.copy()
    k[:, 0] = W.f32_to_bf16_bits(W.bf16_bits_to_f32(k[:, 0]) * np.float32(256.0))   # column 0 of tile 2
    q_dev = dev.append(s, q, k, v)
    q_ref = ora.append(s, q, k, v)
    assert np.array_equal(to_bits(q_dev), q_ref)
    assert_ring_equal(dev, ora)
    for wf in wl.window_frames:
        out = to_bits(dev.attend(s, wf, q_dev))
        check(out, ora.attend(s, wf, q_ref), f"huge key Wf={wf}")
    assert U.poll_status() == 0


def test_remainder_smaller_than_the_grid():
    # Work splits whose remainder has fewer steps than there are thread blocks: 11 heads of one
    # query tile over 2 key tiles (the launch shrinks to a few blocks), and 10 heads x 15 query
    # pairs = 150 items on 148 blocks (one whole round, then 2 items x 30 tiles for everybody).
    sh = W.Shape(batch=1, heads=11, chunk_frames=2, grid_h=8, grid_w=8, ring_frames=2)
    run(W.Workload("tiny11", sh, seed=28, history_starts=((),), measured_starts=(0,), window_frames=(2,)))
    sh = W.Shape(batch=1, heads=10, chunk_frames=3, grid_h=32, grid_w=40, ring_frames=3)
    wl = W.Workload("rem60", sh, seed=29, history_starts=((),), measured_starts=(0,), window_frames=(3,),
                    k_scale=4.0)
    # the two leftover items are the last two query pairs of the last head: rows 3328.. of head 9
    run(wl, rows_fn=lambda L: np.concatenate([W.sample_rows(L, per_tile=2), np.arange(3328, L, 7)]), heads=[0, 9])
