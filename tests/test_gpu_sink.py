"""GPU parity of the sink + sliding-window cache against the oracle (through the C ABI)."""

import numpy as np
import pytest
import torch

import oracle as O
import paper_2609_32518_b200 as U
import workloads as W
from harness import DevicePath, attn_errors, to_bits

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS, REL_L2 = 2e-2, 2e-3, 1.5e-2


def tables(sh, s):
    return O.rope_table(s, sh.chunk_frames, sh.grid_h, sh.grid_w, sh.bands, sh.rope_base)


def check(got_bits, ref, what):
    mx, mean, rel = attn_errors(got_bits, ref)
    assert np.isfinite(O.bf16_bits_to_f32(got_bits)).all(), what
    assert mx <= MAX_ABS and mean <= MEAN_ABS and rel <= REL_L2, f"{what}: {mx:.3e} {mean:.3e} {rel:.3e}"


def test_long_stream_soak_cache_bit_exact_and_attention_in_tolerance():
    # 41 chunks of 3 frames: positions 0..122 through a 3 + 6 frame cache, as in a 30 s clip;
    # T = 8*25 = 200 keys per frame (ragged tiles), 2 heads
    sh = W.Shape(batch=1, heads=2, chunk_frames=3, grid_h=8, grid_w=25, ring_frames=6)
    wl = W.Workload("soak", sh, seed=51, history_starts=((),), measured_starts=(0,), window_frames=(6,),
                    k_scale=4.0)
    dev = DevicePath(sh, sink_frames=3)
    ora = O.SinkRingState(1, 3, 6, sh.tokens_per_frame, sh.heads)
    for c in range(41):
        s = 3 * c
        q, k, v = W.batch_qkv(wl, [s])
        cos, sin = tables(sh, s)
        q_dev = dev.append([s], q, k, v)
        q_ref = O.rope_kv_append_sink(ora, [s], q, k, v, cos, sin)
        assert np.array_equal(to_bits(q_dev), q_ref)
        assert np.array_equal(to_bits(dev.ring_k), ora.cache_k), f"cache K differs after chunk {c}"
        assert np.array_equal(to_bits(dev.ring_v), ora.cache_v), f"cache V differs after chunk {c}"
        if c in (0, 1, 2, 3, 4, 11, 40):
            for sink_attend in (3, 2, 0):
                out = to_bits(dev.attend_sink([s], 6, sink_attend, q_dev))
                ref = O.window_attn_sink(ora, [s], 6, sink_attend, q_ref, 3)
                check(out, ref, f"chunk {c} sink {sink_attend}")
    assert U.poll_status() == 0


def test_zero_keys_mean_of_sink_and_recent_frames_through_the_kernel():
    sh = W.Shape(batch=1, heads=1, chunk_frames=3, grid_h=4, grid_w=40, ring_frames=6)
    dev = DevicePath(sh, sink_frames=3)
    for p in range(21):
        slot = O.sink_slot(p, 3, 6)
        dev.ring_k[0, slot] = 0
        dev.ring_v[0, slot] = float(p)
    q = torch.randn((1, sh.chunk_tokens, 1, 128), device="cuda").to(torch.bfloat16)
    for sink_attend, want in ((3, 12.0), (2, 13.25), (0, 17.5)):
        out = dev.attend_sink([18], 6, sink_attend, q).float()
        assert torch.allclose(out, torch.full_like(out, want), atol=0.07), (sink_attend, out.mean().item())


def test_sink_zero_is_the_plain_rolling_window():
    wl = W.WORKLOADS["cfg1_wrapped"]
    a, b = DevicePath(wl.shape), DevicePath(wl.shape)
    q_dev = None
    for s in list(wl.history_starts[0]) + [16]:
        q, k, v = W.batch_qkv(wl, [s])
        q_dev = a.append([s], q, k, v)
        q2 = torch.empty_like(q_dev)
        cos, sin = b.table(s)
        from harness import to_dev
        U.rope_kv_append_sink(b.abi, 0, [s], to_dev(q), to_dev(k), to_dev(v), cos, sin, q2, b.ring_k, b.ring_v)
        assert torch.equal(q2.view(torch.int16), q_dev.view(torch.int16))
    assert torch.equal(a.ring_k.view(torch.int16), b.ring_k.view(torch.int16))
    out_a = a.attend([16], 6, q_dev)
    out_b = torch.empty_like(out_a)
    U.window_attn_sink(b.abi, 0, [16], 6, 0, q_dev, b.ring_k, b.ring_v, out_b)
    assert torch.equal(out_a.view(torch.int16), out_b.view(torch.int16))


def test_1p3b_shape_nine_frame_cache_sampled_rows():
    # the paper's operating point: 3 sink + 6 recent frames = 14040 keys, last chunk of a clip
    sh = W.Shape(batch=1, heads=12, chunk_frames=3, grid_h=30, grid_w=52, ring_frames=6)
    wl = W.Workload("sink9", sh, seed=52, history_starts=((),), measured_starts=(18,), window_frames=(6,))
    dev = DevicePath(sh, sink_frames=3)
    ora = O.SinkRingState(1, 3, 6, sh.tokens_per_frame, sh.heads)
    q_dev = q_ref = None
    for s in range(0, 21, 3):
        q, k, v = W.batch_qkv(wl, [s])
        cos, sin = tables(sh, s)
        q_dev = dev.append([s], q, k, v)
        q_ref = O.rope_kv_append_sink(ora, [s], q, k, v, cos, sin)
    assert np.array_equal(to_bits(dev.ring_k), ora.cache_k) and np.array_equal(to_bits(dev.ring_v), ora.cache_v)
    rows = W.sample_rows(sh.chunk_tokens, per_tile=3)
    for sink_attend in (3, 2):
        out = to_bits(dev.attend_sink([18], 6, sink_attend, q_dev))
        ref = O.window_attn_sink(ora, [18], 6, sink_attend, q_ref, 3, rows=rows, heads=[0, 6, 11])
        check(out[:, rows][:, :, [0, 6, 11]], ref, f"9-frame cache, sink {sink_attend}")


def test_sink_argument_checks():
    import ctypes
    sh = U.Shape.make(batch=1, heads=2, chunk_frames=2, grid_h=8, grid_w=8, ring_frames=6)
    one = (ctypes.c_int32 * 1)(0)
    f = 0x10000
    L = U.lib()
    assert L.unstep_window_attn_sink(ctypes.byref(sh), 3, one, 6, 4, f, f, f, f, None) == -1   # attend > stored
    assert L.unstep_window_attn_sink(ctypes.byref(sh), -1, one, 6, 0, f, f, f, f, None) == -1
    assert L.unstep_window_attn_sink(ctypes.byref(sh), 3, one, 7, 3, f, f, f, f, None) == -1   # recent > ring
    assert L.unstep_rope_kv_append_sink(ctypes.byref(sh), -2, one, f, f, f, f, f, 0, f, f, f, None) == -1


def test_short_frames_sink_cache_per_frame_tiles():
    # T = 6*7 = 42 keys per frame (< one tile): the per-frame addressing with a sink prefix
    sh = W.Shape(batch=2, heads=2, chunk_frames=3, grid_h=6, grid_w=7, ring_frames=6)
    wl = W.Workload("short_sink", sh, seed=53, history_starts=((), ()), measured_starts=(0, 0),
                    window_frames=(6,), k_scale=4.0)
    dev = DevicePath(sh, sink_frames=2)
    ora = O.SinkRingState(2, 2, 6, sh.tokens_per_frame, sh.heads)
    for c in range(9):
        starts = [3 * c, 3 * c]
        q, k, v = W.batch_qkv(wl, starts)
        cos, sin = tables(sh, 3 * c)
        q_dev = dev.append(starts, q, k, v)
        q_ref = O.rope_kv_append_sink(ora, starts, q, k, v, cos, sin)
        assert np.array_equal(to_bits(dev.ring_k), ora.cache_k)
        for sink_attend in (2, 1):
            out = to_bits(dev.attend_sink(starts, 6, sink_attend, q_dev))
            check(out, O.window_attn_sink(ora, starts, 6, sink_attend, q_ref, 3), f"chunk {c} sink {sink_attend}")
    assert U.poll_status() == 0
