"""Pins for the oracle's sink + sliding-window cache (CPU only)."""

import numpy as np

import oracle as O
import workloads as W
from test_oracle_rope import load_facts


def test_frame_sets_match_the_paper():
    f = load_facts()
    sink, total = int(f["sink_frames"]), int(f["sink_plus_recent_frames"])
    recent = int(f["recent_frames_incl_chunk"])
    assert sink + recent == total
    # cache full: the last chunk of a 21-frame clip sees 3 sink frames + the 6 most recent
    frames = O.sink_window_frames(18, 3, recent, sink)
    assert frames == [0, 1, 2, 15, 16, 17, 18, 19, 20]
    assert len(frames) * 1560 == int(f["window_tokens"])
    # selected layers: two sink frames plus the same six recent frames
    frames8 = O.sink_window_frames(18, 3, recent, int(f["selected_layer_sink_frames"]))
    assert frames8 == [0, 1, 15, 16, 17, 18, 19, 20] and len(frames8) == int(f["selected_layer_frames"])
    # while the recent part still reaches the sink, every frame so far is attended once
    assert O.sink_window_frames(0, 3, recent, sink) == [0, 1, 2]
    assert O.sink_window_frames(3, 3, recent, sink) == [0, 1, 2, 3, 4, 5]
    assert O.sink_window_frames(6, 3, recent, sink) == [0, 1, 2, 3, 4, 5, 6, 7, 8]
    assert O.sink_window_frames(9, 3, recent, sink) == [0, 1, 2, 6, 7, 8, 9, 10, 11]
    # the last chunk of a 30 s clip: positions far beyond the ring capacity
    n = int(f["long_video_latent_frames"])
    assert n == 3 * int(f["long_video_chunks"])
    assert O.sink_window_frames(n - 3, 3, recent, sink) == [0, 1, 2] + list(range(n - 6, n))


def test_sink_slots_never_collide_inside_a_window():
    for sink, C in ((3, 6), (2, 6), (3, 9), (0, 6)):
        for s in range(0, 150, 3):
            frames = O.sink_window_frames(s, 3, min(6, C), sink)
            slots = [O.sink_slot(p, sink, C) for p in frames]
            assert len(set(slots)) == len(slots)
            assert all(sl == p for sl, p in zip(slots, frames) if p < sink)
            assert all(sink <= sl < sink + C for sl, p in zip(slots, frames) if p >= sink)
    assert O.sink_slot(5, 0, 6) == 5 and O.sink_slot(13, 0, 6) == 1      # no sink: the plain ring


def test_zero_keys_mean_of_sink_and_recent_frames():
    T, Hn, Fc, sink, C = 8, 1, 3, 3, 6
    st = O.SinkRingState(1, sink, C, T, Hn)
    q = W.normal_bf16((3,), (1, Fc * T, Hn, 128))
    for p in range(21):
        sl = O.sink_slot(p, sink, C)
        st.cache_k[0, sl] = 0
        st.cache_v[0, sl] = O.f32_to_bf16_bits_rne(np.full((T, Hn, 128), float(p), np.float32))
    o = O.window_attn_sink(st, [18], 6, 3, q, Fc)          # {0,1,2} + {15..20}
    assert np.abs(o - 12.0).max() < 1e-12
    o = O.window_attn_sink(st, [18], 6, 2, q, Fc)          # {0,1} + {15..20}
    assert np.abs(o - 13.25).max() < 1e-12
    o = O.window_attn_sink(st, [18], 6, 0, q, Fc)          # recent only
    assert np.abs(o - 17.5).max() < 1e-12


def test_long_stream_sink_cache_equals_explicit_history():
    # 41 chunks of 3 frames (positions 0..122) through a 3 + 6 frame cache
    sh = W.Shape(batch=1, heads=2, chunk_frames=3, grid_h=2, grid_w=4, ring_frames=6)
    wl = W.Workload("soak", sh, seed=41, history_starts=((),), measured_starts=(0,), window_frames=(6,))
    st = O.SinkRingState(1, 3, 6, sh.tokens_per_frame, sh.heads)
    hist = O.ExplicitHistory(sh.tokens_per_frame)
    for c in range(41):
        s = 3 * c
        q, k, v = W.batch_qkv(wl, [s])
        cos, sin = O.rope_table(s, 3, 2, 4)
        q_out = O.rope_kv_append_sink(st, [s], q, k, v, cos, sin)
        hist.append(s, O.rope_rotate(k[0], cos, sin), v[0])
        if c in (0, 1, 2, 3, 7, 20, 40):
            for sink_attend in (3, 2):
                a = O.window_attn_sink(st, [s], 6, sink_attend, q_out, 3)
                b = O.explicit_frames_attn(hist, O.sink_window_frames(s, 3, 6, sink_attend), q_out[0])
                assert np.abs(a[0] - b).max() < 1e-12
    # the sink prefix still holds frames 0..2 untouched by the 38 later chunks
    for p in range(3):
        assert np.array_equal(st.cache_k[0, p], hist.k[p]) and np.array_equal(st.cache_v[0, p], hist.v[p])


def test_sink_zero_reduces_to_the_plain_ring():
    wl = W.WORKLOADS["cfg1_wrapped"]
    sh = wl.shape
    ring = O.RingState(1, sh.ring_frames, sh.tokens_per_frame, sh.heads)
    st = O.SinkRingState(1, 0, sh.ring_frames, sh.tokens_per_frame, sh.heads)
    q_out = None
    for s in list(wl.history_starts[0]) + [16]:
        q, k, v = W.batch_qkv(wl, [s])
        cos, sin = O.rope_table(s, 2, 8, 8)
        q_out = O.rope_kv_append(ring, [s], q, k, v, cos, sin)
        O.rope_kv_append_sink(st, [s], q, k, v, cos, sin)
    assert np.array_equal(ring.ring_k, st.cache_k) and np.array_equal(ring.ring_v, st.cache_v)
    a = O.window_attn(ring, [16], 6, q_out, 2)
    b = O.window_attn_sink(st, [16], 6, 0, q_out, 2)
    assert np.array_equal(a, b)
