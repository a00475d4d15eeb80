"""Pins for the oracle's window selection and attention (CPU only)."""

import numpy as np
import torch

import oracle as O
import workloads as W


def _f64(bits):
    return O.bf16_bits_to_f32(bits).astype(np.float64)


def _filled_ring(wl, extra=()):
    sh = wl.shape
    ring = O.RingState(sh.batch, sh.ring_frames, sh.tokens_per_frame, sh.heads)
    hist = O.ExplicitHistory(sh.tokens_per_frame)
    q_out = None
    for s in list(wl.history_starts[0]) + list(wl.measured_starts) + list(extra):
        q, k, v = W.batch_qkv(wl, [s])
        cos, sin = O.rope_table(s, sh.chunk_frames, sh.grid_h, sh.grid_w)
        q_out = O.rope_kv_append(ring, [s], q, k, v, cos, sin)
        hist.append(s, O.rope_rotate(k[0], cos, sin), v[0])
    return ring, hist, q_out


def test_bruteforce_equals_blocked_on_tiny():
    rng = np.random.default_rng(0)
    q = rng.standard_normal((5, 128))
    k = rng.standard_normal((37, 128))
    v = rng.standard_normal((37, 128))
    assert np.abs(O.attention_bruteforce(q, k, v) - O.attention_rows(q, k, v, block=2)).max() < 1e-12


def test_cfg1_ring_form_equals_explicit_form_and_bruteforce():
    wl = W.WORKLOADS["cfg1"]
    ring, hist, q_out = _filled_ring(wl)
    s = wl.measured_starts[0]
    k_bits, _ = O.gather_window_ring(ring, 0, s, 2, 6)
    assert k_bits.shape[0] == 384                       # 4 cached frames (256 keys) + the chunk (128)
    a = O.window_attn(ring, [s], 6, q_out, 2)
    b = O.explicit_window_attn(hist, s, 2, 6, q_out[0])
    assert np.abs(a[0] - b).max() < 1e-12
    rows = [0, 63, 64, 127]
    k_e, v_e = hist.window(s, 2, 6)
    bf = O.attention_bruteforce(_f64(q_out[0, rows, 1]), _f64(k_e[:, 1]), _f64(v_e[:, 1]))
    assert np.abs(a[0, rows, 1] - bf).max() < 1e-12


def test_wrapped_ring_form_equals_explicit_form():
    wl = W.WORKLOADS["cfg1_wrapped"]
    ring, hist, q_out = _filled_ring(wl)
    for wf in wl.window_frames:
        a = O.window_attn(ring, [16], wf, q_out, 2)
        b = O.explicit_window_attn(hist, 16, 2, wf, q_out[0])
        assert np.abs(a[0] - b).max() < 1e-12


def test_softmax_rows_sum_to_one_and_constant_v():
    rng = np.random.default_rng(1)
    q = rng.standard_normal((16, 128)) * 3
    k = rng.standard_normal((300, 128)) * 3
    v = np.zeros((300, 128))
    v[np.arange(300), np.arange(300) % 128] = 1.0       # every V row sums to 1
    o = O.attention_rows(q, k, v)
    assert np.abs(o.sum(axis=1) - 1.0).max() < 1e-12 and (o >= 0).all()
    o = O.attention_rows(q, k, np.full((300, 128), -2.5))
    assert np.abs(o + 2.5).max() < 1e-12


def test_zero_keys_give_mean_of_window_frames():
    # K = 0 -> uniform weights -> output = mean of V over the window; V[frame p] = p
    T, Hn, C, Fc = 8, 1, 6, 3
    ring = O.RingState(1, C, T, Hn)

    def put(p):
        ring.ring_k[0, p % C] = 0
        ring.ring_v[0, p % C] = O.f32_to_bf16_bits_rne(np.full((T, Hn, 128), float(p), np.float32))

    q = W.normal_bf16((1,), (1, Fc * T, Hn, 128))
    for p in range(0, 3):
        put(p)
    o = O.window_attn(ring, [0], 6, q, Fc)              # start-up: only frames 0..2 exist
    assert np.abs(o - 1.0).max() < 1e-12
    for p in range(3, 21):
        put(p)                                          # ring now holds frames 15..20, wrapped
    o = O.window_attn(ring, [18], 6, q, Fc)             # frames 15..20
    assert np.abs(o - 17.5).max() < 1e-12
    o = O.window_attn(ring, [18], 4, q, Fc)             # frames 17..20
    assert np.abs(o - 18.5).max() < 1e-12
    o = O.window_attn(ring, [18], 3, q, Fc)             # the chunk alone
    assert np.abs(o - 19.0).max() < 1e-12
    ring9 = O.RingState(1, 9, T, Hn)
    for p in range(0, 21):
        ring9.ring_k[0, p % 9] = 0
        ring9.ring_v[0, p % 9] = O.f32_to_bf16_bits_rne(np.full((T, Hn, 128), float(p), np.float32))
    o = O.window_attn(ring9, [18], 9, q, Fc)            # frames 12..20 -> 16.0
    assert np.abs(o - 16.0).max() < 1e-12


def test_dominant_key_and_permutation_invariance():
    rng = np.random.default_rng(4)
    q = rng.standard_normal((4, 128))
    k = rng.standard_normal((50, 128)) * 0.01
    v = rng.standard_normal((50, 128))
    k[17] = q[2] * 50.0                                  # key 17 dominates row 2
    o = O.attention_rows(q, k, v)
    assert np.abs(o[2] - v[17]).max() < 1e-9
    perm = rng.permutation(50)
    assert np.abs(O.attention_rows(q, k[perm], v[perm]) - o).max() < 1e-12


def test_full_window_matches_library_sdpa():
    wl = W.WORKLOADS["cfg1"]
    ring, hist, q_out = _filled_ring(wl)
    a = O.window_attn(ring, [4], 6, q_out, 2)           # [1, 128, 2, 128]
    k_e, v_e = hist.window(4, 2, 6)
    qt = torch.from_numpy(_f64(q_out[0])).permute(1, 0, 2)[None]     # [1, Hn, L, D]
    kt = torch.from_numpy(_f64(k_e)).permute(1, 0, 2)[None]
    vt = torch.from_numpy(_f64(v_e)).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt)  # default scale 1/sqrt(128)
    ref = ref[0].permute(1, 0, 2).numpy()
    assert np.abs(a[0] - ref).max() < 1e-10


def test_row_and_head_subsets_are_exact_slices():
    wl = W.WORKLOADS["cfg1"]
    ring, _, q_out = _filled_ring(wl)
    full = O.window_attn(ring, [4], 6, q_out, 2)
    rows = W.sample_rows(128, tile=32, per_tile=4)
    sub = O.window_attn(ring, [4], 6, q_out, 2, rows=rows, heads=[1])
    assert np.array_equal(sub[:, :, 0], full[:, rows, 1])


def test_sample_rows_covers_tiles_and_tail():
    rows = W.sample_rows(4680)
    assert rows[0] == 0 and 127 in rows and 128 in rows
    assert set(range(36 * 128, 4680)) <= set(rows.tolist())
    assert len(rows) == 36 * 8 + 72 and len(set(rows.tolist())) == len(rows)
