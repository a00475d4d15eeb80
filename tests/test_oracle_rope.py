"""Pins for the oracle's RoPE table, rotation and ring append (CPU only).

Each test fixes the oracle to something other than itself: a value the paper
prints, a closed form, an invariant, an independent library routine or the
textbook 1-D RoPE written with complex numbers."""

import math
import os

import numpy as np
import pytest
import torch

import oracle as O
import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_facts.txt")


def load_facts():
    facts = {}
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                k, v = (t.strip() for t in line.split("="))
                facts[k] = v
    return facts


# ----------------------------------------------------------------- paper facts
def test_paper_counts_match_workload_shapes():
    f = load_facts()
    sh = W.WORKLOADS["cfg2"].shape
    assert sh.grid_h == int(f["grid_h_480p"]) and sh.grid_w == int(f["grid_w_480p"])
    assert sh.tokens_per_frame == int(f["tokens_per_frame_480p"]) == 1560
    assert sh.chunk_frames == int(f["chunk_frames"])
    assert sh.heads == int(f["heads_1p3b"]) and sh.head_dim == int(f["head_dim"])
    assert O.N_PAIRS == int(f["pairs"])
    wl = W.WORKLOADS["cfg2"]
    assert wl.keys_attended(int(f["max_context_frames"])) == [int(f["max_context_tokens"])]
    assert int(f["window_frames"]) * sh.tokens_per_frame == int(f["window_tokens"])


def test_paper_position_example_chunk_at_6():
    f = load_facts()
    s = int(f["example_chunk_start"])
    want = [int(x) for x in f["example_temporal_positions"].split(",")]
    p_t, p_h, p_w = O.token_positions(s, 3, 30, 52)
    assert sorted(set(p_t.tolist())) == want
    # frame-major, then row, then column
    assert (p_t[:1560] == 6).all() and (p_t[1560:3120] == 7).all()
    assert p_h[0] == 0 and p_w[0] == 0 and p_w[1] == 1 and p_h[52] == 1 and p_w[52] == 0
    assert p_h.max() == 29 and p_w.max() == 51


def test_window_range_counts_the_chunk():
    f = load_facts()
    # steady state of the recent part: six most recent frames include the 3-frame chunk
    lo, hi = O.window_frames_range(18, 3, int(f["recent_frames_incl_chunk"]))
    assert (lo, hi) == (15, 21)
    assert O.window_frames_range(0, 3, 9) == (0, 3)      # start-up: clamped at frame 0
    assert O.window_frames_range(18, 3, 21) == (0, 21)   # all 21 frames of a 5 s clip


# ----------------------------------------------------------------- bf16 helpers
def test_bf16_conversions_match_torch():
    rng = np.random.default_rng(5)
    x = rng.standard_normal(200000).astype(np.float32) * np.float32(3.0)
    # exact ties and near-ties, signed zeros, tiny and huge values
    edge = np.array([1.00390625, 1.01171875, -1.00390625, 0.0, -0.0, 1e-40, 3.3e38, -3.3e38,
                     65280.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, np.inf, -np.inf], dtype=np.float32)
    x = np.concatenate([x, edge])
    ours = O.f32_to_bf16_bits_rne(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    back = O.bf16_bits_to_f32(ours)
    ref_back = torch.from_numpy(ref.view(np.int16)).view(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(back.view(np.uint32), ref_back.view(np.uint32))
    assert np.array_equal(W.f32_to_bf16_bits(x[:-2]), ours[:-2])


# ----------------------------------------------------------------------- table
def test_band_split_and_ladders():
    assert O.band_pairs((44, 42, 42)) == (22, 21, 21)
    omega, which = O.band_frequencies((44, 42, 42), 10000.0)
    assert which.tolist() == [0] * 22 + [1] * 21 + [2] * 21
    # first pair of every band has omega = 1; ladders restart per band and fall
    for j0 in (0, 22, 43):
        assert omega[j0] == 1.0
    assert math.isclose(omega[1], 10000.0 ** (-2 / 44), rel_tol=1e-15)
    assert math.isclose(omega[21], 10000.0 ** (-42 / 44), rel_tol=1e-15)
    assert math.isclose(omega[23], 10000.0 ** (-2 / 42), rel_tol=1e-15)
    assert math.isclose(omega[63], 10000.0 ** (-40 / 42), rel_tol=1e-15)
    assert (np.diff(omega[:22]) < 0).all() and (np.diff(omega[22:43]) < 0).all()
    with pytest.raises(ValueError):
        O.band_pairs((43, 43, 42))
    with pytest.raises(ValueError):
        O.band_pairs((44, 42, 40))


def test_table_closed_forms():
    cos, sin = O.rope_table(0, 2, 8, 8)
    assert cos.dtype == np.float32 and cos.shape == (128, 64)
    # token (0,0,0) at s=0: every angle is 0
    assert (cos[0] == 1.0).all() and (sin[0] == 0.0).all()
    # omega = 1 pairs hold cos/sin of the integer positions
    s0 = 7
    cos, sin = O.rope_table(s0, 2, 8, 8)
    p_t, p_h, p_w = O.token_positions(s0, 2, 8, 8)
    for n in (0, 1, 9, 63, 64, 127):
        assert cos[n, 0] == np.float32(math.cos(p_t[n])) and sin[n, 0] == np.float32(math.sin(p_t[n]))
        assert cos[n, 22] == np.float32(math.cos(p_h[n])) and sin[n, 22] == np.float32(math.sin(p_h[n]))
        assert cos[n, 43] == np.float32(math.cos(p_w[n])) and sin[n, 43] == np.float32(math.sin(p_w[n]))
    # a generic entry from its definition with scalar math
    n, j = 77, 30      # band h, local pair 8
    theta = p_h[n] * 10000.0 ** (-16 / 42)
    assert cos[n, j] == np.float32(math.cos(theta)) and sin[n, j] == np.float32(math.sin(theta))
    n, j = 100, 50     # band w, local pair 7
    theta = p_w[n] * 10000.0 ** (-14 / 42)
    assert cos[n, j] == np.float32(math.cos(theta)) and sin[n, j] == np.float32(math.sin(theta))
    # unit circle to float32 rounding
    assert np.abs(cos.astype(np.float64) ** 2 + sin.astype(np.float64) ** 2 - 1).max() < 2e-7


def test_table_temporal_shift_only_moves_band_t():
    c0, s0 = O.rope_table(0, 2, 8, 8)
    c9, s9 = O.rope_table(9, 2, 8, 8)
    assert np.array_equal(c0[:, 22:], c9[:, 22:]) and np.array_equal(s0[:, 22:], s9[:, 22:])
    assert not np.array_equal(c0[:, :22], c9[:, :22])


# -------------------------------------------------------------------- rotation
def test_rotation_sign_and_pairing():
    # (1, 0) in pair j turns into (cos, sin); (0, 1) into (-sin, cos): counter-clockwise,
    # interleaved pairs (x_2j, x_2j+1)
    cos, sin = O.rope_table(3, 1, 2, 2)
    L = 4
    x = np.zeros((L, 1, 128), dtype=np.float32)
    x[:, 0, 0::2] = 1.0
    y = O.bf16_bits_to_f32(O.rope_rotate(O.f32_to_bf16_bits_rne(x), cos, sin))
    assert np.array_equal(y[:, 0, 0::2], O.bf16_bits_to_f32(O.f32_to_bf16_bits_rne(cos)))
    assert np.array_equal(y[:, 0, 1::2], O.bf16_bits_to_f32(O.f32_to_bf16_bits_rne(sin)))
    x = np.zeros((L, 1, 128), dtype=np.float32)
    x[:, 0, 1::2] = 1.0
    y = O.bf16_bits_to_f32(O.rope_rotate(O.f32_to_bf16_bits_rne(x), cos, sin))
    assert np.array_equal(y[:, 0, 0::2], O.bf16_bits_to_f32(O.f32_to_bf16_bits_rne(-sin)))
    assert np.array_equal(y[:, 0, 1::2], O.bf16_bits_to_f32(O.f32_to_bf16_bits_rne(cos)))


def test_origin_token_is_returned_bit_identical():
    cos, sin = O.rope_table(0, 2, 8, 8)
    x = W.normal_bf16((11,), (128, 2, 128))
    y = O.rope_rotate(x, cos, sin)
    assert np.array_equal(y[0], x[0])
    assert not np.array_equal(y[1], x[1])


def test_rotation_reduces_to_textbook_1d_rope():
    # a 1x1 grid has p_h = p_w = 0, so bands h and w are the identity and band t is
    # ordinary 1-D RoPE over 44 dims: (x_e + i x_o) * exp(i p theta_i), theta_i = 1e4^(-2i/44)
    s, Fc = 5, 4
    theta = O.rope_angles(s, Fc, 1, 1)
    rng = np.random.default_rng(2)
    x = rng.standard_normal((Fc, 3, 128))
    y = O.rope_rotate_f64(x, theta)
    assert np.array_equal(y[..., 44:], x[..., 44:])
    pos = np.arange(s, s + Fc, dtype=np.float64)
    inv_freq = 1.0 / (10000.0 ** (np.arange(0, 44, 2) / 44.0))
    z = (x[..., 0:44:2] + 1j * x[..., 1:44:2]) * np.exp(1j * pos[:, None, None] * inv_freq)
    assert np.abs(y[..., 0:44:2] - z.real).max() < 1e-13
    assert np.abs(y[..., 1:44:2] - z.imag).max() < 1e-13


def test_rotation_norms_inverse_and_relative_position():
    rng = np.random.default_rng(3)
    Fc, Gh, Gw = 2, 4, 5
    x = rng.standard_normal((Fc * Gh * Gw, 2, 128))
    th = O.rope_angles(4, Fc, Gh, Gw)
    y = O.rope_rotate_f64(x, th)
    # pair norms and vector norms are preserved; rotating back restores x
    n_in = x[..., 0::2] ** 2 + x[..., 1::2] ** 2
    n_out = y[..., 0::2] ** 2 + y[..., 1::2] ** 2
    assert np.abs(n_in - n_out).max() < 1e-12
    assert np.abs(O.rope_rotate_f64(y, -th) - x).max() < 1e-12
    # q.k after rotation depends only on the position offset: shift both start frames
    q = rng.standard_normal((Fc * Gh * Gw, 1, 128))
    k = rng.standard_normal((Fc * Gh * Gw, 1, 128))

    def scores(sq, sk):
        qr = O.rope_rotate_f64(q, O.rope_angles(sq, Fc, Gh, Gw))[:, 0]
        kr = O.rope_rotate_f64(k, O.rope_angles(sk, Fc, Gh, Gw))[:, 0]
        return qr @ kr.T

    base = scores(6, 2)
    assert np.abs(scores(46, 42) - base).max() < 1e-11
    assert np.abs(scores(7, 2) - base).max() > 1e-3          # a different offset does change them
    # and on the spatial axes: rotate with all rows/cols shifted by a common amount
    omega, which = O.band_frequencies()

    def scores_shift(dh, dw):
        p_t, p_h, p_w = O.token_positions(0, Fc, Gh, Gw)
        pos = np.stack([p_t, p_h + dh, p_w + dw], 1).astype(np.float64)
        th2 = pos[:, which] * omega
        return O.rope_rotate_f64(q, th2)[:, 0] @ O.rope_rotate_f64(k, th2)[:, 0].T

    assert np.abs(scores_shift(0, 0) - scores_shift(11, 23)).max() < 1e-11


def test_bf16_rotation_matches_torch_float32_ops_and_keeps_norms():
    # the same six float32 operations issued through an independent library (torch CPU)
    wl = W.WORKLOADS["cfg1"]
    q, _, _ = W.chunk_qkv(wl, 0, 4)
    cos, sin = O.rope_table(4, 2, 8, 8)
    ours = O.rope_rotate(q, cos, sin)
    xt = torch.from_numpy(q.view(np.int16)).view(torch.bfloat16).to(torch.float32)
    c = torch.from_numpy(cos)[:, None, :]
    s = torch.from_numpy(sin)[:, None, :]
    xe, xo = xt[..., 0::2], xt[..., 1::2]
    ye = torch.mul(xe, c) - torch.mul(xo, s)
    yo = torch.mul(xe, s) + torch.mul(xo, c)
    yt = torch.stack([ye, yo], dim=-1).reshape(xt.shape).to(torch.bfloat16)
    assert np.array_equal(ours, yt.view(torch.int16).numpy().view(np.uint16))
    # norms preserved to bf16 rounding
    n_in = np.linalg.norm(O.bf16_bits_to_f32(q).astype(np.float64), axis=-1)
    n_out = np.linalg.norm(O.bf16_bits_to_f32(ours).astype(np.float64), axis=-1)
    assert np.abs(n_out / n_in - 1).max() < 2 ** -8


def test_rotation_is_not_fma_contracted():
    # pairs where fl(fl(a*c) - fl(b*s)) and the fused form round to different bf16 values
    # (about 20 per million) must follow the unfused order
    rng = np.random.default_rng(9)
    n = 2_000_000
    xe = O.bf16_bits_to_f32(O.f32_to_bf16_bits_rne(rng.standard_normal(n).astype(np.float32)))
    xo = O.bf16_bits_to_f32(O.f32_to_bf16_bits_rne(rng.standard_normal(n).astype(np.float32)))
    th = rng.uniform(0, 6.28, n)
    c, s = np.cos(th).astype(np.float32), np.sin(th).astype(np.float32)
    unfused = ((xe * c).astype(np.float32) - (xo * s).astype(np.float32)).astype(np.float32)
    fused = (xe.astype(np.float64) * c.astype(np.float64)
             - (xo * s).astype(np.float32).astype(np.float64)).astype(np.float32)
    differ = np.nonzero(O.f32_to_bf16_bits_rne(unfused) != O.f32_to_bf16_bits_rne(fused))[0]
    assert len(differ) >= 5
    m = min(len(differ), 32)
    x = np.zeros((m, 1, 128), dtype=np.float32)
    ct = np.ones((m, 64), dtype=np.float32)
    st = np.zeros((m, 64), dtype=np.float32)
    x[:, 0, 0], x[:, 0, 1] = xe[differ[:m]], xo[differ[:m]]
    ct[:, 0], st[:, 0] = c[differ[:m]], s[differ[:m]]
    y = O.rope_rotate(O.f32_to_bf16_bits_rne(x), ct, st)
    assert np.array_equal(y[:, 0, 0], O.f32_to_bf16_bits_rne(unfused[differ[:m]]))


# ---------------------------------------------------------------------- append
def _stream(wl, ring, hist, starts, tag=0):
    sh = wl.shape
    for s in starts:
        q, k, v = W.batch_qkv(wl, [s] * sh.batch, tag)
        cos, sin = O.rope_table(s, sh.chunk_frames, sh.grid_h, sh.grid_w)
        O.rope_kv_append(ring, [s] * sh.batch, q, k, v, cos, sin)
        if hist is not None:
            hist.append(s, O.rope_rotate(k[0], cos, sin), v[0])


def test_append_slots_sentinels_and_v_bit_copy():
    wl = W.WORKLOADS["cfg1"]
    sh = wl.shape
    ring = O.RingState(1, sh.ring_frames, sh.tokens_per_frame, sh.heads)
    q, k, v = W.batch_qkv(wl, [8])                      # frames 8, 9 -> slots 2, 3 of a 6-frame ring
    cos, sin = O.rope_table(8, 2, 8, 8)
    q_out = O.rope_kv_append(ring, [8], q, k, v, cos, sin)
    assert np.array_equal(ring.ring_v[0, 2], v[0, :64]) and np.array_equal(ring.ring_v[0, 3], v[0, 64:])
    assert np.array_equal(ring.ring_k[0, 2], O.rope_rotate(k[0], cos, sin)[:64])
    for slot in (0, 1, 4, 5):
        assert (ring.ring_k[0, slot] == O.unstep_oracle.SENTINEL).all()
        assert (ring.ring_v[0, slot] == O.unstep_oracle.SENTINEL).all()
    assert np.array_equal(q_out, O.rope_rotate(q, cos, sin))


def test_append_overwrite_is_idempotent():
    wl = W.WORKLOADS["cfg1"]
    sh = wl.shape
    ring_ab = O.RingState(1, sh.ring_frames, sh.tokens_per_frame, sh.heads)
    ring_b = O.RingState(1, sh.ring_frames, sh.tokens_per_frame, sh.heads)
    cos, sin = O.rope_table(4, 2, 8, 8)
    qa, ka, va = W.batch_qkv(wl, [4], tag=0)
    qb, kb, vb = W.batch_qkv(wl, [4], tag=1)
    assert not np.array_equal(ka, kb)
    O.rope_kv_append(ring_ab, [4], qa, ka, va, cos, sin)
    O.rope_kv_append(ring_ab, [4], qb, kb, vb, cos, sin)
    O.rope_kv_append(ring_b, [4], qb, kb, vb, cos, sin)
    assert np.array_equal(ring_ab.ring_k, ring_b.ring_k) and np.array_equal(ring_ab.ring_v, ring_b.ring_v)


def test_ring_equals_explicit_history_after_wraps():
    wl = W.WORKLOADS["cfg1_wrapped"]
    sh = wl.shape
    ring = O.RingState(1, sh.ring_frames, sh.tokens_per_frame, sh.heads)
    hist = O.ExplicitHistory(sh.tokens_per_frame)
    _stream(wl, ring, hist, list(wl.history_starts[0]) + [16])
    for wf in (2, 4, 6):
        k_r, v_r = O.gather_window_ring(ring, 0, 16, 2, wf)
        k_e, v_e = hist.window(16, 2, wf)
        assert k_r.shape[0] == wf * 64
        assert np.array_equal(k_r, k_e) and np.array_equal(v_r, v_e)
