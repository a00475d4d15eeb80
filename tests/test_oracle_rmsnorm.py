"""Pins for the oracle's q/k RMS normalisation (CPU only)."""

import numpy as np
import torch

import oracle as O
import workloads as W


def _x(shape, seed, scale=1.0):
    return W.normal_bf16((seed,), shape, scale=scale)


def test_matches_library_rms_norm():
    x = _x((37, 12, 128), 1)
    g = (1.0 + 0.1 * np.random.default_rng(2).standard_normal(1536)).astype(np.float32)
    ours = O.bf16_bits_to_f32(O.rmsnorm_tokens(x, g, 1e-6)).astype(np.float64)
    xt = torch.from_numpy(O.bf16_bits_to_f32(x).astype(np.float64)).reshape(37, 1536)
    ref = torch.nn.functional.rms_norm(xt, (1536,), torch.from_numpy(g.astype(np.float64)), 1e-6)
    ref = ref.reshape(37, 12, 128).numpy()
    # float32 arithmetic + one bf16 rounding against the float64 library result
    assert np.abs(ours - ref).max() <= 2.0 ** -8 * np.abs(ref).max()
    assert np.abs(ours / np.where(ref == 0, 1, ref) - 1)[np.abs(ref) > 0.1].max() < 2.0 ** -7.5


def test_unit_gain_gives_unit_rms_and_scale_invariance():
    x = _x((16, 12, 128), 3)
    ones = np.ones(1536, np.float32)
    y = O.bf16_bits_to_f32(O.rmsnorm_tokens(x, ones, 0.0)).astype(np.float64).reshape(16, -1)
    assert np.abs(np.sqrt((y ** 2).mean(axis=1)) - 1).max() < 3e-3
    x4 = _x((16, 12, 128), 3, scale=4.0)          # the same tokens times 4 (exact in bf16)
    assert np.array_equal(O.rmsnorm_tokens(x4, ones, 0.0), O.rmsnorm_tokens(x, ones, 0.0))
    # the gain multiplies channel-wise
    g = np.ones(1536, np.float32)
    g[5] = 2.0
    y2 = O.bf16_bits_to_f32(O.rmsnorm_tokens(x, g, 0.0)).reshape(16, -1)
    y1 = O.bf16_bits_to_f32(O.rmsnorm_tokens(x, ones, 0.0)).reshape(16, -1)
    assert np.array_equal(y2[:, 5], 2 * y1[:, 5]) and np.array_equal(np.delete(y2, 5, 1), np.delete(y1, 5, 1))


def test_eps_and_constant_vector_closed_form():
    # a constant vector of value a normalises to a / sqrt(a^2 + eps)
    a, eps = 0.5, 0.75
    x = O.f32_to_bf16_bits_rne(np.full((1, 2, 128), a, np.float32))
    y = O.bf16_bits_to_f32(O.rmsnorm_tokens(x, np.ones(256, np.float32), eps))
    want = O.bf16_bits_to_f32(O.f32_to_bf16_bits_rne(np.array([a / np.sqrt(a * a + eps)], np.float32)))[0]
    assert (y == want).all()


def test_fused_append_is_norm_then_append():
    wl = W.WORKLOADS["cfg1"]
    sh = wl.shape
    q, k, v = W.batch_qkv(wl, [4])
    gq = (1 + 0.05 * np.arange(256) / 256).astype(np.float32)
    gk = (1 - 0.05 * np.arange(256) / 256).astype(np.float32)
    cos, sin = O.rope_table(4, 2, 8, 8)
    a = O.RingState(1, sh.ring_frames, sh.tokens_per_frame, sh.heads)
    b = O.RingState(1, sh.ring_frames, sh.tokens_per_frame, sh.heads)
    qa = O.rmsnorm_rope_kv_append(a, [4], q, k, v, gq, gk, 1e-6, cos, sin)
    qb = O.rope_kv_append(b, [4], O.rmsnorm_tokens(q, gq, 1e-6), O.rmsnorm_tokens(k, gk, 1e-6), v, cos, sin)
    assert np.array_equal(qa, qb) and np.array_equal(a.ring_k, b.ring_k) and np.array_equal(a.ring_v, b.ring_v)
    assert np.array_equal(a.ring_v[0, 4], v[0, :64])       # V is not normalised
