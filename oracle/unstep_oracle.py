"""Plain CPU definition of the UnStep per-layer chunk-attention step.

TEST INFRASTRUCTURE ONLY -- never on the product path.  numpy, fp64 for
everything the paper does not pin to a lower precision.  No blocking, fusion
or reordering beyond what the definitions state, so every function can be
checked against the paper by eye.  Shares nothing with the CUDA library.

What the path computes (paper: appendix "Diffusion transformer runtime" and
appendix "KV attention window"):

  R1  token positions of a chunk: frame, row, column; the temporal position is
      the absolute latent-frame index (a chunk starting at 6 uses 6, 7, 8).
  R2  a float32 cos/sin table, one coefficient vector (64 pairs) per token,
      shared by all heads, keyed by (starting latent frame, grid size).
  R3  the rotation of one coordinate pair (x_2j, x_2j+1), bf16 in, float32
      arithmetic, bf16 out:  y_e = x_e*cos - x_o*sin ; y_o = x_e*sin + x_o*cos.
  R4  the write of the rotated keys and the raw values of the chunk into the
      per-layer KV cache; repeated calls for the same chunk overwrite.
  A1  the key set: the `window_frames` most recent latent frames, the current
      chunk included, clamped at frame 0.
  A2  softmax(q k^T / sqrt(128)) v over that key set, no mask.

Readings where the paper is silent (each is listed with its reason in the
design notes): band split 44/42/42 dims ordered t|h|w along the pair index,
each band with its own ladder base**(-2i/d_band); spatial positions start at
0; token order frame-major, then row, then column; fp64 angle and trig rounded
once to float32; the rotation is 4 multiplies, 1 subtract, 1 add, each rounded
to float32 (no fused multiply-add), then round-to-nearest-even to bf16; the
cache is a ring with slot = frame mod capacity; softmax scale 1/sqrt(128).

Every function here is pinned by tests/test_oracle_*.py (closed forms,
invariants, brute force, the textbook 1-D RoPE special case, a library SDPA
cross-check, and the counts and the position example the paper prints).
"""

from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

HEAD_DIM = 128
N_PAIRS = HEAD_DIM // 2
SENTINEL = np.uint16(0x7FC1)  # a NaN pattern no append ever produces from finite data


# ---------------------------------------------------------------------------
# bf16 <-> float32 (bit-level; bf16 tensors are carried as uint16 arrays)
# ---------------------------------------------------------------------------

def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def f32_to_bf16_bits_rne(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 with round-to-nearest-even (the bf16 store of R3)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    is_nan = (u & np.uint64(0x7FFFFFFF)) > np.uint64(0x7F800000)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = (u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)
    r = np.where(is_nan, (u >> np.uint64(16)) | np.uint64(0x0040), r)
    return r.astype(np.uint16)


# ---------------------------------------------------------------------------
# R1 / R2: positions and the coefficient table
# ---------------------------------------------------------------------------

def band_pairs(bands=(44, 42, 42)):
    """Pairs per band (t, h, w); dims must be even and sum to the head dim."""
    bt, bh, bw = (int(b) for b in bands)
    if bt % 2 or bh % 2 or bw % 2 or bt + bh + bw != HEAD_DIM or min(bt, bh, bw) <= 0:
        raise ValueError("bands must be positive, even and sum to 128")
    return bt // 2, bh // 2, bw // 2


def band_frequencies(bands=(44, 42, 42), base=10000.0):
    """omega[j] for the 64 pairs: band b, local pair i -> base**(-2i/d_b).

    Returns (omega[64] float64, band_of_pair[64] in {0,1,2})."""
    omega = np.empty(N_PAIRS, dtype=np.float64)
    which = np.empty(N_PAIRS, dtype=np.int64)
    j = 0
    for b, d_b in enumerate(int(x) for x in bands):
        for i in range(d_b // 2):
            omega[j] = float(base) ** (-(2.0 * i) / d_b)
            which[j] = b
            j += 1
    assert j == N_PAIRS
    return omega, which


def token_positions(start_frame: int, chunk_frames: int, grid_h: int, grid_w: int):
    """(p_t, p_h, p_w) for the L = Fc*Gh*Gw tokens of a chunk, token
    n = (f*Gh + r)*Gw + c  ->  (start_frame + f, r, c)."""
    f, r, c = np.meshgrid(np.arange(chunk_frames), np.arange(grid_h), np.arange(grid_w),
                          indexing="ij")
    return ((start_frame + f).reshape(-1).astype(np.int64),
            r.reshape(-1).astype(np.int64), c.reshape(-1).astype(np.int64))


def rope_angles(start_frame, chunk_frames, grid_h, grid_w, bands=(44, 42, 42), base=10000.0):
    """theta[n, j] in float64 = position of token n in pair j's band times omega[j]."""
    omega, which = band_frequencies(bands, base)
    p_t, p_h, p_w = token_positions(start_frame, chunk_frames, grid_h, grid_w)
    pos = np.stack([p_t, p_h, p_w], axis=1).astype(np.float64)      # [L, 3]
    return pos[:, which] * omega[None, :]                            # [L, 64]


def rope_table(start_frame, chunk_frames, grid_h, grid_w, bands=(44, 42, 42), base=10000.0):
    """The cached table of R2: (cos, sin), float32 [L, 64], one rounding from fp64."""
    theta = rope_angles(start_frame, chunk_frames, grid_h, grid_w, bands, base)
    return (np.ascontiguousarray(np.cos(theta), dtype=np.float32),
            np.ascontiguousarray(np.sin(theta), dtype=np.float32))


# ---------------------------------------------------------------------------
# R3: the rotation
# ---------------------------------------------------------------------------

def rope_rotate(x_bits: np.ndarray, cos: np.ndarray, sin: np.ndarray) -> np.ndarray:
    """Rotate bf16 x[..., L, Hn, 128] (uint16 bits) by the float32 table
    cos/sin[..., L, 64] (a leading stream axis on the table is optional).

    Every operation is a single float32 operation rounded to nearest; numpy
    never contracts a multiply and an add into one."""
    x = bf16_bits_to_f32(x_bits)
    xe = x[..., 0::2]
    xo = x[..., 1::2]
    c = np.asarray(cos, dtype=np.float32)[..., :, None, :]
    s = np.asarray(sin, dtype=np.float32)[..., :, None, :]
    a = (xe * c).astype(np.float32)
    b = (xo * s).astype(np.float32)
    ye = (a - b).astype(np.float32)
    a2 = (xe * s).astype(np.float32)
    b2 = (xo * c).astype(np.float32)
    yo = (a2 + b2).astype(np.float32)
    y = np.empty(x.shape, dtype=np.float32)
    y[..., 0::2] = ye
    y[..., 1::2] = yo
    return f32_to_bf16_bits_rne(y)


def rope_rotate_f64(x: np.ndarray, theta: np.ndarray) -> np.ndarray:
    """The same rotation in exact-angle float64 (x[..., L, Hn, 128], theta[L, 64]);
    used only to state the invariants of the rotation without rounding noise."""
    x = np.asarray(x, dtype=np.float64)
    c = np.cos(theta)[:, None, :]
    s = np.sin(theta)[:, None, :]
    y = np.empty_like(x)
    y[..., 0::2] = x[..., 0::2] * c - x[..., 1::2] * s
    y[..., 1::2] = x[..., 0::2] * s + x[..., 1::2] * c
    return y


# ---------------------------------------------------------------------------
# R4: append into the ring
# ---------------------------------------------------------------------------

@dataclass
class RingState:
    """Per-layer KV ring: bf16 bits [B, C, T, Hn, 128]; frame p lives in slot p % C."""
    batch: int
    ring_frames: int
    tokens_per_frame: int
    heads: int
    ring_k: np.ndarray = field(init=False)
    ring_v: np.ndarray = field(init=False)

    def __post_init__(self):
        shape = (self.batch, self.ring_frames, self.tokens_per_frame, self.heads, HEAD_DIM)
        self.ring_k = np.full(shape, SENTINEL, dtype=np.uint16)
        self.ring_v = np.full(shape, SENTINEL, dtype=np.uint16)


def rope_kv_append(ring: RingState, start_frames, q_bits, k_bits, v_bits, cos, sin):
    """R3 + R4 for one chunk of every stream.

    q/k/v_bits: uint16 [B, L, Hn, 128]; cos/sin: float32 [L, 64] (shared) or
    [B, L, 64].  Returns q_out bits; ring_k/ring_v are updated in place.
    Calling again with the same start frame overwrites the same slots."""
    B, L, Hn, D = q_bits.shape
    T = ring.tokens_per_frame
    assert D == HEAD_DIM and L % T == 0 and B == ring.batch and Hn == ring.heads
    Fc = L // T
    q_out = rope_rotate(q_bits, cos, sin)
    k_rot = rope_rotate(k_bits, cos, sin)
    for b in range(B):
        s = int(start_frames[b])
        assert s >= 0
        for f in range(Fc):
            slot = (s + f) % ring.ring_frames
            ring.ring_k[b, slot] = k_rot[b, f * T:(f + 1) * T]
            ring.ring_v[b, slot] = v_bits[b, f * T:(f + 1) * T]
    return q_out


# ---------------------------------------------------------------------------
# A1 / A2: the key set and the attention itself
# ---------------------------------------------------------------------------

def window_frames_range(start_frame: int, chunk_frames: int, window_frames: int):
    """Half-open range of absolute frames attended: the window counts the chunk."""
    hi = start_frame + chunk_frames
    return max(0, hi - window_frames), hi


def gather_window_ring(ring: RingState, b: int, start_frame: int, chunk_frames: int,
                       window_frames: int):
    """Keys and values (bf16 bits, [S, Hn, 128]) of stream b's window, read
    through slot = frame % C, in order of absolute frame."""
    lo, hi = window_frames_range(start_frame, chunk_frames, window_frames)
    slots = [p % ring.ring_frames for p in range(lo, hi)]
    k = np.concatenate([ring.ring_k[b, s] for s in slots], axis=0)
    v = np.concatenate([ring.ring_v[b, s] for s in slots], axis=0)
    return k, v


def attention_rows(q: np.ndarray, k: np.ndarray, v: np.ndarray, block: int = 512) -> np.ndarray:
    """softmax(q k^T / sqrt(d)) v in float64 for q[n, d], k[S, d], v[S, d].
    Query rows are independent; `block` only bounds the score matrix held."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    scale = 1.0 / math.sqrt(q.shape[-1])
    out = np.empty((q.shape[0], v.shape[1]), dtype=np.float64)
    for r0 in range(0, q.shape[0], block):
        z = (q[r0:r0 + block] @ k.T) * scale
        w = np.exp(z - z.max(axis=1, keepdims=True))
        out[r0:r0 + block] = (w @ v) / w.sum(axis=1, keepdims=True)
    return out


def attention_bruteforce(q: np.ndarray, k: np.ndarray, v: np.ndarray) -> np.ndarray:
    """The definition as scalar loops (tiny inputs only)."""
    n, d = q.shape
    S = k.shape[0]
    scale = 1.0 / math.sqrt(d)
    out = np.zeros((n, v.shape[1]), dtype=np.float64)
    for i in range(n):
        z = [scale * sum(float(q[i, t]) * float(k[m, t]) for t in range(d)) for m in range(S)]
        zmax = max(z)
        w = [math.exp(zm - zmax) for zm in z]
        wsum = sum(w)
        for m in range(S):
            out[i] += (w[m] / wsum) * v[m].astype(np.float64)
    return out


def window_attn(ring: RingState, start_frames, window_frames: int, q_rot_bits: np.ndarray,
                chunk_frames: int, rows=None, heads=None) -> np.ndarray:
    """Ring form of A1+A2.  q_rot_bits: uint16 [B, L, Hn, 128] (the q_out of the
    append).  Returns float64 [B, len(rows) or L, len(heads) or Hn, 128]."""
    B, L, Hn, D = q_rot_bits.shape
    rows = np.arange(L) if rows is None else np.asarray(rows, dtype=np.int64)
    heads = list(range(Hn)) if heads is None else list(heads)
    out = np.empty((B, len(rows), len(heads), D), dtype=np.float64)
    for b in range(B):
        k_bits, v_bits = gather_window_ring(ring, b, int(start_frames[b]), chunk_frames,
                                            window_frames)
        for hi_, h in enumerate(heads):
            q = bf16_bits_to_f32(q_rot_bits[b, rows, h]).astype(np.float64)
            k = bf16_bits_to_f32(k_bits[:, h]).astype(np.float64)
            v = bf16_bits_to_f32(v_bits[:, h]).astype(np.float64)
            out[b, :, hi_] = attention_rows(q, k, v)
    return out


class ExplicitHistory:
    """Unbounded linear history of one stream: frame p -> (K bits, V bits) [T, Hn, 128].
    The 'explicit concatenation' form the ring must agree with."""

    def __init__(self, tokens_per_frame: int):
        self.T = tokens_per_frame
        self.k = {}
        self.v = {}

    def append(self, start_frame: int, k_rot_bits: np.ndarray, v_bits: np.ndarray):
        L = k_rot_bits.shape[0]
        assert L % self.T == 0
        for f in range(L // self.T):
            self.k[start_frame + f] = k_rot_bits[f * self.T:(f + 1) * self.T].copy()
            self.v[start_frame + f] = v_bits[f * self.T:(f + 1) * self.T].copy()

    def window(self, start_frame, chunk_frames, window_frames):
        lo, hi = window_frames_range(start_frame, chunk_frames, window_frames)
        k = np.concatenate([self.k[p] for p in range(lo, hi)], axis=0)
        v = np.concatenate([self.v[p] for p in range(lo, hi)], axis=0)
        return k, v


def explicit_window_attn(history: ExplicitHistory, start_frame: int, chunk_frames: int,
                         window_frames: int, q_rot_bits: np.ndarray, rows=None,
                         heads=None) -> np.ndarray:
    """Explicit-slice form of A1+A2 for one stream; q_rot_bits uint16 [L, Hn, 128]."""
    L, Hn, D = q_rot_bits.shape
    rows = np.arange(L) if rows is None else np.asarray(rows, dtype=np.int64)
    heads = list(range(Hn)) if heads is None else list(heads)
    k_bits, v_bits = history.window(start_frame, chunk_frames, window_frames)
    out = np.empty((len(rows), len(heads), D), dtype=np.float64)
    for hi_, h in enumerate(heads):
        q = bf16_bits_to_f32(q_rot_bits[rows, h]).astype(np.float64)
        k = bf16_bits_to_f32(k_bits[:, h]).astype(np.float64)
        v = bf16_bits_to_f32(v_bits[:, h]).astype(np.float64)
        out[:, hi_] = attention_rows(q, k, v)
    return out


# ---------------------------------------------------------------------------
# Sink + sliding window (Sec. "Limited KV attention window", appendix "KV attention
# window"): the first `sink` latent frames are never evicted, the ring keeps the most
# recent frames; once the cache is full a chunk attends the sink frames plus the
# `recent` most recent frames, the current chunk included.  Before that (the recent
# part still reaches back to the sink) it attends every frame so far.
# ---------------------------------------------------------------------------

def sink_slot(frame: int, sink_frames: int, ring_frames: int) -> int:
    """Cache slot of an absolute frame: sink frames sit in a prefix that is never
    overwritten, later frames in a ring behind it."""
    if frame < sink_frames:
        return frame
    return sink_frames + (frame - sink_frames) % ring_frames


def sink_window_frames(start_frame: int, chunk_frames: int, recent_frames: int, sink_attend: int):
    """Absolute frames attended, in increasing order."""
    hi = start_frame + chunk_frames
    lo = max(0, hi - recent_frames)
    return list(range(0, min(sink_attend, lo))) + list(range(lo, hi))


@dataclass
class SinkRingState:
    """Per-layer KV cache with a sink prefix: bf16 bits [B, sink + C, T, Hn, 128]."""
    batch: int
    sink_frames: int
    ring_frames: int
    tokens_per_frame: int
    heads: int
    cache_k: np.ndarray = field(init=False)
    cache_v: np.ndarray = field(init=False)

    def __post_init__(self):
        shape = (self.batch, self.sink_frames + self.ring_frames, self.tokens_per_frame, self.heads,
                 HEAD_DIM)
        self.cache_k = np.full(shape, SENTINEL, dtype=np.uint16)
        self.cache_v = np.full(shape, SENTINEL, dtype=np.uint16)


def rope_kv_append_sink(state: SinkRingState, start_frames, q_bits, k_bits, v_bits, cos, sin):
    """R3 + R4 with the sink prefix: same rotation, slot = sink_slot(frame)."""
    B, L, Hn, D = q_bits.shape
    T = state.tokens_per_frame
    assert D == HEAD_DIM and L % T == 0 and B == state.batch and Hn == state.heads
    q_out = rope_rotate(q_bits, cos, sin)
    k_rot = rope_rotate(k_bits, cos, sin)
    for b in range(B):
        s = int(start_frames[b])
        for f in range(L // T):
            slot = sink_slot(s + f, state.sink_frames, state.ring_frames)
            state.cache_k[b, slot] = k_rot[b, f * T:(f + 1) * T]
            state.cache_v[b, slot] = v_bits[b, f * T:(f + 1) * T]
    return q_out


def window_attn_sink(state: SinkRingState, start_frames, recent_frames: int, sink_attend: int,
                     q_rot_bits: np.ndarray, chunk_frames: int, rows=None, heads=None) -> np.ndarray:
    """A1 + A2 with the key set sink ∪ recent, read through sink_slot."""
    B, L, Hn, D = q_rot_bits.shape
    assert sink_attend <= state.sink_frames
    rows = np.arange(L) if rows is None else np.asarray(rows, dtype=np.int64)
    heads = list(range(Hn)) if heads is None else list(heads)
    out = np.empty((B, len(rows), len(heads), D), dtype=np.float64)
    for b in range(B):
        frames = sink_window_frames(int(start_frames[b]), chunk_frames, recent_frames, sink_attend)
        slots = [sink_slot(p, state.sink_frames, state.ring_frames) for p in frames]
        k_bits = np.concatenate([state.cache_k[b, s] for s in slots], axis=0)
        v_bits = np.concatenate([state.cache_v[b, s] for s in slots], axis=0)
        for hi_, h in enumerate(heads):
            q = bf16_bits_to_f32(q_rot_bits[b, rows, h]).astype(np.float64)
            k = bf16_bits_to_f32(k_bits[:, h]).astype(np.float64)
            v = bf16_bits_to_f32(v_bits[:, h]).astype(np.float64)
            out[b, :, hi_] = attention_rows(q, k, v)
    return out


def explicit_frames_attn(history: ExplicitHistory, frames, q_rot_bits: np.ndarray, rows=None,
                         heads=None) -> np.ndarray:
    """Attention of q_rot_bits [L, Hn, 128] over an explicit list of frames of the history."""
    L, Hn, D = q_rot_bits.shape
    rows = np.arange(L) if rows is None else np.asarray(rows, dtype=np.int64)
    heads = list(range(Hn)) if heads is None else list(heads)
    k_bits = np.concatenate([history.k[p] for p in frames], axis=0)
    v_bits = np.concatenate([history.v[p] for p in frames], axis=0)
    out = np.empty((len(rows), len(heads), D), dtype=np.float64)
    for hi_, h in enumerate(heads):
        q = bf16_bits_to_f32(q_rot_bits[rows, h]).astype(np.float64)
        k = bf16_bits_to_f32(k_bits[:, h]).astype(np.float64)
        v = bf16_bits_to_f32(v_bits[:, h]).astype(np.float64)
        out[:, hi_] = attention_rows(q, k, v)
    return out


# ---------------------------------------------------------------------------
# RMS normalisation of q and k in front of the rotation (appendix "Diffusion transformer
# runtime": q and k pass through the projection and an RMS norm before the head split).  The
# paper gives no formula; this is the textbook RMSNorm over the whole token vector (all heads,
# Hn*128 wide) with a learned per-channel gain:
#     y = x / sqrt(mean(x^2) + eps) * g
# Readings: the mean of squares is accumulated in float64 (so that it does not depend on the
# order of summation) and rounded to float32; sqrt, reciprocal and the two products are single
# float32 operations; the result is rounded to bf16 (the tensor the rotation loads is bf16).
# ---------------------------------------------------------------------------

def rmsnorm_tokens(x_bits: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x_bits: bf16 bits [..., Hn, 128]; gain: float32 [Hn*128].  Returns bf16 bits."""
    x = bf16_bits_to_f32(x_bits)
    lead = x.shape[:-2]
    width = x.shape[-2] * x.shape[-1]
    flat = x.reshape(lead + (width,))
    ms = (flat.astype(np.float64) ** 2).sum(axis=-1) / np.float64(width)
    ms32 = ms.astype(np.float32)
    r = (np.float32(1.0) / np.sqrt((ms32 + np.float32(eps)).astype(np.float32))).astype(np.float32)
    y = ((flat * r[..., None]).astype(np.float32) * np.asarray(gain, dtype=np.float32)).astype(np.float32)
    return f32_to_bf16_bits_rne(y).reshape(x_bits.shape)


def rmsnorm_rope_kv_append(state, start_frames, q_bits, k_bits, v_bits, gain_q, gain_k, eps, cos, sin):
    """RMSNorm of q and k, then the append (plain ring or sink cache, by the type of `state`)."""
    qn = rmsnorm_tokens(q_bits, gain_q, eps)
    kn = rmsnorm_tokens(k_bits, gain_k, eps)
    if isinstance(state, SinkRingState):
        return rope_kv_append_sink(state, start_frames, qn, kn, v_bits, cos, sin)
    return rope_kv_append(state, start_frames, qn, kn, v_bits, cos, sin)
