"""Seeded synthetic inputs shaped like the paper's workloads.

This module only makes inputs: shapes, seeds, random bf16 bit patterns and the
chunk schedule of each configuration.  It holds none of the method's
arithmetic (no RoPE, no ring indexing, no attention) and is the one module
that both the CPU oracle's tests and the CUDA path's tests/benchmark use, so
that both sides see the same bytes.

The inputs stand in for the activations of a Wan2.1-class causal video DiT
(1.3B: 12 heads x 128, 30x52 = 1560 tokens per latent frame, 3-frame chunks;
14B/720p: 40 heads x 128, 45x80 = 3600 tokens per frame): after the q/k
RMS-norm those activations are O(1) per coordinate, which N(0,1) reproduces.
bf16 tensors are carried on the host as uint16 bit patterns.
"""

from __future__ import annotations

from dataclasses import dataclass, field, replace

import numpy as np


@dataclass(frozen=True)
class Shape:
    batch: int
    heads: int
    chunk_frames: int
    grid_h: int
    grid_w: int
    ring_frames: int
    head_dim: int = 128
    bands: tuple = (44, 42, 42)
    rope_base: float = 10000.0

    @property
    def tokens_per_frame(self) -> int:
        return self.grid_h * self.grid_w

    @property
    def chunk_tokens(self) -> int:
        return self.chunk_frames * self.tokens_per_frame


@dataclass(frozen=True)
class Workload:
    """One configuration: a shape, a seed, the chunks streamed before the
    measured one, and the measured chunk(s)."""
    name: str
    shape: Shape
    seed: int
    history_starts: tuple        # per stream: start frames appended before the measured chunk
    measured_starts: tuple       # per stream: start frame of the measured chunk
    window_frames: tuple         # window lengths (frames, chunk included) to attend with
    k_scale: float = 1.0
    note: str = ""
    sink_frames: int = 0         # slots of the never-evicted prefix (0 = plain rolling window)
    sink_attend: int = 0         # sink frames attended

    def keys_attended(self, window_frames: int):
        fc = self.shape.chunk_frames
        out = []
        for s in self.measured_starts:
            hi = s + fc
            lo = max(0, hi - window_frames)
            out.append((min(self.sink_attend, lo) + hi - lo) * self.shape.tokens_per_frame)
        return out

    def attn_flops(self, window_frames: int) -> float:
        sh = self.shape
        return float(sum(4.0 * sh.chunk_tokens * S * sh.head_dim * sh.heads
                         for S in self.keys_attended(window_frames)))

    def append_bytes(self, distinct_tables: int | None = None) -> float:
        sh = self.shape
        nt = len(set(self.measured_starts)) if distinct_tables is None else distinct_tables
        return float(6 * sh.batch * sh.chunk_tokens * sh.heads * sh.head_dim * 2
                     + nt * 2 * sh.chunk_tokens * (sh.head_dim // 2) * 4)


_S13 = Shape(batch=1, heads=12, chunk_frames=3, grid_h=30, grid_w=52, ring_frames=21)

WORKLOADS = {
    # tiny: 2 heads, 8x8 grid, 2-frame chunks, 4 cached frames + chunk = 384 keys
    "cfg1": Workload("cfg1", Shape(batch=1, heads=2, chunk_frames=2, grid_h=8, grid_w=8,
                                   ring_frames=6),
                     seed=0, history_starts=((0, 2),), measured_starts=(4,), window_frames=(6,)),
    # the same tiny shape with the ring wrapped: chunks 0..14 streamed, measured at 16
    "cfg1_wrapped": Workload("cfg1_wrapped", Shape(batch=1, heads=2, chunk_frames=2, grid_h=8,
                                                   grid_w=8, ring_frames=6),
                             seed=0, history_starts=(tuple(range(0, 16, 2)),),
                             measured_starts=(16,), window_frames=(6, 4, 2)),
    # 1.3B-class: final chunk of a 21-frame clip, 18 cached + 3 = 32760 keys
    "cfg2": Workload("cfg2", _S13, seed=1, history_starts=(tuple(range(0, 18, 3)),),
                     measured_starts=(18,), window_frames=(21,)),
    # window sweep, K x4, ring wrapped more than twice, measured at s=42
    "cfg3": Workload("cfg3", _S13, seed=2, history_starts=(tuple(range(0, 42, 3)),),
                     measured_starts=(42,), window_frames=(3, 6, 9, 12, 21), k_scale=4.0),
    # second point of the sweep: measured at s=51 (slots 9..11), where only the 21-frame window wraps
    "cfg3_s51": Workload("cfg3_s51", _S13, seed=2, history_starts=(tuple(range(0, 51, 3)),),
                         measured_starts=(51,), window_frames=(3, 6, 9, 12, 21), k_scale=4.0),
    # tight ring (capacity = window = 9 frames, the minimal-memory deployment), measured at s = 3*C
    "cfg3_tight": Workload("cfg3_tight", replace(_S13, ring_frames=9), seed=2,
                           history_starts=(tuple(range(0, 27, 3)),), measured_starts=(27,),
                           window_frames=(9,), k_scale=4.0),
    # four streams at fill levels 0/6/12/18, clean-cache re-append pattern
    "cfg4": Workload("cfg4", replace(_S13, batch=4), seed=3,
                     history_starts=((), (0, 3), (0, 3, 6, 9), (0, 3, 6, 9, 12, 15)),
                     measured_starts=(0, 6, 12, 18), window_frames=(21,)),
    # 14B-class 720p layer: 9 cached + 3 = 43200 keys
    "cfg5": Workload("cfg5", Shape(batch=1, heads=40, chunk_frames=3, grid_h=45, grid_w=80,
                                   ring_frames=12),
                     seed=4, history_starts=((0, 3, 6),), measured_starts=(9,),
                     window_frames=(12,)),
}


# the paper's operating point: 3 sink + 6 recent frames = 14040 keys, last chunk of a 21-frame clip
WORKLOADS["cfg2_sink9"] = Workload("cfg2_sink9", replace(_S13, ring_frames=6), seed=5,
                                   history_starts=(tuple(range(0, 18, 3)),), measured_starts=(18,),
                                   window_frames=(6,), sink_frames=3, sink_attend=3)
# the last chunk of a 30 s clip (123 latent frames) through the same 9-frame cache
WORKLOADS["cfg2_sink9_long"] = Workload("cfg2_sink9_long", replace(_S13, ring_frames=6), seed=6,
                                        history_starts=(tuple(range(0, 120, 3)),), measured_starts=(120,),
                                        window_frames=(6,), sink_frames=3, sink_attend=3)


def with_heads(wl: Workload, heads: int) -> Workload:
    """The same workload with another number of heads (a rank's share when heads are split over GPUs)."""
    return replace(wl, shape=replace(wl.shape, heads=heads))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Nearest-even bf16 bit pattern of finite float32 data (input generation only)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(
        np.float32)


def normal_bf16(seed_key, shape, scale: float = 1.0) -> np.ndarray:
    """N(0,1)*scale as bf16 bits, from PCG64 seeded by an integer tuple."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence(list(seed_key))))
    x = rng.standard_normal(size=shape, dtype=np.float32)
    bits = f32_to_bf16_bits(x)
    if scale != 1.0:
        # power-of-two scales are exact in bf16
        bits = f32_to_bf16_bits(bf16_bits_to_f32(bits) * np.float32(scale))
    return bits


def chunk_qkv(wl: Workload, stream: int, start_frame: int, tag: int = 0):
    """(q, k, v) bf16 bits [L, Hn, 128] of one chunk of one stream.  `tag`
    distinguishes repeated appends of the same chunk (noisy pass 0, clean pass 1)."""
    sh = wl.shape
    dims = (sh.chunk_tokens, sh.heads, sh.head_dim)
    key = (wl.seed, stream, start_frame, tag)
    q = normal_bf16(key + (0,), dims)
    k = normal_bf16(key + (1,), dims, scale=wl.k_scale)
    v = normal_bf16(key + (2,), dims)
    return q, k, v


def batch_qkv(wl: Workload, start_frames, tag: int = 0):
    """Stacked (q, k, v) [B, L, Hn, 128] for one chunk of every stream."""
    parts = [chunk_qkv(wl, b, int(s), tag) for b, s in enumerate(start_frames)]
    return tuple(np.stack([p[i] for p in parts], axis=0) for i in range(3))


def sample_rows(n_rows: int, tile: int = 128, per_tile: int = 8, seed: int = 0) -> np.ndarray:
    """Stratified query-row sample: first and last row of every `tile`-row tile,
    `per_tile` rows in all from each tile, and the whole ragged tail tile."""
    rng = np.random.Generator(np.random.PCG64(seed))
    rows = []
    for t0 in range(0, n_rows, tile):
        t1 = min(t0 + tile, n_rows)
        if t1 - t0 < tile:
            rows.extend(range(t0, t1))
            continue
        pick = {t0, t1 - 1}
        while len(pick) < per_tile:
            pick.add(int(rng.integers(t0, t1)))
        rows.extend(sorted(pick))
    return np.asarray(rows, dtype=np.int64)
