"""Shared plumbing of the GPU parity tests: the same seeded bytes go to the CPU
oracle and, through the C ABI, to the CUDA library."""

from __future__ import annotations

import numpy as np
import torch

import oracle as O
import paper_2609_32518_b200 as U
import workloads as W

SENTINEL = 0x7FC1


def to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def to_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def abi_shape(sh: W.Shape) -> U.Shape:
    return U.Shape.make(sh.batch, sh.heads, sh.chunk_frames, sh.grid_h, sh.grid_w, sh.ring_frames,
                        head_dim=sh.head_dim, bands=sh.bands, rope_base=sh.rope_base)


class DevicePath:
    """Device buffers of one layer and the calls on them."""

    def __init__(self, sh: W.Shape, use_oracle_table: bool = True, sink_frames: int = 0):
        self.sh = sh
        self.abi = abi_shape(sh)
        self.sink = sink_frames
        ring_shape = (sh.batch, sink_frames + sh.ring_frames, sh.tokens_per_frame, sh.heads, sh.head_dim)
        fill = torch.tensor(SENTINEL, dtype=torch.int16)
        self.ring_k = torch.full(ring_shape, int(fill), dtype=torch.int16, device="cuda").view(torch.bfloat16)
        self.ring_v = torch.full(ring_shape, int(fill), dtype=torch.int16, device="cuda").view(torch.bfloat16)
        self.use_oracle_table = use_oracle_table
        self._tables = {}

    def table(self, s: int):
        """Device (cos, sin) for a chunk starting at s: the oracle's bytes uploaded, or
        the library's own table."""
        if s not in self._tables:
            sh = self.sh
            if self.use_oracle_table:
                c, sn = O.rope_table(s, sh.chunk_frames, sh.grid_h, sh.grid_w, sh.bands, sh.rope_base)
                self._tables[s] = (torch.from_numpy(c).cuda(), torch.from_numpy(sn).cuda())
            else:
                c = torch.empty((sh.chunk_tokens, 64), dtype=torch.float32, device="cuda")
                sn = torch.empty_like(c)
                U.rope_table(self.abi, s, c, sn)
                self._tables[s] = (c, sn)
        return self._tables[s]

    def append(self, starts, q_bits, k_bits, v_bits, in_place: bool = False) -> torch.Tensor:
        starts = [int(s) for s in starts]
        if len(set(starts)) == 1:
            cos, sin = self.table(starts[0])
            stride = 0
        else:
            cos = torch.stack([self.table(s)[0] for s in starts]).contiguous()
            sin = torch.stack([self.table(s)[1] for s in starts]).contiguous()
            stride = self.sh.chunk_tokens * 64
        q = to_dev(q_bits)
        q_out = q if in_place else torch.empty_like(q)
        if self.sink:
            U.rope_kv_append_sink(self.abi, self.sink, starts, q, to_dev(k_bits), to_dev(v_bits), cos, sin,
                                  q_out, self.ring_k, self.ring_v, table_stream_stride=stride)
        else:
            U.rope_kv_append(self.abi, starts, q, to_dev(k_bits), to_dev(v_bits), cos, sin, q_out,
                             self.ring_k, self.ring_v, table_stream_stride=stride)
        return q_out

    def attend_sink(self, starts, recent_frames: int, sink_attend: int, q_rot: torch.Tensor) -> torch.Tensor:
        out = torch.full_like(q_rot.view(torch.int16), SENTINEL).view(torch.bfloat16)
        U.window_attn_sink(self.abi, self.sink, [int(s) for s in starts], recent_frames, sink_attend,
                           q_rot, self.ring_k, self.ring_v, out)
        return out

    def attend(self, starts, window_frames: int, q_rot: torch.Tensor) -> torch.Tensor:
        out = torch.full_like(q_rot.view(torch.int16), SENTINEL).view(torch.bfloat16)
        U.window_attn(self.abi, [int(s) for s in starts], window_frames, q_rot, self.ring_k,
                      self.ring_v, out)
        return out


class OraclePath:
    def __init__(self, sh: W.Shape):
        self.sh = sh
        self.ring = O.RingState(sh.batch, sh.ring_frames, sh.tokens_per_frame, sh.heads)
        self._tables = {}

    def table(self, s):
        if s not in self._tables:
            sh = self.sh
            self._tables[s] = O.rope_table(s, sh.chunk_frames, sh.grid_h, sh.grid_w, sh.bands,
                                           sh.rope_base)
        return self._tables[s]

    def append(self, starts, q_bits, k_bits, v_bits) -> np.ndarray:
        starts = [int(s) for s in starts]
        if len(set(starts)) == 1:
            cos, sin = self.table(starts[0])
        else:
            cos = np.stack([self.table(s)[0] for s in starts])
            sin = np.stack([self.table(s)[1] for s in starts])
        return O.rope_kv_append(self.ring, starts, q_bits, k_bits, v_bits, cos, sin)

    def attend(self, starts, window_frames, q_rot_bits, rows=None, heads=None):
        return O.window_attn(self.ring, starts, window_frames, q_rot_bits, self.sh.chunk_frames,
                             rows=rows, heads=heads)


def stream_history(wl: W.Workload, dev: DevicePath, ora: OraclePath, check_ring: bool = True):
    """Append every history chunk of every stream on both sides (streams advance
    together where their schedules allow, else one by one is emulated by re-appending)."""
    sh = wl.shape
    depth = max(len(h) for h in wl.history_starts)
    for i in range(depth):
        # streams whose history is shorter re-append their last chunk (an overwrite, harmless)
        starts = [h[min(i, len(h) - 1)] if len(h) else None for h in wl.history_starts]
        if any(s is None for s in starts):
            # streams with empty history take a placeholder chunk at the measured start
            starts = [wl.measured_starts[b] if s is None else s for b, s in enumerate(starts)]
        q, k, v = W.batch_qkv(wl, starts)
        dev.append(starts, q, k, v)
        ora.append(starts, q, k, v)
        if check_ring:
            assert_ring_equal(dev, ora)


def assert_ring_equal(dev: DevicePath, ora: OraclePath):
    gk, gv = to_bits(dev.ring_k), to_bits(dev.ring_v)
    bad_k = int((gk != ora.ring.ring_k).sum())
    bad_v = int((gv != ora.ring.ring_v).sum())
    assert bad_k == 0 and bad_v == 0, f"ring mismatch: {bad_k} K elements, {bad_v} V elements"


def attn_errors(got_bits: np.ndarray, ref: np.ndarray):
    """(max abs, mean abs, relative L2) of a bf16 result against the float64 oracle."""
    got = O.bf16_bits_to_f32(got_bits).astype(np.float64)
    err = np.abs(got - ref)
    rel = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))
    return float(err.max()), float(err.mean()), rel
