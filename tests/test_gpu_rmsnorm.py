"""GPU parity of the fused RMSNorm + RoPE + append against the oracle: bit-exact."""

import numpy as np
import pytest
import torch

import oracle as O
import paper_2609_32518_b200 as U
import workloads as W
from harness import DevicePath, to_bits, to_dev

pytestmark = pytest.mark.gpu


def gains(width, seed):
    rng = np.random.default_rng(seed)
    return ((1.0 + 0.2 * rng.standard_normal(width)).astype(np.float32),
            (1.0 + 0.2 * rng.standard_normal(width)).astype(np.float32))


def run(sh, starts_list, sink=0, eps=1e-6, seed=61, in_place=False, scale=1.0):
    wl = W.Workload("norm", sh, seed=seed, history_starts=((),) * sh.batch,
                    measured_starts=tuple(starts_list[0]), window_frames=(sh.ring_frames,), k_scale=scale)
    gq, gk = gains(sh.heads * 128, seed)
    dev = DevicePath(sh, sink_frames=sink)
    ora = (O.SinkRingState(sh.batch, sink, sh.ring_frames, sh.tokens_per_frame, sh.heads) if sink
           else O.RingState(sh.batch, sh.ring_frames, sh.tokens_per_frame, sh.heads))
    gq_d, gk_d = torch.from_numpy(gq).cuda(), torch.from_numpy(gk).cuda()
    for starts in starts_list:
        q, k, v = W.batch_qkv(wl, starts)
        same = len(set(starts)) == 1
        tabs = [O.rope_table(s, sh.chunk_frames, sh.grid_h, sh.grid_w) for s in (starts[:1] if same else starts)]
        cos = np.stack([t[0] for t in tabs]) if not same else tabs[0][0]
        sin = np.stack([t[1] for t in tabs]) if not same else tabs[0][1]
        q_ref = O.rmsnorm_rope_kv_append(ora, starts, q, k, v, gq, gk, eps, cos, sin)
        qd = to_dev(q)
        q_out = qd if in_place else torch.empty_like(qd)
        U.rmsnorm_rope_kv_append(dev.abi, sink, list(starts), qd, to_dev(k), to_dev(v), gq_d, gk_d, eps,
                                 torch.from_numpy(np.ascontiguousarray(cos)).cuda(),
                                 torch.from_numpy(np.ascontiguousarray(sin)).cuda(), q_out, dev.ring_k,
                                 dev.ring_v, table_stream_stride=0 if same else sh.chunk_tokens * 64)
        assert np.array_equal(to_bits(q_out), q_ref), "q_out differs"
        ck = ora.cache_k if sink else ora.ring_k
        cv = ora.cache_v if sink else ora.ring_v
        assert np.array_equal(to_bits(dev.ring_k), ck), "cache K differs"
        assert np.array_equal(to_bits(dev.ring_v), cv), "cache V differs"


def test_tiny_and_wrapped():
    sh = W.WORKLOADS["cfg1"].shape
    run(sh, [(0,), (2,), (4,), (6,), (8,)])


def test_ragged_streams_own_tables_sink_and_in_place():
    sh = W.Shape(batch=3, heads=3, chunk_frames=3, grid_h=5, grid_w=7, ring_frames=6)
    run(sh, [(0, 3, 9), (3, 6, 12), (21, 9, 15)], sink=3, in_place=True, scale=4.0)


def test_1p3b_shape():
    run(W.WORKLOADS["cfg2"].shape, [(18,)], eps=1e-5)


def test_14b_shape():
    run(W.WORKLOADS["cfg5"].shape, [(9,)])


@pytest.mark.parametrize("heads", [1, 5, 6, 7, 13, 17, 18, 19, 33, 64, 65, 70])
def test_every_block_width_and_the_wide_token_kernel(heads):
    # 1..4 vectors per thread, blocks of 32 to 256 threads with and without idle lanes, and (from
    # 65 heads on) the warp-per-token kernel; two streams, the ring wrapped
    sh = W.Shape(batch=2, heads=heads, chunk_frames=2, grid_h=3, grid_w=7, ring_frames=4)
    run(sh, [(0, 2), (2, 4), (4, 6)], seed=70 + heads, scale=2.0)


def test_argument_checks():
    import ctypes
    sh = U.Shape.make(batch=1, heads=2, chunk_frames=2, grid_h=8, grid_w=8, ring_frames=6)
    one = (ctypes.c_int32 * 1)(0)
    f = 0x10000
    L = U.lib()
    args = [f] * 5
    assert L.unstep_rmsnorm_rope_kv_append(ctypes.byref(sh), 0, one, f, f, f, None, f, 1e-6, f, f, 0, f, f, f, None) == -1
    assert L.unstep_rmsnorm_rope_kv_append(ctypes.byref(sh), 0, one, f, f, f, f, f, -1.0, f, f, 0, f, f, f, None) == -1
    assert L.unstep_rmsnorm_rope_kv_append(ctypes.byref(sh), 0, one, f, f, f, f, f + 4, 1e-6, f, f, 0, f, f, f, None) == -1
