"""The checking build of the library (-DUNSTEP_CHECK) with guard bands around every output.

No memory checker can be run on the kernels here, so the library carries its own: in a checking
build every global store of the three kernels is tested against the extent of the buffer it
belongs to, and a store outside is skipped and reported through the status word instead of being
made.  This file runs the shapes with the most index arithmetic (tiny, ragged tiles, more streams
than one launch carries, a sink prefix, the fused norm) through that build, with every output
placed between two bands of sentinel values, and asserts: status 0 (no store was refused), bands
intact (no store landed outside), results equal to the oracle.  The checking build is loaded in a
child process (UNSTEP_LIB_VARIANT=check), so the normal library of this process is untouched.
"""

import os
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GUARD = 4096          # bf16 elements (8 KB) of sentinel before and after each buffer
BAND = 0x7FA5         # a NaN pattern that neither the kernels nor the other sentinels produce


def _child():
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import ctypes
    import torch
    import oracle as O
    import paper_2609_32518_b200 as U
    import workloads as W
    from harness import OraclePath, abi_shape, attn_errors, to_dev

    assert os.path.basename(U.lib()._name) == "libunstep_check.so"

    class Guarded:
        """A bf16 device buffer of `numel` elements between two sentinel bands."""

        def __init__(self, shape, fill=0x7FC1):
            self.n = int(np.prod(shape))
            self.raw = torch.full((self.n + 2 * GUARD,), BAND, dtype=torch.int16, device="cuda")
            self.raw[GUARD:GUARD + self.n] = fill
            self.t = self.raw[GUARD:GUARD + self.n].view(torch.bfloat16).view(shape)
            assert self.t.data_ptr() % 16 == 0 and self.t.is_contiguous()

        def intact(self):
            lo, hi = self.raw[:GUARD], self.raw[GUARD + self.n:]
            return bool((lo == BAND).all()) and bool((hi == BAND).all())

        def bits(self):
            return self.t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)

    def run(wl, extra_history=(), sink=0, sink_attend=0, norm=False):
        sh = wl.shape
        abi = abi_shape(sh)
        cache_shape = (sh.batch, sink + sh.ring_frames, sh.tokens_per_frame, sh.heads, sh.head_dim)
        act_shape = (sh.batch, sh.chunk_tokens, sh.heads, sh.head_dim)
        ck, cv = Guarded(cache_shape), Guarded(cache_shape)
        if sink:
            ora_state = O.SinkRingState(sh.batch, sink, sh.ring_frames, sh.tokens_per_frame, sh.heads)
        else:
            ora_state = O.RingState(sh.batch, sh.ring_frames, sh.tokens_per_frame, sh.heads)
        gain = None
        if norm:
            rng = np.random.Generator(np.random.PCG64(7))
            gain = [(1.0 + 0.1 * rng.standard_normal(sh.heads * sh.head_dim)).astype(np.float32) for _ in range(2)]
        tabs = {}

        def table(s):
            if s not in tabs:
                # the library's own table kernel, into guarded float32 buffers
                n = sh.chunk_tokens * 64
                raw = [torch.full((n + 2 * GUARD,), float("nan"), dtype=torch.float32, device="cuda") for _ in range(2)]
                c, sn = (r[GUARD:GUARD + n].view(sh.chunk_tokens, 64) for r in raw)
                U.rope_table(abi, s, c, sn)
                torch.cuda.synchronize()
                for r in raw:
                    assert torch.isnan(r[:GUARD]).all() and torch.isnan(r[GUARD + n:]).all(), "table wrote outside"
                oc, os_ = O.rope_table(s, sh.chunk_frames, sh.grid_h, sh.grid_w, sh.bands, sh.rope_base)
                assert np.abs(c.cpu().numpy() - oc).max() < 1e-6 and np.abs(sn.cpu().numpy() - os_).max() < 1e-6
                # parity of the cache is defined on the oracle's table bytes
                tabs[s] = (torch.from_numpy(oc).cuda(), torch.from_numpy(os_).cuda(), oc, os_)
            return tabs[s]

        def append(starts, tag=0):
            starts = [int(s) for s in starts]
            q, k, v = W.batch_qkv(wl, starts, tag)
            cos = torch.stack([table(s)[0] for s in starts]).contiguous()
            sin = torch.stack([table(s)[1] for s in starts]).contiguous()
            ocos = np.stack([table(s)[2] for s in starts])
            osin = np.stack([table(s)[3] for s in starts])
            stride = sh.chunk_tokens * 64
            q_out = Guarded(act_shape)
            if norm:
                gq, gk = (torch.from_numpy(x).cuda() for x in gain)
                U.rmsnorm_rope_kv_append(abi, sink, starts, to_dev(q), to_dev(k), to_dev(v), gq, gk, 1e-6, cos, sin,
                                         q_out.t, ck.t, cv.t, table_stream_stride=stride)
                q_ref = O.rmsnorm_rope_kv_append(ora_state, starts, q, k, v, gain[0], gain[1], 1e-6, ocos, osin)
            elif sink:
                U.rope_kv_append_sink(abi, sink, starts, to_dev(q), to_dev(k), to_dev(v), cos, sin, q_out.t, ck.t, cv.t,
                                      table_stream_stride=stride)
                q_ref = O.rope_kv_append_sink(ora_state, starts, q, k, v, ocos, osin)
            else:
                U.rope_kv_append(abi, starts, to_dev(q), to_dev(k), to_dev(v), cos, sin, q_out.t, ck.t, cv.t,
                                 table_stream_stride=stride)
                q_ref = O.rope_kv_append(ora_state, starts, q, k, v, ocos, osin)
            torch.cuda.synchronize()
            assert U.poll_status() == 0, "a store of the append was refused"
            assert q_out.intact() and ck.intact() and cv.intact(), "the append wrote outside its buffers"
            assert np.array_equal(q_out.bits(), q_ref)
            ok_k = ora_state.cache_k if sink else ora_state.ring_k
            ok_v = ora_state.cache_v if sink else ora_state.ring_v
            assert np.array_equal(ck.bits(), ok_k) and np.array_equal(cv.bits(), ok_v)
            return q_out, q_ref

        for starts in extra_history:
            append(starts)
        q_out, q_ref = append(wl.measured_starts)
        for wf in wl.window_frames:
            out = Guarded(act_shape)
            starts = [int(s) for s in wl.measured_starts]
            if sink:
                U.window_attn_sink(abi, sink, starts, wf, sink_attend, q_out.t, ck.t, cv.t, out.t)
                ref = O.window_attn_sink(ora_state, starts, wf, sink_attend, q_ref, sh.chunk_frames)
            else:
                U.window_attn(abi, starts, wf, q_out.t, ck.t, cv.t, out.t)
                ref = O.window_attn(ora_state, starts, wf, q_ref, sh.chunk_frames)
            torch.cuda.synchronize()
            assert U.poll_status() == 0, "a store of the attention was refused"
            assert out.intact() and q_out.intact() and ck.intact() and cv.intact(), "the attention wrote outside"
            mx, mean, rel = attn_errors(out.bits(), ref)
            assert mx <= 2e-2 and mean <= 2e-3 and rel <= 1.5e-2, (wl.name, wf, mx, mean, rel)
        print("ok", wl.name, flush=True)

    # the checks are armed: one store past the end is skipped and reported
    probe = torch.zeros(5, dtype=torch.int32, device="cuda")
    lib = U.lib()
    lib.unstep_selftest_bounds_check.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
    lib.unstep_selftest_bounds_check.restype = ctypes.c_int
    assert lib.unstep_selftest_bounds_check(ctypes.c_void_p(probe.data_ptr()), None) == 0
    torch.cuda.synchronize()
    assert probe.cpu().tolist() == [7, 7, 7, 7, 0]
    assert U.poll_status() == -6 and U.poll_status() == 0

    cfg1 = W.WORKLOADS["cfg1"]
    run(cfg1, extra_history=[[0], [2]])
    w = W.WORKLOADS["cfg1_wrapped"]
    run(w, extra_history=[[s] for s in w.history_starts[0]])
    # ragged tiles: T = 200 keys per frame, L = 600 queries, two streams at different fill levels
    sh = W.Shape(batch=2, heads=3, chunk_frames=3, grid_h=8, grid_w=25, ring_frames=7)
    run(W.Workload("ragged", sh, seed=22, history_starts=((), ()), measured_starts=(12, 3),
                   window_frames=(7, 5, 3), k_scale=4.0), extra_history=[[0, 0], [3, 0], [6, 0], [9, 0]])
    # 35 and 37 streams: more than one launch carries, frames shorter than a tile
    for nstreams, seed in ((35, 24), (37, 33)):
        sh = W.Shape(batch=nstreams, heads=1, chunk_frames=1, grid_h=4, grid_w=10, ring_frames=4)
        starts = tuple(3 + (b % 5) for b in range(nstreams))
        run(W.Workload(f"many{nstreams}", sh, seed=seed, history_starts=((),) * nstreams, measured_starts=starts,
                       window_frames=(4, 2, 1)), extra_history=[[s - back for s in starts] for back in (3, 2, 1)])
    # sink prefix in front of the ring, ring wrapped
    sh = W.Shape(batch=2, heads=2, chunk_frames=3, grid_h=8, grid_w=25, ring_frames=6)
    run(W.Workload("sink", sh, seed=34, history_starts=((), ()), measured_starts=(12, 9), window_frames=(6,),
                   sink_frames=3, sink_attend=3), extra_history=[[0, 0], [3, 3], [6, 6], [9, 6]], sink=3, sink_attend=3)
    # the fused norm in front of the append, ragged queries
    sh = W.Shape(batch=2, heads=3, chunk_frames=2, grid_h=3, grid_w=5, ring_frames=6)
    run(W.Workload("norm", sh, seed=35, history_starts=((), ()), measured_starts=(6, 2), window_frames=(6, 2)),
        extra_history=[[0, 0], [2, 0], [4, 0]], norm=True)
    print("all ok")


@pytest.mark.gpu
def test_checking_build_reports_no_refused_store_and_guard_bands_stay_intact():
    env = dict(os.environ, UNSTEP_LIB_VARIANT="check")
    res = subprocess.run([sys.executable, os.path.abspath(__file__), "--child"], env=env, capture_output=True,
                         text=True, timeout=900)
    assert res.returncode == 0 and "all ok" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]


def test_checking_build_compiles_and_exports_its_selftest():
    import ctypes
    from paper_2609_32518_b200 import build as B
    lib = ctypes.CDLL(B.build(variant="check"))
    assert hasattr(lib, "unstep_selftest_bounds_check") and hasattr(lib, "unstep_window_attn")
    import paper_2609_32518_b200 as U
    assert not hasattr(U.lib(), "unstep_selftest_bounds_check")      # the normal build carries no checks
    assert "store" in U.strerror(-6)


if __name__ == "__main__":
    if "--child" in sys.argv:
        _child()
