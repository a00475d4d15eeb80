"""Clock-stamp timeline of the attention kernel's roles (a debugging aid, not part of the path).

Builds a copy of the library with -DUNSTEP_TRACE into a temporary directory (the in-tree
library is left alone), runs `unstep_window_attn` a few times on random data of one workload
shape and prints, for CTA 0, the clock64 stamps that the kernel's roles leave per key tile:

  softmax warps (one line per warp 0..3 of each query tile's group):
      wait = starts waiting for S, s_rdy = S complete, ld = first scores in registers,
      p = P handed to the tensor core
  MMA issuers: wait_p = starts waiting for P, got_p = P arrived, got_turn = its turn on the
      tensor pipe, pv = P V issued, qk = next Q K^T issued and committed

  python -m paper_2609_32518_b200.timeline [--workload cfg2] [--window 21] [--tiles 8:14]

The numbers are cycles relative to the first stamp shown; a traced run is slower than a normal
one (every stamp is a global store), so read differences, not the total.
"""

from __future__ import annotations

import argparse
import ctypes
import os
import subprocess
import sys
import tempfile


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--window", type=int, default=None)
    ap.add_argument("--tiles", default="8:14", help="key-tile range lo:hi of CTA 0's first item (below 64)")
    args = ap.parse_args()

    import numpy as np
    import torch
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    if root not in sys.path:
        sys.path.insert(0, root)
    import workloads as W
    from . import build as B

    tmp = tempfile.mkdtemp(prefix="unstep_trace_")
    so = os.path.join(tmp, "libunstep_trace.so")
    cmd = [B._nvcc()] + B.NVCC_FLAGS + ["-DUNSTEP_TRACE", "-I", B.INCLUDE, "-I", B.CSRC, "-o", so]
    cmd += [os.path.join(B.CSRC, s) for s in B.SOURCES]
    subprocess.check_call(cmd, stderr=subprocess.DEVNULL)
    B.LIB_PATH = so                      # the binding loads whatever build() returns
    B.build = lambda *a, **k: so
    from . import binding as U

    wl = W.WORKLOADS[args.workload]
    sh = wl.shape
    wf = args.window if args.window is not None else wl.window_frames[-1]
    abi = U.Shape.make(sh.batch, sh.heads, sh.chunk_frames, sh.grid_h, sh.grid_w, sh.ring_frames)
    dev = torch.device("cuda", 0)
    gen = torch.Generator(device=dev).manual_seed(1)
    cache = (sh.batch, wl.sink_frames + sh.ring_frames, sh.tokens_per_frame, sh.heads, sh.head_dim)
    ck = torch.randn(cache, generator=gen, device=dev).to(torch.bfloat16)
    cv = torch.randn(cache, generator=gen, device=dev).to(torch.bfloat16)
    q = torch.randn((sh.batch, sh.chunk_tokens, sh.heads, sh.head_dim), generator=gen, device=dev).to(torch.bfloat16)
    out = torch.empty_like(q)
    starts = list(wl.measured_starts)
    for _ in range(3):
        if wl.sink_frames:
            U.window_attn_sink(abi, wl.sink_frames, starts, wf, wl.sink_attend, q, ck, cv, out)
        else:
            U.window_attn(abi, starts, wf, q, ck, cv, out)
    torch.cuda.synchronize()

    lib = U.lib()
    buf = (ctypes.c_longlong * (12 * 64 * 8))()
    lib.unstep_debug_read_trace.argtypes = [ctypes.c_void_p]
    lib.unstep_debug_read_trace.restype = ctypes.c_int
    if lib.unstep_debug_read_trace(buf) != 0:
        raise RuntimeError("reading the trace failed")
    t = np.array(buf[:], dtype=np.int64).reshape(12, 64, 8)
    lo, hi = (int(x) for x in args.tiles.split(":"))
    base = t[0, lo, 0]
    np.set_printoptions(linewidth=200)
    print(f"workload {args.workload}, window {wf} frames, CTA 0, key tiles {lo}..{hi - 1}; cycles since tile {lo}")
    for a in (0, 1):
        for w in range(4):
            print(f"softmax group {a} warp {w}: [wait, s_rdy, ld, p]")
            print(t[2 * w + a, lo:hi][:, [0, 1, 2, 5]] - base)
    for a in (0, 1):
        print(f"MMA issuer {a}: [wait_p, got_p, -, got_turn, pv, qk]")
        print(t[8 + a, lo:hi, :6] - base)
    print("device status:", U.poll_status())


if __name__ == "__main__":
    main()
