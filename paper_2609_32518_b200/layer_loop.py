"""Host-side bookkeeping for a stack of self-attention layers and a CUDA-graph replay of one
chunk step across all of them.

The paper's runtime lesson (Sec. "DiT runtime stack") is that in few-step causal models the
per-call host work around attention shows up in end-to-end throughput: positions live on the
CPU, cos/sin tables are cached per starting frame, nothing is read back from the GPU.  This
module keeps exactly that state on the host -- one KV cache per layer, one table per
(start frame, grid) -- and issues the C-ABI calls for a chunk.  Because every call's arguments
are plain host values, the launches of a whole chunk step (all layers) can be captured once
per starting frame into a CUDA graph and replayed for each denoising call of that chunk
(the repeated calls overwrite the same cache entries).

Only argument marshalling happens here; all arithmetic is in the CUDA library.

  python -m paper_2609_32518_b200.layer_loop [--layers 30] [--workload cfg2_sink9] [--steps 20]
prints one JSON line with microseconds per layer per chunk, eager and under graph replay.
"""

from __future__ import annotations

import argparse
import json
import os
import sys

from . import binding as U


class ChunkStepper:
    """KV caches of `n_layers` layers of one model plus the cached RoPE tables."""

    def __init__(self, shape: U.Shape, n_layers: int, window_frames: int, sink_frames: int = 0,
                 sink_attend: int = 0, device=None):
        import torch
        self.shape, self.n_layers = shape, n_layers
        self.window, self.sink, self.sink_attend = window_frames, sink_frames, sink_attend
        self.device = device if device is not None else torch.device("cuda", torch.cuda.current_device())
        cache = (shape.batch, sink_frames + shape.ring_frames, shape.tokens_per_frame, shape.heads,
                 shape.head_dim)
        self.cache_k = [torch.zeros(cache, dtype=torch.bfloat16, device=self.device) for _ in range(n_layers)]
        self.cache_v = [torch.zeros(cache, dtype=torch.bfloat16, device=self.device) for _ in range(n_layers)]
        self._tables = {}
        self._graphs = {}
        # Every graph of this stepper is captured on this one stream.  The attention call keeps its
        # scratch per stream and a capture freezes the scratch pointers into the graph, so one
        # capture stream means one scratch for all graphs (replays of one stepper run one after
        # the other on the caller's stream and may share it).
        self._capture_stream = torch.cuda.Stream(device=self.device)

    def table(self, start_frame: int):
        """cos/sin of the chunk starting at `start_frame`, built once and kept (the paper's cache)."""
        import torch
        key = (int(start_frame), self.shape.chunk_frames, self.shape.grid_h, self.shape.grid_w)
        if key not in self._tables:
            cos = torch.empty((self.shape.chunk_tokens, 64), dtype=torch.float32, device=self.device)
            sin = torch.empty_like(cos)
            U.rope_table(self.shape, int(start_frame), cos, sin)
            self._tables[key] = (cos, sin)
        return self._tables[key]

    def layer_step(self, layer: int, start_frame: int, q, k, v, q_rot, out):
        """Append the chunk's K/V of one layer and attend; all streams share `start_frame`."""
        starts = [int(start_frame)] * self.shape.batch
        cos, sin = self.table(start_frame)
        ck, cv = self.cache_k[layer], self.cache_v[layer]
        if self.sink:
            U.rope_kv_append_sink(self.shape, self.sink, starts, q, k, v, cos, sin, q_rot, ck, cv)
            U.window_attn_sink(self.shape, self.sink, starts, self.window, self.sink_attend, q_rot, ck, cv, out)
        else:
            U.rope_kv_append(self.shape, starts, q, k, v, cos, sin, q_rot, ck, cv)
            U.window_attn(self.shape, starts, self.window, q_rot, ck, cv, out)

    def chunk_step(self, start_frame: int, qkv, q_rot, outs):
        """All layers of one chunk, eagerly.  qkv[l] = (q, k, v), outs[l] = attention output."""
        for layer in range(self.n_layers):
            q, k, v = qkv[layer]
            self.layer_step(layer, start_frame, q, k, v, q_rot[layer], outs[layer])

    def chunk_graph(self, start_frame: int, qkv, q_rot, outs):
        """A CUDA graph of chunk_step for this starting frame over these buffers (captured on
        first use).  Replaying it re-runs every layer on whatever the buffers hold then.

        The graph holds the attention scratch of the stepper's capture stream: replay the graphs of
        a stepper one after the other (one stream), not concurrently, and capture them again after
        `shutdown()` of the library, which frees that scratch."""
        import torch
        key = int(start_frame)
        if key not in self._graphs:
            self.table(start_frame)                  # built outside the capture
            side = self._capture_stream
            side.wait_stream(torch.cuda.current_stream(self.device))
            with torch.cuda.stream(side):            # first call on this stream: scratch set-up
                self.chunk_step(start_frame, qkv, q_rot, outs)
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                self.chunk_step(start_frame, qkv, q_rot, outs)
            self._graphs[key] = graph
        return self._graphs[key]


def _bench(args):
    import torch
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    if root not in sys.path:
        sys.path.insert(0, root)
    import workloads as W

    wl = W.WORKLOADS[args.workload]
    sh = wl.shape
    abi = U.Shape.make(sh.batch, sh.heads, sh.chunk_frames, sh.grid_h, sh.grid_w, sh.ring_frames)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    stepper = ChunkStepper(abi, args.layers, wl.window_frames[-1], wl.sink_frames, wl.sink_attend, dev)
    gen = torch.Generator(device=dev).manual_seed(7)
    for ck, cv in zip(stepper.cache_k, stepper.cache_v):
        ck.copy_(torch.randn(ck.shape, generator=gen, device=dev))
        cv.copy_(torch.randn(cv.shape, generator=gen, device=dev))
    dims = (sh.batch, sh.chunk_tokens, sh.heads, sh.head_dim)
    qkv = [tuple(torch.randn(dims, generator=gen, device=dev).to(torch.bfloat16) for _ in range(3))
           for _ in range(args.layers)]
    q_rot = [torch.empty(dims, dtype=torch.bfloat16, device=dev) for _ in range(args.layers)]
    outs = [torch.empty(dims, dtype=torch.bfloat16, device=dev) for _ in range(args.layers)]
    start = wl.measured_starts[0]

    def timed(fn):
        for _ in range(3):
            fn()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0.record()
        for _ in range(args.steps):
            fn()
        t1.record()
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) * 1e3 / args.steps / args.layers

    eager_us = timed(lambda: stepper.chunk_step(start, qkv, q_rot, outs))
    eager_out = [o.clone() for o in outs]
    graph = stepper.chunk_graph(start, qkv, q_rot, outs)
    graph_us = timed(graph.replay)
    same = all(torch.equal(a.view(torch.int16), b.view(torch.int16)) for a, b in zip(eager_out, outs))
    print(json.dumps({"workload": args.workload, "layers": args.layers, "steps": args.steps,
                      "keys": wl.keys_attended(wl.window_frames[-1]),
                      "us_per_layer_chunk_eager": eager_us, "us_per_layer_chunk_graph": graph_us,
                      "graph_equals_eager": bool(same), "device_status": U.poll_status(),
                      "launches_per_chunk_step": 2 * args.layers}))


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=30)
    ap.add_argument("--workload", default="cfg2_sink9")
    ap.add_argument("--steps", type=int, default=20)
    _bench(ap.parse_args())
