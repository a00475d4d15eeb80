"""ctypes binding of libunstep.so: same names as the C ABI, argument marshalling only."""

from __future__ import annotations

import ctypes
from ctypes import c_char_p, c_double, c_float, c_int, c_int32, c_int64, c_void_p, POINTER

from . import build as _build

EXPORTS = ("unstep_rope_table", "unstep_rope_kv_append", "unstep_window_attn",
           "unstep_window_attn_noalloc", "unstep_rope_kv_append_sink", "unstep_window_attn_sink",
           "unstep_rmsnorm_rope_kv_append", "unstep_window_attn_plan", "unstep_attn_workers", "unstep_selftest_wait_limit", "unstep_shutdown", "unstep_strerror", "unstep_poll_status", "unstep_launch_count")


class UnstepError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class Shape(ctypes.Structure):
    """Mirror of unstep_shape_t."""
    _fields_ = [("batch", c_int32), ("heads", c_int32), ("head_dim", c_int32),
                ("chunk_frames", c_int32), ("grid_h", c_int32), ("grid_w", c_int32),
                ("ring_frames", c_int32), ("band_t", c_int32), ("band_h", c_int32),
                ("band_w", c_int32), ("rope_base", c_double)]

    @classmethod
    def make(cls, batch, heads, chunk_frames, grid_h, grid_w, ring_frames, head_dim=128,
             bands=(44, 42, 42), rope_base=10000.0):
        return cls(batch, heads, head_dim, chunk_frames, grid_h, grid_w, ring_frames,
                   bands[0], bands[1], bands[2], rope_base)

    @property
    def tokens_per_frame(self):
        return self.grid_h * self.grid_w

    @property
    def chunk_tokens(self):
        return self.chunk_frames * self.grid_h * self.grid_w


_lib = None


def lib() -> ctypes.CDLL:
    """Load (building first if stale) the CUDA library; raises if that is impossible."""
    global _lib
    if _lib is None:
        import os
        path = _build.build(variant=os.environ.get("UNSTEP_LIB_VARIANT", ""))
        L = ctypes.CDLL(path)
        L.unstep_rope_table.restype = c_int
        L.unstep_rope_table.argtypes = [POINTER(Shape), c_int32, c_void_p, c_void_p, c_void_p]
        L.unstep_rope_kv_append.restype = c_int
        L.unstep_rope_kv_append.argtypes = [POINTER(Shape), POINTER(c_int32), c_void_p, c_void_p,
                                            c_void_p, c_void_p, c_void_p, c_int64, c_void_p,
                                            c_void_p, c_void_p, c_void_p]
        L.unstep_window_attn.restype = c_int
        L.unstep_window_attn.argtypes = [POINTER(Shape), POINTER(c_int32), c_int32, c_void_p,
                                         c_void_p, c_void_p, c_void_p, c_void_p]
        L.unstep_window_attn_noalloc.restype = c_int
        L.unstep_window_attn_noalloc.argtypes = L.unstep_window_attn.argtypes
        L.unstep_rope_kv_append_sink.restype = c_int
        L.unstep_rope_kv_append_sink.argtypes = [POINTER(Shape), c_int32, POINTER(c_int32), c_void_p,
                                                 c_void_p, c_void_p, c_void_p, c_void_p, c_int64,
                                                 c_void_p, c_void_p, c_void_p, c_void_p]
        L.unstep_window_attn_sink.restype = c_int
        L.unstep_window_attn_sink.argtypes = [POINTER(Shape), c_int32, POINTER(c_int32), c_int32, c_int32,
                                              c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.unstep_rmsnorm_rope_kv_append.restype = c_int
        L.unstep_rmsnorm_rope_kv_append.argtypes = [POINTER(Shape), c_int32, POINTER(c_int32), c_void_p,
                                                    c_void_p, c_void_p, c_void_p, c_void_p, c_float,
                                                    c_void_p, c_void_p, c_int64, c_void_p, c_void_p,
                                                    c_void_p, c_void_p]
        L.unstep_window_attn_plan.restype = c_int
        L.unstep_window_attn_plan.argtypes = [POINTER(Shape), c_int32, POINTER(c_int32), c_int32, c_int32,
                                              c_int32, POINTER(c_int32), c_int32, POINTER(c_int32)]
        L.unstep_attn_workers.restype = c_int
        L.unstep_attn_workers.argtypes = [POINTER(c_int32), POINTER(c_int32)]
        L.unstep_selftest_wait_limit.restype = c_int
        L.unstep_selftest_wait_limit.argtypes = [c_int64, c_void_p]
        L.unstep_shutdown.restype = None
        L.unstep_shutdown.argtypes = []
        L.unstep_strerror.restype = c_char_p
        L.unstep_strerror.argtypes = [c_int]
        L.unstep_poll_status.restype = c_int
        L.unstep_poll_status.argtypes = []
        L.unstep_launch_count.restype = c_int64
        L.unstep_launch_count.argtypes = []
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().unstep_strerror(int(code)).decode()


def _stream_ptr(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return c_void_p(int(getattr(stream, "cuda_stream", stream)))


def _dev_ptr(t, dtype, numel, name):
    import torch
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name}: expected a CUDA tensor")
    if t.dtype != dtype or not t.is_contiguous() or t.numel() != numel:
        raise ValueError(f"{name}: expected contiguous {dtype} with {numel} elements, got "
                         f"{t.dtype} {tuple(t.shape)}")
    return c_void_p(t.data_ptr())


def _starts(shape: Shape, start_frame):
    vals = [int(s) for s in start_frame]
    if len(vals) != shape.batch:
        raise ValueError("start_frame needs one entry per stream")
    return (c_int32 * len(vals))(*vals)


def _check(rc: int, where: str):
    if rc != 0:
        raise UnstepError(rc, where)


def rope_table(shape: Shape, start_frame: int, cos, sin, stream=None):
    """unstep_rope_table: fill float32 cos/sin [L, 64] for the chunk starting at start_frame."""
    import torch
    n = shape.chunk_tokens * 64
    _check(lib().unstep_rope_table(ctypes.byref(shape), int(start_frame),
                                   _dev_ptr(cos, torch.float32, n, "cos"),
                                   _dev_ptr(sin, torch.float32, n, "sin"), _stream_ptr(stream)),
           "unstep_rope_table")


def rope_kv_append(shape: Shape, start_frame, q_in, k_in, v_in, cos, sin, q_out, ring_k, ring_v,
                   table_stream_stride: int = 0, stream=None):
    """unstep_rope_kv_append: rotate q/k, write k/v of the chunk into ring slots."""
    import torch
    bf = torch.bfloat16
    n = shape.batch * shape.chunk_tokens * shape.heads * shape.head_dim
    nr = shape.batch * shape.ring_frames * shape.tokens_per_frame * shape.heads * shape.head_dim
    ntab = shape.chunk_tokens * 64 + (shape.batch - 1) * int(table_stream_stride)
    _check(lib().unstep_rope_kv_append(
        ctypes.byref(shape), _starts(shape, start_frame), _dev_ptr(q_in, bf, n, "q_in"),
        _dev_ptr(k_in, bf, n, "k_in"), _dev_ptr(v_in, bf, n, "v_in"),
        _dev_ptr(cos, torch.float32, ntab, "cos"), _dev_ptr(sin, torch.float32, ntab, "sin"),
        int(table_stream_stride), _dev_ptr(q_out, bf, n, "q_out"),
        _dev_ptr(ring_k, bf, nr, "ring_k"), _dev_ptr(ring_v, bf, nr, "ring_v"),
        _stream_ptr(stream)), "unstep_rope_kv_append")


def window_attn(shape: Shape, start_frame, window_frames: int, q_rot, ring_k, ring_v, out,
                stream=None):
    """unstep_window_attn: attention of the chunk's queries over the retained window."""
    import torch
    bf = torch.bfloat16
    n = shape.batch * shape.chunk_tokens * shape.heads * shape.head_dim
    nr = shape.batch * shape.ring_frames * shape.tokens_per_frame * shape.heads * shape.head_dim
    _check(lib().unstep_window_attn(
        ctypes.byref(shape), _starts(shape, start_frame), int(window_frames),
        _dev_ptr(q_rot, bf, n, "q_rot"), _dev_ptr(ring_k, bf, nr, "ring_k"),
        _dev_ptr(ring_v, bf, nr, "ring_v"), _dev_ptr(out, bf, n, "out"), _stream_ptr(stream)),
        "unstep_window_attn")


def window_attn_noalloc(shape: Shape, start_frame, window_frames: int, q_rot, ring_k, ring_v, out,
                        stream=None):
    """unstep_window_attn_noalloc: the same attention for callers that must not allocate device
    memory (a process whose memory is owned by a framework allocator, a latency-critical loop,
    a deployment with a fixed footprint).  Its scratch is a fixed ~40 MB array inside the
    library; all calls on a device share it, so calls that may overlap on the GPU must be
    serialised by the caller.  Raises UnstepError(-5) when the problem exceeds the array."""
    import torch
    bf = torch.bfloat16
    n = shape.batch * shape.chunk_tokens * shape.heads * shape.head_dim
    nr = shape.batch * shape.ring_frames * shape.tokens_per_frame * shape.heads * shape.head_dim
    _check(lib().unstep_window_attn_noalloc(
        ctypes.byref(shape), _starts(shape, start_frame), int(window_frames),
        _dev_ptr(q_rot, bf, n, "q_rot"), _dev_ptr(ring_k, bf, nr, "ring_k"),
        _dev_ptr(ring_v, bf, nr, "ring_v"), _dev_ptr(out, bf, n, "out"), _stream_ptr(stream)),
        "unstep_window_attn_noalloc")


def rope_kv_append_sink(shape: Shape, sink_frames: int, start_frame, q_in, k_in, v_in, cos, sin, q_out,
                        cache_k, cache_v, table_stream_stride: int = 0, stream=None):
    """unstep_rope_kv_append_sink: the append with a sink prefix of `sink_frames` slots."""
    import torch
    bf = torch.bfloat16
    n = shape.batch * shape.chunk_tokens * shape.heads * shape.head_dim
    nr = (shape.batch * (shape.ring_frames + int(sink_frames)) * shape.tokens_per_frame * shape.heads
          * shape.head_dim)
    ntab = shape.chunk_tokens * 64 + (shape.batch - 1) * int(table_stream_stride)
    _check(lib().unstep_rope_kv_append_sink(
        ctypes.byref(shape), int(sink_frames), _starts(shape, start_frame),
        _dev_ptr(q_in, bf, n, "q_in"), _dev_ptr(k_in, bf, n, "k_in"), _dev_ptr(v_in, bf, n, "v_in"),
        _dev_ptr(cos, torch.float32, ntab, "cos"), _dev_ptr(sin, torch.float32, ntab, "sin"),
        int(table_stream_stride), _dev_ptr(q_out, bf, n, "q_out"), _dev_ptr(cache_k, bf, nr, "cache_k"),
        _dev_ptr(cache_v, bf, nr, "cache_v"), _stream_ptr(stream)), "unstep_rope_kv_append_sink")


def rmsnorm_rope_kv_append(shape: Shape, sink_frames: int, start_frame, q_in, k_in, v_in, gain_q, gain_k,
                           eps: float, cos, sin, q_out, cache_k, cache_v, table_stream_stride: int = 0,
                           stream=None):
    """unstep_rmsnorm_rope_kv_append: RMSNorm of q and k, rotation and cache write in one kernel."""
    import torch
    bf = torch.bfloat16
    n = shape.batch * shape.chunk_tokens * shape.heads * shape.head_dim
    nr = (shape.batch * (shape.ring_frames + int(sink_frames)) * shape.tokens_per_frame * shape.heads
          * shape.head_dim)
    ntab = shape.chunk_tokens * 64 + (shape.batch - 1) * int(table_stream_stride)
    ng = shape.heads * shape.head_dim
    _check(lib().unstep_rmsnorm_rope_kv_append(
        ctypes.byref(shape), int(sink_frames), _starts(shape, start_frame),
        _dev_ptr(q_in, bf, n, "q_in"), _dev_ptr(k_in, bf, n, "k_in"), _dev_ptr(v_in, bf, n, "v_in"),
        _dev_ptr(gain_q, torch.float32, ng, "gain_q"), _dev_ptr(gain_k, torch.float32, ng, "gain_k"),
        c_float(eps), _dev_ptr(cos, torch.float32, ntab, "cos"), _dev_ptr(sin, torch.float32, ntab, "sin"),
        int(table_stream_stride), _dev_ptr(q_out, bf, n, "q_out"), _dev_ptr(cache_k, bf, nr, "cache_k"),
        _dev_ptr(cache_v, bf, nr, "cache_v"), _stream_ptr(stream)), "unstep_rmsnorm_rope_kv_append")


def window_attn_sink(shape: Shape, sink_frames: int, start_frame, recent_frames: int, sink_attend: int,
                     q_rot, cache_k, cache_v, out, stream=None):
    """unstep_window_attn_sink: attention over sink frames + the recent window."""
    import torch
    bf = torch.bfloat16
    n = shape.batch * shape.chunk_tokens * shape.heads * shape.head_dim
    nr = (shape.batch * (shape.ring_frames + int(sink_frames)) * shape.tokens_per_frame * shape.heads
          * shape.head_dim)
    _check(lib().unstep_window_attn_sink(
        ctypes.byref(shape), int(sink_frames), _starts(shape, start_frame), int(recent_frames),
        int(sink_attend), _dev_ptr(q_rot, bf, n, "q_rot"), _dev_ptr(cache_k, bf, nr, "cache_k"),
        _dev_ptr(cache_v, bf, nr, "cache_v"), _dev_ptr(out, bf, n, "out"), _stream_ptr(stream)),
        "unstep_window_attn_sink")


def window_attn_plan(shape: Shape, start_frame, recent_frames: int, max_workers: int, sink_frames: int = 0,
                     sink_attend: int = 0):
    """unstep_window_attn_plan: the segments of one attention launch as rows of 10 ints (worker,
    stream, head, query pair, query tiles, first key tile, end key tile, tiles of the item, parts,
    scratch slot).  Host only."""
    n = c_int32(0)
    starts = _starts(shape, start_frame)
    args = (ctypes.byref(shape), int(sink_frames), starts, int(recent_frames), int(sink_attend),
            int(max_workers))
    _check(lib().unstep_window_attn_plan(*args, None, 0, ctypes.byref(n)), "unstep_window_attn_plan")
    buf = (c_int32 * (10 * max(n.value, 1)))()
    _check(lib().unstep_window_attn_plan(*args, buf, n.value, ctypes.byref(n)), "unstep_window_attn_plan")
    return [tuple(buf[10 * i:10 * i + 10]) for i in range(n.value)]


def attn_workers():
    """unstep_attn_workers: (workers of a full-size attention launch, thread blocks per worker)."""
    a, b = c_int32(0), c_int32(0)
    _check(lib().unstep_attn_workers(ctypes.byref(a), ctypes.byref(b)), "unstep_attn_workers")
    return a.value, b.value


def selftest_wait_limit(limit_cycles: int, stream=None):
    """unstep_selftest_wait_limit: make a bounded device-side wait run out (diagnostic)."""
    _check(lib().unstep_selftest_wait_limit(int(limit_cycles), _stream_ptr(stream)),
           "unstep_selftest_wait_limit")


def shutdown():
    """unstep_shutdown: free the scratch buffers the attention calls created."""
    lib().unstep_shutdown()


def poll_status() -> int:
    return int(lib().unstep_poll_status())


def launch_count() -> int:
    return int(lib().unstep_launch_count())
