"""B200 (sm_100a) chunk-attention hot path of a causal video DiT: RoPE table,
fused RoPE + KV-ring append, windowed attention.  All computation happens in the
CUDA library behind the C ABI declared in include/unstep.h; this package only
marshals arguments.  There is no CPU fallback: without the library or a GPU the
calls raise."""

from .binding import (  # noqa: F401
    UnstepError,
    Shape,
    lib,
    rope_table,
    rope_kv_append,
    window_attn,
    window_attn_noalloc,
    rope_kv_append_sink,
    window_attn_sink,
    rmsnorm_rope_kv_append,
    window_attn_plan,
    attn_workers,
    poll_status,
    shutdown,
    selftest_wait_limit,
    launch_count,
    strerror,
    EXPORTS,
)
