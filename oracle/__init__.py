"""CPU oracle for the UnStep chunk-attention hot path.

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain definition of what
the CUDA library must compute.  It is imported by the test-suite, by the smoke
check and by the CPU-baseline leg of the benchmark, and by nothing else.  It
shares no code, table or constant with the CUDA path and never imports it.
"""

from . import unstep_oracle  # noqa: F401
from .unstep_oracle import (  # noqa: F401
    HEAD_DIM,
    N_PAIRS,
    band_pairs,
    band_frequencies,
    token_positions,
    rope_angles,
    rope_table,
    rope_rotate,
    rope_rotate_f64,
    RingState,
    rope_kv_append,
    window_frames_range,
    gather_window_ring,
    attention_rows,
    attention_bruteforce,
    window_attn,
    ExplicitHistory,
    explicit_window_attn,
    bf16_bits_to_f32,
    f32_to_bf16_bits_rne,
    sink_slot,
    sink_window_frames,
    SinkRingState,
    rope_kv_append_sink,
    window_attn_sink,
    explicit_frames_attn,
    rmsnorm_tokens,
    rmsnorm_rope_kv_append,
)
