"""A stack of layers stepped chunk by chunk, eagerly and by CUDA-graph replay, against the oracle."""

import numpy as np
import pytest
import torch

import oracle as O
import paper_2609_32518_b200 as U
import workloads as W
from harness import abi_shape, attn_errors, to_bits, to_dev
from paper_2609_32518_b200.layer_loop import ChunkStepper

pytestmark = pytest.mark.gpu


def test_three_layers_four_chunks_two_calls_each_graph_replay_matches_oracle():
    sh = W.Shape(batch=1, heads=2, chunk_frames=3, grid_h=8, grid_w=25, ring_frames=6)
    n_layers, sink = 3, 3
    wls = [W.Workload(f"layer{l}", sh, seed=70 + l, history_starts=((),), measured_starts=(0,),
                      window_frames=(6,)) for l in range(n_layers)]
    stepper = ChunkStepper(abi_shape(sh), n_layers, window_frames=6, sink_frames=sink, sink_attend=3)
    for ck, cv in zip(stepper.cache_k, stepper.cache_v):          # NaN sentinels outside what gets written
        ck.view(torch.int16).fill_(0x7FC1)
        cv.view(torch.int16).fill_(0x7FC1)
    oracles = [O.SinkRingState(1, sink, 6, sh.tokens_per_frame, sh.heads) for _ in range(n_layers)]
    dims = (1, sh.chunk_tokens, sh.heads, 128)
    bufs = [tuple(torch.empty(dims, dtype=torch.bfloat16, device="cuda") for _ in range(3)) for _ in range(n_layers)]
    q_rot = [torch.empty(dims, dtype=torch.bfloat16, device="cuda") for _ in range(n_layers)]
    outs = [torch.empty(dims, dtype=torch.bfloat16, device="cuda") for _ in range(n_layers)]
    for chunk in range(4):
        s = 3 * chunk
        cos, sin = O.rope_table(s, 3, 8, 25)
        for call in range(2):                                      # noisy pass, then clean pass: overwrite
            refs = []
            for l in range(n_layers):
                q, k, v = W.batch_qkv(wls[l], [s], tag=call)
                for dst, src in zip(bufs[l], (q, k, v)):
                    dst.copy_(to_dev(src))
                q_ref = O.rope_kv_append_sink(oracles[l], [s], q, k, v, cos, sin)
                refs.append((q_ref, O.window_attn_sink(oracles[l], [s], 6, 3, q_ref, 3)))
            if call == 0:
                stepper.chunk_step(s, bufs, q_rot, outs)           # eager
            else:
                stepper.chunk_graph(s, bufs, q_rot, outs).replay() # captured on first use, then replayed
            torch.cuda.synchronize()
            for l in range(n_layers):
                assert np.array_equal(to_bits(q_rot[l]), refs[l][0])
                assert np.array_equal(to_bits(stepper.cache_k[l]), oracles[l].cache_k)
                assert np.array_equal(to_bits(stepper.cache_v[l]), oracles[l].cache_v)
                mx, mean, rel = attn_errors(to_bits(outs[l]), refs[l][1])
                assert mx <= 2e-2 and mean <= 2e-3 and rel <= 1.5e-2, (chunk, call, l, mx, mean, rel)
    assert U.poll_status() == 0
    assert len(stepper._tables) == 4                               # one table per starting frame, reused
