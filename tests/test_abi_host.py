"""Host-side checks of the C ABI that need no GPU: the library builds and loads,
exports every function the header declares, and rejects bad arguments before it
touches a device."""

import ctypes
import os
import re

import pytest

import paper_2609_32518_b200 as U

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE = 0x10000  # a non-null, 16-byte aligned address that is never dereferenced


def declared_functions():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        text = re.sub(r"#ifdef UNSTEP_(TRACE|CHECK).*?#endif", "", text, flags=re.S)   # diagnostic builds only
        names |= set(re.findall(r"\b(unstep_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_function():
    lib = U.lib()
    declared = declared_functions()
    assert {"unstep_rope_table", "unstep_rope_kv_append", "unstep_window_attn"} <= declared
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in include/ but not exported"
    assert set(U.EXPORTS) <= declared


def test_strerror_and_counter():
    assert U.strerror(0) == "ok"
    assert "invalid" in U.strerror(-1) and "128" in U.strerror(-2)
    assert "CUDA" in U.strerror(-3) and "wait" in U.strerror(-4)
    assert U.strerror(-99) == "unknown status"
    assert U.launch_count() >= 0


def good_shape(**kw):
    args = dict(batch=1, heads=2, chunk_frames=2, grid_h=8, grid_w=8, ring_frames=6)
    args.update(kw)
    return U.Shape.make(**args)


def call_table(shape, start=0, cos=FAKE, sin=FAKE):
    return U.lib().unstep_rope_table(ctypes.byref(shape), start, cos, sin, None)


def call_append(shape, starts=(0,), ptrs=None, stride=0):
    p = [FAKE] * 8 if ptrs is None else ptrs
    arr = (ctypes.c_int32 * len(starts))(*starts) if starts is not None else None
    return U.lib().unstep_rope_kv_append(ctypes.byref(shape), arr, p[0], p[1], p[2], p[3], p[4],
                                         stride, p[5], p[6], p[7], None)


def call_attn(shape, starts=(0,), wf=2, ptrs=None):
    p = [FAKE] * 4 if ptrs is None else ptrs
    arr = (ctypes.c_int32 * len(starts))(*starts) if starts is not None else None
    return U.lib().unstep_window_attn(ctypes.byref(shape), arr, wf, p[0], p[1], p[2], p[3], None)


INVALID, UNSUPPORTED = -1, -2


@pytest.mark.parametrize("kw", [dict(chunk_frames=0), dict(grid_h=0), dict(grid_w=-3),
                                dict(bands=(43, 43, 42)), dict(bands=(44, 42, 40)),
                                dict(bands=(0, 64, 64)), dict(rope_base=0.0), dict(head_dim=0)])
def test_bad_shapes_are_rejected_everywhere(kw):
    sh = good_shape(**kw)
    assert call_table(sh) == INVALID
    assert call_append(sh) == INVALID
    assert call_attn(sh) == INVALID


def test_head_dim_other_than_128_is_unsupported():
    sh = good_shape(head_dim=64, bands=(22, 21, 21))
    assert call_table(sh) == UNSUPPORTED
    assert call_attn(good_shape(head_dim=256)) == UNSUPPORTED


def test_table_argument_checks():
    sh = good_shape()
    assert call_table(sh, start=-1) == INVALID
    assert call_table(sh, cos=None) == INVALID
    assert call_table(sh, sin=FAKE + 4) == INVALID
    assert U.lib().unstep_rope_table(None, 0, FAKE, FAKE, None) == INVALID


def test_append_argument_checks():
    sh = good_shape()
    for i in range(8):
        ptrs = [FAKE] * 8
        ptrs[i] = None
        assert call_append(sh, ptrs=ptrs) == INVALID
        ptrs[i] = FAKE + 8
        assert call_append(sh, ptrs=ptrs) == INVALID
    assert call_append(sh, starts=None) == INVALID
    assert call_append(sh, starts=(-1,)) == INVALID
    assert call_append(sh, stride=-4) == INVALID
    assert call_append(sh, stride=6) == INVALID
    for kw in (dict(batch=0), dict(heads=0), dict(ring_frames=0), dict(ring_frames=1)):
        assert call_append(good_shape(**kw)) == INVALID


def test_attn_argument_checks():
    sh = good_shape()
    for i in range(4):
        ptrs = [FAKE] * 4
        ptrs[i] = None
        assert call_attn(sh, ptrs=ptrs) == INVALID
        ptrs[i] = FAKE + 2
        assert call_attn(sh, ptrs=ptrs) == INVALID
    assert call_attn(sh, starts=None) == INVALID
    assert call_attn(sh, starts=(-2,)) == INVALID
    assert call_attn(sh, wf=1) == INVALID      # window shorter than the chunk
    assert call_attn(sh, wf=7) == INVALID      # window longer than the ring
    assert call_attn(sh, starts=(2 ** 31 - 1,)) == INVALID


def test_binding_refuses_cpu_tensors():
    import torch
    sh = good_shape()
    t = torch.zeros(128 * 64, dtype=torch.float32)
    with pytest.raises(TypeError):
        U.rope_table(sh, 0, t, t)
