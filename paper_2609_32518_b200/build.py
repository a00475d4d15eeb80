"""Builds libunstep.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""

from __future__ import annotations

import os
import shutil
import subprocess

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB_PATH = os.path.join(PKG_DIR, "libunstep.so")
SOURCES = ["api.cu", "rope.cu", "attn.cu"]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: cannot build libunstep.so")


def _inputs():
    files = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    files += [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE)]
    return files


# Diagnostic variants of the library, built beside the normal one as libunstep_<name>.so and
# loaded instead of it when the environment variable UNSTEP_LIB_VARIANT names one.
VARIANTS = {
    "check": ["-DUNSTEP_CHECK"],
    "abl3": ["-DNORM_ABL=3"],   # every global store bounds-checked, violations reported, never made
}


def lib_path(variant: str = "") -> str:
    return LIB_PATH if not variant else os.path.join(PKG_DIR, f"libunstep_{variant}.so")


def is_stale(variant: str = "") -> bool:
    path = lib_path(variant)
    if not os.path.exists(path):
        return True
    built = os.path.getmtime(path)
    return any(os.path.getmtime(f) > built for f in _inputs())


def build(force: bool = False, verbose: bool = False, variant: str = "") -> str:
    """Compile the library (or a diagnostic variant of it) if it is missing or older than its
    sources; return its path."""
    if variant and variant not in VARIANTS:
        raise ValueError(f"unknown library variant {variant!r}")
    path = lib_path(variant)
    if not force and not is_stale(variant):
        return path
    extra = os.environ.get("UNSTEP_NVCC_FLAGS", "").split()  # e.g. -DUNSTEP_TRACE for a debug build
    extra += VARIANTS.get(variant, [])
    cmd = [_nvcc()] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + [
        "-I", INCLUDE, "-I", CSRC, "-o", path + ".tmp"] + [os.path.join(CSRC, s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    os.replace(path + ".tmp", path)
    if verbose:
        print(res.stderr)
    return path


if __name__ == "__main__":
    print(build(force=True, verbose=True))
