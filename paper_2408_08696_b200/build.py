"""Builds the CUDA shared libraries in-tree with nvcc for sm_100a (no JIT cache, no torch extension)."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
INCLUDE = os.path.join(ROOT, "include")

LIB_TR = os.path.join(PKG, "libtr.so")
LIB_SYNTH = os.path.join(PKG, "libtr_synth.so")

TR_SOURCES = ["tr_api.cu", "topk.cu", "topk_noalloc.cu", "tail.cu", "attn_tc.cu", "attn_pair.cu", "commit.cu", "lm_head.cu"]
SYNTH_SOURCES = ["synth.cu"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared", "-I", INCLUDE, "-I", CSRC,
]


def _nvcc():
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found; the CUDA libraries cannot be built")
    return exe


def _stale(lib, sources):
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in sources] + [
        os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))
    ] + [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force=False, verbose=False, extra=()):
    for lib, sources in ((LIB_TR, TR_SOURCES), (LIB_SYNTH, SYNTH_SOURCES)):
        if not force and not _stale(lib, sources):
            continue
        cmd = [_nvcc(), *NVCC_FLAGS, *extra, "-o", lib] + [os.path.join(CSRC, s) for s in sources]
        if verbose:
            print(" ".join(cmd), flush=True)
        subprocess.run(cmd, check=True)
    return LIB_TR, LIB_SYNTH


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose=True,
          extra=("-Xptxas", "-v") if "--ptxas" in sys.argv else ())
