"""Compiles the CUDA sources into ``libevo.so`` next to this file (sm_100a only)."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libevo.so")
LIB_DEBUG = os.path.join(HERE, "libevo_debug.so")     # checked build: -DEVO_DEBUG (bounds checks, guard words)
SOURCES = ["evo.cu", "solver_kernels.cu", "rollout_mlp.cu", "rollout_mlp_tiled.cu", "rollout_tl_tc.cu", "rollout_cnn.cu", "rollout_cnn_tc.cu", "gradient_static.cu", "rollout_s2s.cu", "rollout_paint.cu"]
HEADERS = ["internal.h", "noise.cuh", "tasks.cuh", "async.cuh", "umma.cuh", "fp32x2.cuh", os.path.join("..", "..", "include", "evo.h")]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; the CUDA library cannot be built")


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    files = [os.path.join(CSRC, s) for s in SOURCES] + [os.path.normpath(os.path.join(CSRC, h)) for h in HEADERS]
    return any(os.path.getmtime(f) > t for f in files)


def build_library(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = LIB_DEBUG if debug else LIB
    if not force and not is_stale(lib):
        return lib
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "--shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v" if verbose else "-O3"] + \
          (["-DEVO_DEBUG"] if debug else []) + ["-o", lib] + [os.path.join(CSRC, s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return lib


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv))
    print(build_library(force=True, debug=True))
