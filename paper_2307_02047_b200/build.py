"""Builds the C-ABI CUDA library in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_HERE, "csrc", "came_api.cu")
DEPS = [SRC] + [os.path.join(_HERE, "csrc", h) for h in
                ("came_kernels.cuh", "came_pipelined.cuh", "came_stream.cuh")] + \
       [os.path.join(os.path.dirname(_HERE), "include", "came_b200.h")]
LIB = os.path.join(_HERE, "libcame_b200.so")
LIB_DEBUG = os.path.join(_HERE, "libcame_b200_debug.so")     # -DCAME_DEBUG_BOUNDS (see the header)

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "--cudart", "static"]


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(d) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile ``libcame_b200.so`` (or, with ``debug``, the bounds-checking
    ``libcame_b200_debug.so``) next to this file if it is missing or stale."""
    lib = LIB_DEBUG if debug else LIB
    if force or needs_build(lib):
        nvcc = os.environ.get("NVCC", "nvcc")
        cmd = [nvcc] + NVCC_FLAGS + (["-DCAME_DEBUG_BOUNDS"] if debug else []) + \
              (["-Xptxas", "-v"] if verbose else []) + ["-o", lib, SRC]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
        if verbose:
            print(res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose=True))
