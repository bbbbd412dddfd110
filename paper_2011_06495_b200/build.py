"""Builds the CUDA library in-tree with nvcc for sm_100a (no JIT cache, no pip install)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "csrc", "mv_sparse.cu")
SRCS = [SRC, os.path.join(HERE, "csrc", "mv_wire.cu")]
HDRS = [os.path.join(os.path.dirname(HERE), "include", h) for h in ("mv_sparse.h", "mv_wire.h")]
LIB = os.path.join(HERE, "libmvsparse.so")
LIB_DEBUG = os.path.join(HERE, "libmvsparse_debug.so")      # the checked build (-DMV_DEBUG), see mv_debug_status

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-lineinfo",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-Xcompiler", "-fPIC", "-shared",
    # IEEE arithmetic: no fast-math, denormals kept, so acc = err + grads matches any IEEE host
    "-ftz=false", "-prec-div=true", "-fmad=false",
]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(f) > t for f in (*SRCS, *HDRS, os.path.abspath(__file__)))


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compiles the library; debug=True compiles the checked variant (device-side bounds checks that set
    status bits instead of clamping silently) into libmvsparse_debug.so."""
    lib = LIB_DEBUG if debug else LIB
    if not force and not needs_build(lib):
        return lib
    cmd = [nvcc_path(), *NVCC_FLAGS, *(["-DMV_DEBUG"] if debug else []), "-o", lib, *SRCS]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed building libmvsparse.so")
    if verbose:
        print(res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
