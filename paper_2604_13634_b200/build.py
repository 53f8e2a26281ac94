"""Build the C-ABI CUDA library in-tree for sm_100a (nvcc cross-compiles without a GPU)."""

from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libcsd.so")
LIB_DEBUG = os.path.join(HERE, "libcsd_debug.so")     # the same sources with -DCSD_DEBUG: every index checked
SOURCES = ["csd_api.cu"]
HEADERS = ["csd_common.cuh", "csd_ocm.cuh", "csd_step.cuh", "csd_sampled.cuh", "csd_lmhead.cuh", os.path.join("..", "..", "include", "csd.h")]

NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-shared", "-Xcompiler", "-fPIC", "--use_fast_math=false"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile the library (debug=True: the bounds-checked variant, loaded when CSD_DEBUG=1 is set)."""
    lib = LIB_DEBUG if debug else LIB
    if not force and not needs_build(lib):
        return lib
    flags = [f for f in NVCC_FLAGS if not f.startswith("--use_fast_math")]
    cmd = [_nvcc(), *flags, *(["-DCSD_DEBUG"] if debug else []), *(["-Xptxas", "-v"] if verbose else []), "-o", lib,
           *[os.path.join(CSRC, f) for f in SOURCES]]
    proc = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if verbose or proc.returncode != 0:
        sys.stderr.write(proc.stdout)
    if proc.returncode != 0:
        raise RuntimeError(f"nvcc failed building {os.path.basename(lib)}")
    return lib


if __name__ == "__main__":
    build(force=True, verbose=True)
    build(force=True, debug=True)
    print(LIB, LIB_DEBUG)
