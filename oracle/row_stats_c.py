"""ctypes loader for the C restatement of the oracle's per-row statistics.

Test infrastructure only (see row_stats.c).  `build()` compiles the single C
file with gcc; `row_stats_batch` runs it over all rows of a logits tensor and
returns (m, t, s) shaped like the leading dimensions, ready for
`csd_oracle.verify(..., stats=...)`.
"""

from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "row_stats.c")
_LIB = os.path.join(_HERE, "libcsd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.csd_oracle_row_stats.restype = ctypes.c_int
        lib.csd_oracle_row_stats.argtypes = [
            ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
        lib.csd_oracle_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().csd_oracle_max_threads())


def row_stats_batch(z: np.ndarray, is_bf16_bits: bool = False, n_threads: int = 0):
    """z: C-contiguous [..., V] array of float32, or of uint16/int16 bf16 bit patterns."""
    lib = _load()
    z = np.ascontiguousarray(z)
    if is_bf16_bits:
        assert z.dtype.itemsize == 2
        dtype = 1
    else:
        assert z.dtype == np.float32
        dtype = 0
    lead, V = z.shape[:-1], z.shape[-1]
    rows = int(np.prod(lead)) if lead else 1
    offs = (np.arange(rows, dtype=np.int64) * V)
    m = np.empty(rows, dtype=np.float64)
    t = np.empty(rows, dtype=np.int64)
    s = np.empty(rows, dtype=np.float64)
    nt = n_threads if n_threads > 0 else max_threads()
    scratch = np.empty(nt * V, dtype=np.float64)
    rc = lib.csd_oracle_row_stats(z.ctypes.data, dtype, rows, V, offs.ctypes.data,
                                  m.ctypes.data, t.ctypes.data, s.ctypes.data,
                                  scratch.ctypes.data, nt)
    if rc != 0:
        raise RuntimeError("csd_oracle_row_stats failed")
    return m.reshape(lead), t.reshape(lead), s.reshape(lead)
