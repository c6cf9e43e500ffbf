"""Seeded synthetic inputs for the fused-operator workloads.

This package only *makes inputs*: uniform / normal dense arrays and random CSR
matrices, each value a pure function of (seed, stream, index).  It contains none
of the fused-operator arithmetic, and is the one piece shared by the CUDA path's
tests and benchmarks and by the CPU checker, so both always read identical bytes.

The generator is a small C library (``gen.c``, built on demand with gcc); see the
header of that file for the exact definition of every draw.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB_PATH = os.path.join(_HERE, "libdatagen.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile gen.c into libdatagen.so next to it (no-op when up to date)."""
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC)):
        return _LIB_PATH
    tmp = _LIB_PATH + ".tmp%d" % os.getpid()
    cmd = ["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-fno-fast-math",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            i64, u64, f64 = ctypes.c_int64, ctypes.c_uint64, ctypes.c_double
            p = ctypes.c_void_p
            lib.dg_uniform.argtypes = [u64, u64, i64, i64, f64, f64, p]
            lib.dg_normal.argtypes = [u64, u64, i64, i64, f64, f64, p]
            lib.dg_csr_count.argtypes = [u64, u64, i64, i64, i64, f64, p]
            lib.dg_csr_fill.argtypes = [u64, u64, i64, i64, i64, f64, f64, f64, p, p, p]
            for f in (lib.dg_uniform, lib.dg_normal, lib.dg_csr_count, lib.dg_csr_fill):
                f.restype = None
            _lib = lib
    return _lib


def _out(count, out):
    if out is None:
        return np.empty(count, dtype=np.float64)
    assert out.dtype == np.float64 and out.flags.c_contiguous and out.size == count
    return out


def uniform(seed, stream, count, lo=0.0, hi=1.0, offset=0, out=None):
    """Elements [offset, offset+count) of the uniform[lo, hi) array (seed, stream)."""
    out = _out(count, out)
    _load().dg_uniform(seed, stream, offset, count, lo, hi, out.ctypes.data)
    return out


def normal(seed, stream, count, mean=0.0, std=1.0, offset=0, out=None):
    """Elements [offset, offset+count) of the N(mean, std^2) array (seed, stream)."""
    out = _out(count, out)
    _load().dg_normal(seed, stream, offset, count, mean, std, out.ctypes.data)
    return out


def csr_bernoulli(seed, stream, rows, cols, density, lo=0.0, hi=1.0, row0=0):
    """Rows [row0, row0+rows) of a random CSR matrix with `cols` columns.

    Each cell is stored independently with probability `density`; stored values
    are uniform[lo, hi).  Returns (rowptr int32[rows+1], colidx int32[nnz],
    vals float64[nnz]); rowptr[0] == 0 and column indices ascend within a row.
    Uses streams `stream` (positions) and `stream + 1` (values).
    """
    lib = _load()
    counts = np.empty(rows, dtype=np.int64)
    lib.dg_csr_count(seed, stream, row0, rows, cols, density, counts.ctypes.data)
    rowptr64 = np.zeros(rows + 1, dtype=np.int64)
    np.cumsum(counts, out=rowptr64[1:])
    nnz = int(rowptr64[-1])
    if nnz >= 2 ** 31:
        raise ValueError("nnz does not fit int32 row offsets")
    colidx = np.empty(nnz, dtype=np.int32)
    vals = np.empty(nnz, dtype=np.float64)
    lib.dg_csr_fill(seed, stream, row0, rows, cols, density, lo, hi,
                    rowptr64.ctypes.data, colidx.ctypes.data, vals.ctypes.data)
    return rowptr64.astype(np.int32), colidx, vals


from .workloads import (  # noqa: E402
    cell_workload, magg_workload, row_dense_workload, row_csr_workload, outer_workload,
    row_b1_workload,
)

__all__ = [
    "build", "uniform", "normal", "csr_bernoulli",
    "cell_workload", "magg_workload", "row_dense_workload", "row_csr_workload",
    "outer_workload", "row_b1_workload",
]
