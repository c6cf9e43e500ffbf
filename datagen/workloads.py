"""The five benchmark workloads as seeded arrays (host numpy, float64 / int32).

Shapes, distributions and seeds follow the five benchmark configurations; every
function takes the sizes as arguments so the same recipe serves the small
parity cases and the full-size runs.  Stream numbers name the arrays of one
workload: 0 = X (CSR: 0 positions, 1 values), 2 = Y / v / U, 3 = Z / w / V.
"""
from __future__ import annotations

import numpy as np


def _gen():
    import datagen
    return datagen


def cell_workload(rows=1000, cols=1000, seed=0):
    """sum(X*Y*Z): three dense uniform[0,1) matrices."""
    g = _gen()
    n = rows * cols
    return {
        "X": g.uniform(seed, 0, n).reshape(rows, cols),
        "Y": g.uniform(seed, 2, n).reshape(rows, cols),
        "Z": g.uniform(seed, 3, n).reshape(rows, cols),
    }


def magg_workload(rows=1_000_000, cols=100, seed=1, out=None):
    """(sum(X*Y), sum(X*Z), sum(X*X)): three dense N(0,1) matrices.

    `out`, if given, maps "X"/"Y"/"Z" to preallocated flat float64 arrays
    (e.g. views of pinned host buffers) that receive the values.
    """
    g = _gen()
    n = rows * cols
    out = out or {}
    return {
        "X": g.normal(seed, 0, n, out=out.get("X")).reshape(rows, cols),
        "Y": g.normal(seed, 2, n, out=out.get("Y")).reshape(rows, cols),
        "Z": g.normal(seed, 3, n, out=out.get("Z")).reshape(rows, cols),
    }


def row_dense_workload(rows=1_000_000, cols=1000, seed=2, out=None):
    """t(X) %*% (w * (X %*% v)): X dense N(0,1), v N(0,1), w uniform[0,1)."""
    g = _gen()
    out = out or {}
    return {
        "X": g.normal(seed, 0, rows * cols, out=out.get("X")).reshape(rows, cols),
        "v": g.normal(seed, 2, cols, out=out.get("v")),
        "w": g.uniform(seed, 3, rows, out=out.get("w")),
    }


def row_csr_workload(rows=10_000_000, cols=1000, density=0.01, seed=3):
    """Same expression with X in CSR: Bernoulli(density) cells, values uniform[0,1)."""
    g = _gen()
    rowptr, colidx, vals = g.csr_bernoulli(seed, 0, rows, cols, density, 0.0, 1.0)
    return {
        "rows": rows, "cols": cols,
        "rowptr": rowptr, "colidx": colidx, "vals": vals,
        "v": g.normal(seed, 2, cols),
        "w": g.uniform(seed, 3, rows),
    }


def outer_workload(rows=100_000, cols=100_000, rank=100, density=0.001, seed=4):
    """sum((X != 0) * (X - U %*% t(V))^2): X CSR with values uniform[1,5),
    U (rows x rank) and V (cols x rank) dense N(0, std 0.1)."""
    g = _gen()
    rowptr, colidx, vals = g.csr_bernoulli(seed, 0, rows, cols, density, 1.0, 5.0)
    return {
        "rows": rows, "cols": cols, "rank": rank,
        "rowptr": rowptr, "colidx": colidx, "vals": vals,
        "U": g.normal(seed, 2, rows * rank, 0.0, 0.1).reshape(rows, rank),
        "V": g.normal(seed, 3, cols * rank, 0.0, 0.1).reshape(cols, rank),
    }


def row_b1_workload(rows=1_000_000, cols=1000, k=2, seed=5, out=None):
    """Row template with a matrix-valued row intermediate: X dense N(0,1)
    (rows x cols), V dense N(0,1) (cols x k), and P (rows x k) uniform[0, 1/(k+1))
    - entries shaped like the first k of k+1 class probabilities, so that a
    row of P sums to less than one."""
    g = _gen()
    out = out or {}
    return {
        "X": g.normal(seed, 0, rows * cols, out=out.get("X")).reshape(rows, cols),
        "V": g.normal(seed, 2, cols * k).reshape(cols, k),
        "P": g.uniform(seed, 3, rows * k, 0.0, 1.0 / (k + 1), out=out.get("P")).reshape(rows, k),
    }


def csr_to_dense(rows, cols, rowptr, colidx, vals):
    """Scatter a CSR matrix into a dense array (format conversion only)."""
    d = np.zeros((rows, cols), dtype=np.float64)
    rid = np.repeat(np.arange(rows), np.diff(rowptr.astype(np.int64)))
    d[rid, colidx] = vals
    return d
