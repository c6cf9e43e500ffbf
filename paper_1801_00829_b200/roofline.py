"""Roofline arithmetic of the fused operators (host side).

The minimal traffic of a fused operator is every input read once plus the
output written once; the time bound is bytes / bandwidth, the form the paper's
cost model uses for read and write times (Section 4.3).
"""
from __future__ import annotations


def ideal_seconds(nbytes: float, gb_per_s: float) -> float:
    """Time to move nbytes at gb_per_s (1 GB = 1e9 bytes)."""
    return float(nbytes) / (float(gb_per_s) * 1e9)


def algorithmic_bytes(template: str, **kw) -> int:
    """Bytes a fused operator must move once (inputs read once, output written).

    cell / magg: rows, cols, n_inputs (main + cell-shaped sides), n_out
    row_dense  : rows, cols                      (X, v, w; q out)
    row_csr    : rows, cols, nnz                 (vals, colidx, rowptr, w, v; q out)
    outer      : rows, cols, nnz, rank           (vals, colidx, rowptr, U, V; scalar out)
    """
    if template in ("cell", "magg"):
        return 8 * kw["rows"] * kw["cols"] * kw["n_inputs"] + 8 * kw.get("n_out", 1)
    if template == "row_dense":
        return 8 * kw["rows"] * kw["cols"] + 8 * kw["rows"] + 8 * kw["cols"] + 8 * kw["cols"]
    if template == "row_csr":
        return (12 * kw["nnz"] + 4 * (kw["rows"] + 1) + 8 * kw["rows"] + 8 * kw["cols"]
                + 8 * kw["cols"])
    if template == "outer":
        return (12 * kw["nnz"] + 4 * (kw["rows"] + 1)
                + 8 * kw["rank"] * (kw["rows"] + kw["cols"]) + 8)
    raise ValueError(template)
