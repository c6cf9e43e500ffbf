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


def operator_cost(read_bytes: float, write_bytes: float, flops: float,
                  read_gb_per_s: float, write_gb_per_s: float, gflop_per_s: float) -> float:
    """Time estimate of one (basic or fused) operator in the form of the paper's cost
    model (Section 4.3): write time plus the larger of read and compute time, each
    a size divided by a peak rate."""
    t_w = float(write_bytes) / (float(write_gb_per_s) * 1e9)
    t_r = float(read_bytes) / (float(read_gb_per_s) * 1e9)
    t_c = float(flops) / (float(gflop_per_s) * 1e9)
    return t_w + max(t_r, t_c)


def operator_sizes(template: str, **kw):
    """(read bytes, write bytes, flops) of the five benchmark expressions as fused
    operators.  Sparsity-exploiting operators count stored cells only (the model
    scales by the sparsity of the main input, Section 4.3)."""
    if template == "cell":          # sum(X*Y*Z)
        cells = kw["rows"] * kw["cols"]
        return 8 * cells * 3, 8, 3 * cells
    if template == "magg":          # sum(X*Y), sum(X*Z), sum(X*X)
        cells = kw["rows"] * kw["cols"]
        return 8 * cells * 3, 24, 6 * cells
    if template == "row_dense":     # t(X) (w * (X v))
        cells = kw["rows"] * kw["cols"]
        return 8 * cells + 8 * kw["rows"] + 8 * kw["cols"], 8 * kw["cols"], 4 * cells + kw["rows"]
    if template == "row_csr":
        nnz = kw["nnz"]
        return (12 * nnz + 4 * (kw["rows"] + 1) + 8 * kw["rows"] + 8 * kw["cols"], 8 * kw["cols"],
                4 * nnz + kw["rows"])
    if template == "outer":         # sum((X != 0) * (X - U V^T)^2)
        nnz, rank = kw["nnz"], kw["rank"]
        return (12 * nnz + 4 * (kw["rows"] + 1) + 8 * rank * (kw["rows"] + kw["cols"]), 8,
                (2 * rank + 4) * nnz)
    raise ValueError(template)


def unfused_plan_sizes(template: str, **kw):
    """The same expressions as plans of basic operators with materialised
    intermediates: a list of (read bytes, write bytes, flops), one per operator
    (Fig. 1: what fusion removes)."""
    if template == "cell":          # T1 = X*Y ; T2 = T1*Z ; sum(T2)
        b = 8 * kw["rows"] * kw["cols"]
        c = kw["rows"] * kw["cols"]
        return [(2 * b, b, c), (2 * b, b, c), (b, 8, c)]
    if template == "magg":          # three times: T = X*S ; sum(T)
        b = 8 * kw["rows"] * kw["cols"]
        c = kw["rows"] * kw["cols"]
        return [(2 * b, b, c), (b, 8, c)] * 2 + [(b, b, c), (b, 8, c)]
    if template == "row_dense":     # t1 = X v ; t2 = w*t1 ; q = X^T t2
        b = 8 * kw["rows"] * kw["cols"]
        c = kw["rows"] * kw["cols"]
        m, n = 8 * kw["rows"], 8 * kw["cols"]
        return [(b + n, m, 2 * c), (2 * m, m, kw["rows"]), (b + m, n, 2 * c)]
    if template == "row_csr":
        x = 12 * kw["nnz"] + 4 * (kw["rows"] + 1)
        m, n = 8 * kw["rows"], 8 * kw["cols"]
        return [(x + n, m, 2 * kw["nnz"]), (2 * m, m, kw["rows"]), (x + m, n, 2 * kw["nnz"])]
    if template == "outer":         # P = U V^T ; D = X - P ; S = D*D ; W = X != 0 ; M = W*S ; sum(M)
        cells = kw["rows"] * kw["cols"]
        d = 8 * cells
        x = 12 * kw["nnz"] + 4 * (kw["rows"] + 1)
        uv = 8 * kw["rank"] * (kw["rows"] + kw["cols"])
        return [(uv, d, 2 * kw["rank"] * cells), (x + d, d, cells), (d, d, cells), (x, d, cells),
                (2 * d, d, cells), (d, 8, cells)]
    raise ValueError(template)


def plan_cost(operators, read_gb_per_s, write_gb_per_s, gflop_per_s) -> float:
    """Sum of operator_cost over a plan's operators (the paper's C(P | q))."""
    return sum(operator_cost(r, w, f, read_gb_per_s, write_gb_per_s, gflop_per_s) for r, w, f in operators)
