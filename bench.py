#!/usr/bin/env python
"""Benchmark of the fused-operator hot path.

A step is one pass of the whole path: the five fused operators (Cell, MAgg,
Row dense, Row CSR, Outer) each run once on their full-size seeded workload.
The reported value is effective input bandwidth: the bytes the five operators
must read once, divided by the time of a step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-paper-suite]

`--impl reference` times the CPU checker (oracle/) on bounded samples of the same
workloads; it runs on host cores only.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "effective_hbm_bandwidth_all_fused_ops"
UNIT = "GB/s"

XYZ = [("mul", "t0", "a", "side0"), ("mul", "t1", "t0", "side1")]
MAGG3 = [("mul", "t0", "a", "side0"), ("mul", "t1", "a", "side1"), ("mul", "t2", "a", "a")]
WD = [("mul", "t0", "side0", "d")]
WSLOSS = [("ne", "t0", "a", 0.0), ("sub", "t1", "a", "d"), ("mul", "t2", "t1", "t1"),
          ("mul", "t3", "t0", "t2")]

# dram__bytes_read.sum + dram__bytes_write.sum per unit of work, from the ncu captures summarised
# under profiles/ (row_dense: 200 000 x 1000 capture, per row; traffic grows in proportion to the
# rows).  A kernel that changed since its capture is listed as None.
NCU_DRAM_BYTES_PER_UNIT = {
    "cell": 24.014e6 / 1e6,                      # per cell (3 inputs)
    "magg": (480.018e6 + 3.727e6) / 2e7,         # per cell (3 inputs; 200 000 x 100 capture)
    "row_dense": (1601.696e6 + 7.937e6) / 2e5,   # per row of 1000 columns (200 000 x 1000 capture)
    "row_csr": (264.047e6 + 3.881e6) / 19998162, # per stored cell (2 000 000 x 1000 @ 0.01 capture)
    "outer": (1390.703e6 + 4.754e6) / 9996322,   # per stored cell (full-size capture, outer_bulk_kernel)
}

FULL = {
    "cell": dict(rows=1000, cols=1000),
    "magg": dict(rows=1_000_000, cols=100),
    "row_dense": dict(rows=1_000_000, cols=1000),
    "row_csr": dict(rows=10_000_000, cols=1000, density=0.01),
    "outer": dict(rows=100_000, cols=100_000, rank=100, density=0.001),
}
OPS = ["cell", "magg", "row_dense", "row_csr", "outer"]


def scaled(shapes, frac):
    """The same workloads with the row counts scaled by `frac` (columns, rank, density kept)."""
    out = {}
    for k, s in shapes.items():
        s = dict(s)
        if k != "cell":
            s["rows"] = max(8, int(round(s["rows"] * frac)))
        out[k] = s
    return out


# ---------------------------------------------------------------------- inputs
def make_host_inputs(shapes, pinned):
    """Seeded inputs of all five workloads as torch CPU tensors (pinned if asked)."""
    import torch
    import datagen

    def buf(n, dtype=torch.float64):
        return torch.empty(n, dtype=dtype, pin_memory=pinned)

    h = {}
    s = shapes["cell"]
    n = s["rows"] * s["cols"]
    for name, stream in (("X", 0), ("Y", 2), ("Z", 3)):
        t = buf(n)
        datagen.uniform(0, stream, n, out=t.numpy())
        h["cell." + name] = t.view(s["rows"], s["cols"])
    s = shapes["magg"]
    n = s["rows"] * s["cols"]
    for name, stream in (("X", 0), ("Y", 2), ("Z", 3)):
        t = buf(n)
        datagen.normal(1, stream, n, out=t.numpy())
        h["magg." + name] = t.view(s["rows"], s["cols"])
    s = shapes["row_dense"]
    t = buf(s["rows"] * s["cols"])
    datagen.normal(2, 0, s["rows"] * s["cols"], out=t.numpy())
    h["row_dense.X"] = t.view(s["rows"], s["cols"])
    h["row_dense.v"] = buf(s["cols"])
    datagen.normal(2, 2, s["cols"], out=h["row_dense.v"].numpy())
    h["row_dense.w"] = buf(s["rows"])
    datagen.uniform(2, 3, s["rows"], out=h["row_dense.w"].numpy())
    s = shapes["row_csr"]
    rp, ci, va = datagen.csr_bernoulli(3, 0, s["rows"], s["cols"], s["density"], 0.0, 1.0)
    for name, arr, dt in (("rowptr", rp, torch.int32), ("colidx", ci, torch.int32), ("vals", va, torch.float64)):
        t = buf(arr.size, dt)
        t.numpy()[:] = arr
        h["row_csr." + name] = t
    h["row_csr.v"] = buf(s["cols"])
    datagen.normal(3, 2, s["cols"], out=h["row_csr.v"].numpy())
    h["row_csr.w"] = buf(s["rows"])
    datagen.uniform(3, 3, s["rows"], out=h["row_csr.w"].numpy())
    s = shapes["outer"]
    rp, ci, va = datagen.csr_bernoulli(4, 0, s["rows"], s["cols"], s["density"], 1.0, 5.0)
    for name, arr, dt in (("rowptr", rp, torch.int32), ("colidx", ci, torch.int32), ("vals", va, torch.float64)):
        t = buf(arr.size, dt)
        t.numpy()[:] = arr
        h["outer." + name] = t
    t = buf(s["rows"] * s["rank"])
    datagen.normal(4, 2, s["rows"] * s["rank"], 0.0, 0.1, out=t.numpy())
    h["outer.U"] = t.view(s["rows"], s["rank"])
    t = buf(s["cols"] * s["rank"])
    datagen.normal(4, 3, s["cols"] * s["rank"], 0.0, 0.1, out=t.numpy())
    h["outer.V"] = t.view(s["cols"], s["rank"])
    return h


def algorithmic_bytes(shapes, host):
    from paper_1801_00829_b200 import algorithmic_bytes as ab
    s = shapes
    return {
        "cell": ab("cell", rows=s["cell"]["rows"], cols=s["cell"]["cols"], n_inputs=3),
        "magg": ab("magg", rows=s["magg"]["rows"], cols=s["magg"]["cols"], n_inputs=3, n_out=3),
        "row_dense": ab("row_dense", rows=s["row_dense"]["rows"], cols=s["row_dense"]["cols"]),
        "row_csr": ab("row_csr", rows=s["row_csr"]["rows"], cols=s["row_csr"]["cols"],
                      nnz=int(host["row_csr.vals"].numel())),
        "outer": ab("outer", rows=s["outer"]["rows"], cols=s["outer"]["cols"],
                    nnz=int(host["outer.vals"].numel()), rank=s["outer"]["rank"]),
    }


def upload(host, dev_bufs, stream_sync=False):
    """Copies every host tensor into its preallocated device tensor (async on the current stream)."""
    for k, t in host.items():
        dev_bufs[k].copy_(t, non_blocking=True)


def alloc_device(host, device):
    import torch
    return {k: torch.empty(t.shape, dtype=t.dtype, device=device) for k, t in host.items()}


class Step:
    """The five fused-operator calls on device-resident inputs."""

    def __init__(self, fo, shapes, d):
        import torch
        self.fo, self.d = fo, d
        dev = d["cell.X"].device
        s = shapes
        self.csr4 = fo.CSR(s["row_csr"]["rows"], s["row_csr"]["cols"], d["row_csr.rowptr"],
                           d["row_csr.colidx"], d["row_csr.vals"])
        self.csr5 = fo.CSR(s["outer"]["rows"], s["outer"]["cols"], d["outer.rowptr"],
                           d["outer.colidx"], d["outer.vals"])
        self.out = {
            "cell": torch.empty(1, dtype=torch.float64, device=dev),
            "magg": torch.empty(3, dtype=torch.float64, device=dev),
            "row_dense": torch.empty(s["row_dense"]["cols"], dtype=torch.float64, device=dev),
            "row_csr": torch.empty(s["row_csr"]["cols"], dtype=torch.float64, device=dev),
            "outer": torch.empty(1, dtype=torch.float64, device=dev),
        }
        self.launches = 0
        self.enabled = set(OPS)

    def run(self, name):
        fo, d, o = self.fo, self.d, self.out
        if name == "cell":
            fo.fused_cell(XYZ, "t1", d["cell.X"], [("cell", d["cell.Y"]), ("cell", d["cell.Z"])],
                          out=o["cell"])
        elif name == "magg":
            fo.fused_magg(MAGG3, ["t0", "t1", "t2"], d["magg.X"],
                          [("cell", d["magg.Y"]), ("cell", d["magg.Z"])], out=o["magg"])
        elif name == "row_dense":
            fo.fused_row(WD, "t0", d["row_dense.X"], d["row_dense.v"], [("row", d["row_dense.w"])],
                         out=o["row_dense"])
        elif name == "row_csr":
            fo.fused_row(WD, "t0", self.csr4, d["row_csr.v"], [("row", d["row_csr.w"])],
                         out=o["row_csr"])
        elif name == "outer":
            fo.fused_outer(WSLOSS, "t3", self.csr5, d["outer.U"], d["outer.V"], out=o["outer"])
        self.launches += 1

    def all(self, events=None):
        for i, name in enumerate(OPS):
            if name not in self.enabled:
                continue
            if events is not None:
                events[i][0].record()
            self.run(name)
            if events is not None:
                events[i][1].record()


def time_variants(fo, step, shapes, reps=10):
    """Other variants of the four templates on the inputs already resident (not part
    of the timed step): CUDA events, `reps` runs each after 2 warm-ups, inputs larger
    than L2.  Returns {name: {ms, gbs, bytes}}."""
    import torch
    d = step.d
    mr, mc = shapes["magg"]["rows"], shapes["magg"]["cols"]
    rr, rc = shapes["row_dense"]["rows"], shapes["row_dense"]["cols"]
    orow, rank = shapes["outer"]["rows"], shapes["outer"]["rank"]
    nnz5 = step.csr5.nnz
    sides = [("cell", d["magg.Y"]), ("cell", d["magg.Z"])]
    dev = d["magg.X"].device
    o_row = torch.empty(mr, dtype=torch.float64, device=dev)
    o_col = torch.empty(mc, dtype=torch.float64, device=dev)
    o_all = torch.empty((mr, mc), dtype=torch.float64, device=dev)
    o_one = torch.empty(1, dtype=torch.float64, device=dev)
    o_rr = torch.empty(rr, dtype=torch.float64, device=dev)
    o_rn = torch.empty((rr, rc), dtype=torch.float64, device=dev)
    o_nnz = torch.empty(nnz5, dtype=torch.float64, device=dev)
    o_right = torch.empty((orow, rank), dtype=torch.float64, device=dev)
    ocol = shapes["outer"]["cols"]
    o_left = torch.empty((ocol, rank), dtype=torch.float64, device=dev)
    generic = [("sub", "t0", "a", "side0"), ("abs", "t1", "t0"), ("fma", "t2", "t1", "side1", 0.5)]
    outer_generic = [("sub", "t1", "a", "d"), ("abs", "t2", "t1"), ("add", "t3", "t2", 0.25)]
    row_generic = [("mul", "t0", "side0", "d"), ("abs", "t1", "t0"), ("sub", "t2", "t1", 0.5)]
    o_rc = torch.empty(rc, dtype=torch.float64, device=dev)

    def interpreted(fn):
        fo.force_interpreter(True)
        try:
            fn()
        finally:
            fo.force_interpreter(False)

    in3 = 3 * 8 * mr * mc
    outer_in = 12 * nnz5 + 4 * (orow + 1) + 8 * rank * (orow + shapes["outer"]["cols"])
    cases = [
        ("cell_row_agg", lambda: fo.fused_cell(XYZ, "t1", d["magg.X"], sides, agg="row", out=o_row), in3 + 8 * mr),
        ("cell_col_agg", lambda: fo.fused_cell(XYZ, "t1", d["magg.X"], sides, agg="col", out=o_col), in3 + 8 * mc),
        ("cell_no_agg", lambda: fo.fused_cell(XYZ, "t1", d["magg.X"], sides, agg="none", out=o_all), in3 + 8 * mr * mc),
        # the cell-wise operator of the ALS-CG update rule (Section 2.2): I + 1e-6 * U * r, r a column vector
        ("cell_no_agg_scaled_add_vector_side",
         lambda: fo.fused_cell([("mul", "t0", "a", 1e-6), ("mul", "t1", "t0", "side1"), ("add", "t2", "side0", "t1")],
                               "t2", d["magg.X"], [("cell", d["magg.Y"]), ("row", o_row)], agg="none", out=o_all),
         3 * 8 * mr * mc + 8 * mr),
        ("cell_full_agg_runtime_compiled_chain",
         lambda: fo.fused_cell(generic, "t2", d["magg.X"], sides, agg="full", out=o_one), in3 + 8),
        ("cell_full_agg_interpreted_chain", lambda: interpreted(
            lambda: fo.fused_cell(generic, "t2", d["magg.X"], sides, agg="full", out=o_one)), in3 + 8),
        # the same chain in the row-wise and column kernels (compiled at run time too), against the
        # built-in product chain of cell_row_agg / cell_col_agg above
        ("cell_row_agg_runtime_compiled_chain",
         lambda: fo.fused_cell(generic, "t2", d["magg.X"], sides, agg="row", out=o_row), in3 + 8 * mr),
        ("cell_col_agg_runtime_compiled_chain",
         lambda: fo.fused_cell(generic, "t2", d["magg.X"], sides, agg="col", out=o_col), in3 + 8 * mc),
        ("cell_row_agg_interpreted_chain", lambda: interpreted(
            lambda: fo.fused_cell(generic, "t2", d["magg.X"], sides, agg="row", out=o_row)), in3 + 8 * mr),
        ("row_dense_row_agg", lambda: fo.fused_row(WD, "t0", d["row_dense.X"], d["row_dense.v"],
                                                   [("row", d["row_dense.w"])], agg="row", out=o_rr),
         8 * rr * rc + 16 * rr + 8 * rc),
        ("row_dense_full_agg", lambda: fo.fused_row(WD, "t0", d["row_dense.X"], d["row_dense.v"],
                                                    [("row", d["row_dense.w"])], agg="full", out=o_one),
         8 * rr * rc + 8 * rr + 8 * rc),
        ("row_dense_no_agg", lambda: fo.fused_row(WD, "t0", d["row_dense.X"], d["row_dense.v"],
                                                  [("row", d["row_dense.w"])], agg="none", out=o_rn),
         2 * 8 * rr * rc + 8 * rr + 8 * rc),
        ("outer_no_agg", lambda: fo.fused_outer(WSLOSS, "t3", step.csr5, d["outer.U"], d["outer.V"],
                                                agg="none", out=o_nnz), outer_in + 8 * nnz5),
        ("outer_right_mm", lambda: fo.fused_outer(WSLOSS, "t3", step.csr5, d["outer.U"], d["outer.V"],
                                                  agg="right", out=o_right), outer_in + 8 * orow * rank),
        # the sparsity-exploiting half of the ALS-CG update rule, Eq. 1: ((X != 0) * (U t(V))) V
        ("outer_right_mm_als_cg", lambda: fo.fused_outer([("ne", "t0", "a", 0.0), ("mul", "t1", "t0", "d")], "t1",
                                                         step.csr5, d["outer.U"], d["outer.V"], agg="right",
                                                         out=o_right), outer_in + 8 * orow * rank),
        ("outer_x_log_uvt_plus_eps", lambda: fo.fused_outer(
            [("add", "t0", "d", "s0"), ("log", "t1", "t0"), ("mul", "t2", "a", "t1")], "t2", step.csr5,
            d["outer.U"], d["outer.V"], [10.0], agg="full", out=o_one), outer_in + 8),
        ("outer_left_mm", lambda: fo.fused_outer(WSLOSS, "t3", step.csr5, d["outer.U"], d["outer.V"],
                                                 agg="left", out=o_left), outer_in + 8 * ocol * rank),
        # a chain without an inline form (|a - d| + 0.25): compiled at run time, and interpreted
        ("outer_full_agg_runtime_compiled_chain", lambda: fo.fused_outer(
            outer_generic, "t3", step.csr5, d["outer.U"], d["outer.V"], out=o_one), outer_in + 8),
        ("outer_right_mm_runtime_compiled_chain", lambda: fo.fused_outer(
            outer_generic, "t3", step.csr5, d["outer.U"], d["outer.V"], agg="right", out=o_right),
         outer_in + 8 * orow * rank),
        ("outer_full_agg_interpreted_chain", lambda: interpreted(lambda: fo.fused_outer(
            outer_generic, "t3", step.csr5, d["outer.U"], d["outer.V"], out=o_one)), outer_in + 8),
        # the Row chain |w * d| - 0.5: compiled at run time, and interpreted (once per row, warp-wide)
        ("row_dense_col_t_agg_runtime_compiled_chain", lambda: fo.fused_row(
            row_generic, "t2", d["row_dense.X"], d["row_dense.v"], [("row", d["row_dense.w"])], out=o_rc),
         8 * rr * rc + 8 * rr + 16 * rc),
        ("row_dense_col_t_agg_interpreted_chain", lambda: interpreted(lambda: fo.fused_row(
            row_generic, "t2", d["row_dense.X"], d["row_dense.v"], [("row", d["row_dense.w"])], out=o_rc)),
         8 * rr * rc + 8 * rr + 16 * rc),
    ]
    # sparse-safe Cell / MAgg (Section 5.2's sparse variants): X at density 0.1 as the CSR driver,
    # dense Y and Z read at the stored cells
    g = torch.Generator(device=dev)
    g.manual_seed(5)
    mask = torch.rand((mr, mc), generator=g, device=dev) < 0.1
    counts = mask.sum(dim=1, dtype=torch.int32)
    rowptr = torch.zeros(mr + 1, dtype=torch.int32, device=dev)
    rowptr[1:] = torch.cumsum(counts, 0)
    colidx = mask.nonzero()[:, 1].to(torch.int32).contiguous()
    Xs = fo.CSR(mr, mc, rowptr, colidx, d["magg.X"][mask].contiguous())
    del mask
    o_three = torch.empty(3, dtype=torch.float64, device=dev)
    sparse_in = 12 * Xs.nnz + 4 * (mr + 1) + 16 * Xs.nnz       # X once, one Y and one Z value per stored cell
    cases += [
        ("cell_csr_full_agg_density_0.1", lambda: fo.fused_cell(XYZ, "t1", Xs, sides, agg="full", out=o_one),
         sparse_in + 8),
        ("magg_csr_density_0.1", lambda: fo.fused_magg(MAGG3, ["t0", "t1", "t2"], Xs, sides, out=o_three),
         sparse_in + 24),
    ]
    # tall, narrow dense rows (the 10-column shape of the paper's end-to-end data, Section 5.3): the MAgg
    # input seen as (10 * rows) x 10
    if mc % 10 == 0:
        Xn = d["magg.X"].view(mr * (mc // 10), 10)
        g.manual_seed(7)
        vn = torch.randn(10, generator=g, dtype=torch.float64, device=dev)
        wn = torch.rand(Xn.shape[0], generator=g, dtype=torch.float64, device=dev)
        o_n = torch.empty(10, dtype=torch.float64, device=dev)
        cases.append(("row_dense_10cols_col_t_agg",
                      lambda: fo.fused_row(WD, "t0", Xn, vn, [("row", wn)], out=o_n),
                      8 * Xn.shape[0] * 10 + 8 * Xn.shape[0] + 160))
    # Row template with matrix-valued row intermediates (Section 5.2: t(X) %*% (X %*% V) with
    # V 1000 x 2 on the dense Row input; the Eq. 2 inner loop for k classes on the 100-column input)
    MLR_PRE = [("mul", "t0", "side0", "d")]
    MLR_POST = [("mul", "t0", "side0", "d"), ("mul", "t1", "side0", "rowsum"), ("sub", "t2", "t0", "t1")]
    g.manual_seed(6)
    V2 = torch.randn((rc, 2), generator=g, dtype=torch.float64, device=dev)
    P2 = torch.rand((rr, 2), generator=g, dtype=torch.float64, device=dev) / 3.0
    o_h2 = torch.empty((rc, 2), dtype=torch.float64, device=dev)
    cases += [
        ("row_b1_mmchain_k2", lambda: fo.fused_row_b1(None, None, [], "d", d["row_dense.X"], V2, out=o_h2),
         8 * rr * rc + 2 * 8 * rc * 2),
        ("row_b1_mlogreg_k2", lambda: fo.fused_row_b1(MLR_PRE, "t0", MLR_POST, "t2", d["row_dense.X"], V2,
                                                      [("cell", P2)], out=o_h2),
         8 * rr * rc + 8 * rr * 2 + 2 * 8 * rc * 2),
    ]
    for kk in (2, 8, 32):
        Vk = torch.randn((mc, kk), generator=g, dtype=torch.float64, device=dev)
        Pk = torch.rand((mr, kk), generator=g, dtype=torch.float64, device=dev) / (kk + 1)
        o_hk = torch.empty((mc, kk), dtype=torch.float64, device=dev)
        cases.append(("row_b1_mlogreg_100cols_k%d" % kk,
                      lambda Vk=Vk, Pk=Pk, o_hk=o_hk: fo.fused_row_b1(MLR_PRE, "t0", MLR_POST, "t2", d["magg.X"], Vk,
                                                                      [("cell", Pk)], out=o_hk),
                      8 * mr * mc + 8 * mr * kk + 2 * 8 * mc * kk))
    res = {}
    for name, fn, nbytes in cases:
        for _ in range(2):
            fn()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for a, b in ev:
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        ms = statistics.mean(a.elapsed_time(b) for a, b in ev)
        res[name] = {"ms": ms, "bytes": nbytes, "gbs": nbytes / (ms * 1e-3) / 1e9}
        if name.startswith("row_b1_mlogreg_100cols_k"):
            kk = int(name.rsplit("k", 1)[1])
            res[name]["fp64_tflops"] = 4.0 * mr * mc * kk / (ms * 1e-3) / 1e12
    return res


def _event_times(fn, reps, warm=2, before=None):
    """Milliseconds of `reps` runs of fn() (CUDA events on the current stream) after `warm` untimed runs;
    before() runs untimed ahead of every timed run."""
    import torch
    for _ in range(warm):
        fn()
    out = []
    for _ in range(reps):
        if before is not None:
            before()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        out.append(a.elapsed_time(b))
    return out


def machine_probes(fo, step, shapes):
    """Rates the rooflines are quoted against besides the copy peak: a read-only streaming sum through
    the Cell kernel, whole-row gathers from an L2-resident matrix, and fp64 multiply-add issue."""
    import torch
    d = step.d
    dev = d["row_dense.X"].device
    one = torch.empty(1, dtype=torch.float64, device=dev)
    X = d["row_dense.X"]
    ms = min(_event_times(lambda: fo.fused_cell([("mov", "t0", "a")], "t0", X, agg="full", out=one), 5))
    res = {"stream_sum_gbs": X.numel() * 8 / (ms * 1e-3) / 1e9,
           "stream_sum": "sum(X) over the %dx%d Row input, Cell kernel" % tuple(X.shape)}
    V = d["outer.V"]
    g = torch.Generator(device=dev)
    g.manual_seed(7)
    n = 10_000_000
    out = torch.empty(fo.probe_out_len(), dtype=torch.float64, device=dev)
    for label, nrows in (("l2_gather_gbs", min(V.shape[0], 40_000)), ("gather_all_rows_gbs", V.shape[0])):
        idx = torch.randint(0, nrows, (n,), generator=g, device=dev, dtype=torch.int32)
        moved = [0]

        def run(idx=idx):
            moved[0] = fo.probe_l2_gather(V, idx, out)
        ms = min(_event_times(run, 5))
        res[label] = moved[0] / (ms * 1e-3) / 1e9
        res[label + "_rows"] = nrows
    res["l2_gather"] = ("%d random rows of %d doubles from the first rows of V (%.0f MB resident set, resp. "
                        "all of V)" % (n, V.shape[1], 40_000 * V.shape[1] * 8 / 1e6))
    # the same rows through the bulk-copy engine (a differently shaped measurement of the same rate)
    idx = torch.randint(0, V.shape[0], (n,), generator=g, device=dev, dtype=torch.int32)
    moved = [0]

    def run_bulk(idx=idx):
        moved[0] = fo.probe_bulk_gather(V, idx, out)
    ms = min(_event_times(run_bulk, 5))
    res["bulk_gather_all_rows_gbs"] = moved[0] / (ms * 1e-3) / 1e9
    res["bulk_gather_wait_ran_out"] = bool(out[fo.probe_bulk_flag_index()].item() != 0.0)
    res["sm_count"] = torch.cuda.get_device_properties(dev).multi_processor_count
    flops = [0]

    def fma():
        flops[0] = fo.probe_fp64_fma(20_000, out)
    ms = min(_event_times(fma, 5))
    res["fp64_fma_tflops"] = flops[0] / (ms * 1e-3) / 1e12
    return res


def size_sweep(fo, device, cols=1000, rows_list=(1_000, 10_000, 100_000, 1_000_000), reps=10):
    """Cell sum(X*Y*Z) and the three-aggregate MAgg over rows x 1000 inputs, rows from 1e3 to 1e6
    (Section 5.2's sweep), cold L2: a 512 MB buffer is overwritten before every timed run."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(11)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=device)
    one = torch.empty(1, dtype=torch.float64, device=device)
    three = torch.empty(3, dtype=torch.float64, device=device)
    res = []
    for rows in rows_list:
        X, Y, Z = (torch.rand((rows, cols), generator=g, dtype=torch.float64, device=device) for _ in range(3))
        sides = [("cell", Y), ("cell", Z)]
        nbytes = 3 * 8 * rows * cols
        entry = {"rows": rows, "cols": cols, "bytes": nbytes}
        for name, fn in (("cell", lambda: fo.fused_cell(XYZ, "t1", X, sides, out=one)),
                         ("magg", lambda: fo.fused_magg(MAGG3, ["t0", "t1", "t2"], X, sides, out=three))):
            ms = _event_times(fn, reps, before=flush.zero_)
            entry[name] = {"us_min": min(ms) * 1e3, "us_median": statistics.median(ms) * 1e3,
                           "us_mean": statistics.mean(ms) * 1e3,
                           "gbs_at_median": nbytes / (statistics.median(ms) * 1e-3) / 1e9}
        res.append(entry)
        del X, Y, Z
    return res


def cell_phases(fo, device, rows=1000, cols=1000, reps=8):
    """Where the small Cell workload (config 1: 24 MB) spends its time: the streaming kernel's own
    phase stamps (GPU global timer, ns; cold L2) for 1 .. 8 CTAs per SM, and CUDA events around the call."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(13)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=device)
    one = torch.empty(1, dtype=torch.float64, device=device)
    X, Y, Z = (torch.rand((rows, cols), generator=g, dtype=torch.float64, device=device) for _ in range(3))
    sides = [("cell", Y), ("cell", Z)]
    res = {}
    try:
        for cps in (1, 2, 3, 4, 6, 8):
            fo.tune("cell.ctas_per_sm", cps)
            fo.tune("cell.stamps", 0)
            ev = _event_times(lambda: fo.fused_cell(XYZ, "t1", X, sides, out=one), reps, before=flush.zero_)
            fo.tune("cell.stamps", 1)
            ph = []
            for _ in range(reps):
                flush.zero_()
                fo.fused_cell(XYZ, "t1", X, sides, out=one)
                st = fo.cell_stamps(device)
                ph.append((st[1] - st[0], st[2] - st[1], st[3] - st[2], st[3] - st[0]))
            med = [int(statistics.median(p[i] for p in ph[2:])) for i in range(4)]
            res["ctas_per_sm_%d" % cps] = {"scan_ns": med[0], "publish_ns": med[1], "final_ns": med[2],
                                           "kernel_ns": med[3], "events_us_min": min(ev) * 1e3}
    finally:
        fo.tune("cell.ctas_per_sm", None)
        fo.tune("cell.stamps", None)
    return res


# ---------------------------------------------------------------------- clocks
def _device_csr(fo, rows, cols, density, g, device, lo=0.0, hi=1.0, chunk_rows=None):
    """A Bernoulli(density) CSR matrix built on the device (values uniform[lo, hi)), row chunk by
    row chunk so that the dense mask of a chunk stays small."""
    import torch
    if density >= 1.0:
        rowptr = (torch.arange(rows + 1, device=device, dtype=torch.int64) * cols).to(torch.int32)
        colidx = torch.arange(cols, device=device, dtype=torch.int32).repeat(rows)
        vals = torch.rand(rows * cols, generator=g, dtype=torch.float64, device=device) * (hi - lo) + lo
        return fo.CSR(rows, cols, rowptr, colidx, vals)
    chunk_rows = chunk_rows or max(1, (64 << 20) // cols)
    counts, cols_l = [], []
    for r0 in range(0, rows, chunk_rows):
        nr = min(chunk_rows, rows - r0)
        mask = torch.rand((nr, cols), generator=g, device=device) < density
        counts.append(mask.sum(dim=1, dtype=torch.int32))
        cols_l.append(mask.nonzero()[:, 1].to(torch.int32))
        del mask
    rowptr = torch.zeros(rows + 1, dtype=torch.int32, device=device)
    rowptr[1:] = torch.cumsum(torch.cat(counts), 0)
    colidx = torch.cat(cols_l).contiguous()
    vals = torch.rand(colidx.numel(), generator=g, dtype=torch.float64, device=device) * (hi - lo) + lo
    return fo.CSR(rows, cols, rowptr, colidx, vals)


def paper_suite(fo, device, reps=5, peak_gbs=6650.0, fp64_tflops=37.0, l2_gather_gbs=18500.0):
    """The operator micro-benchmarks of Section 5.2 at the paper's own sizes (inputs made on the
    device from a seeded torch generator; parity of every kernel used here is covered by the tests):
    Cell sum(X*Y*Z), MAgg (sum(X*Y), sum(X*Z)), Row t(X)(Xv) and t(X)(XV) over x * 10^3 inputs,
    x = 10^3 .. 10^6, dense and at sparsity 0.1; Outer sum(X * log(U t(V) + 1e-15)) over
    2*10^4 x 2*10^4 at rank 100, sparsity 1 .. 10^-4.  Cold L2 (a 512 MB buffer is rewritten
    before every run); times are the minimum of `reps` runs.  Every entry carries its roofline:
    the bytes the operator must read once over the copy bandwidth (`*_frac`: ideal / measured
    time); the Outer entries the slowest of three terms - compulsory bytes over the copy
    bandwidth, gathered factor rows over the L2 gather rate (per-cell schedule) or the tile
    products over the fp64 rate (tiled schedule, densely stored X), and the stored cells'
    logarithms over a measured log rate."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(12)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=device)
    one = torch.empty(1, dtype=torch.float64, device=device)
    two = torch.empty(2, dtype=torch.float64, device=device)
    magg2 = [("mul", "t0", "a", "side0"), ("mul", "t1", "a", "side1")]
    cols = 1000
    qv = torch.empty(cols, dtype=torch.float64, device=device)
    qm = torch.empty((cols, 2), dtype=torch.float64, device=device)
    v = torch.randn(cols, generator=g, dtype=torch.float64, device=device)
    V2 = torch.randn((cols, 2), generator=g, dtype=torch.float64, device=device)

    def t_us(fn):
        return min(_event_times(fn, reps, before=flush.zero_)) * 1e3

    out = {"cell_magg_row": [], "outer": []}
    for rows in (1_000, 10_000, 100_000, 1_000_000):
        X, Y, Z = (torch.rand((rows, cols), generator=g, dtype=torch.float64, device=device) for _ in range(3))
        sides = [("cell", Y), ("cell", Z)]
        Xs = _device_csr(fo, rows, cols, 0.1, g, device)
        e = {"rows": rows, "cols": cols, "dense_bytes_per_input": 8 * rows * cols, "sparse_nnz": Xs.nnz}
        e["cell_dense_us"] = t_us(lambda: fo.fused_cell(XYZ, "t1", X, sides, out=one))
        e["cell_sparse_us"] = t_us(lambda: fo.fused_cell(XYZ, "t1", Xs, sides, out=one))
        Ys = _device_csr(fo, rows, cols, 0.1, g, device)
        Zs = _device_csr(fo, rows, cols, 0.1, g, device)
        ssides = [("cell", Ys), ("cell", Zs)]
        e["cell_all_sparse_us"] = t_us(lambda: fo.fused_cell(XYZ, "t1", Xs, ssides, out=one))
        e["magg_all_sparse_us"] = t_us(lambda: fo.fused_magg(magg2, ["t0", "t1"], Xs, ssides, out=two))
        del Ys, Zs, ssides
        e["magg_dense_us"] = t_us(lambda: fo.fused_magg(magg2, ["t0", "t1"], X, sides, out=two))
        e["magg_sparse_us"] = t_us(lambda: fo.fused_magg(magg2, ["t0", "t1"], Xs, sides, out=two))
        e["row_xtxv_dense_us"] = t_us(lambda: fo.fused_row([], "d", X, v, out=qv))
        e["row_xtxv_sparse_us"] = t_us(lambda: fo.fused_row([], "d", Xs, v, out=qv))
        e["row_xtxV2_dense_us"] = t_us(lambda: fo.fused_row_b1(None, None, [], "d", X, V2, out=qm))
        # rooflines: bytes each operator must read once (sparse: 12 per stored cell + row offsets; a dense
        # side read at a stored cell costs its 8 bytes, a sparse side its own 12 per stored cell)
        dense3, csr = 3 * 8 * rows * cols, 12 * Xs.nnz + 4 * (rows + 1)
        algo = {"cell_dense": dense3, "magg_dense": dense3, "cell_sparse": csr + 16 * Xs.nnz,
                "magg_sparse": csr + 16 * Xs.nnz, "cell_all_sparse": 3 * csr, "magg_all_sparse": 3 * csr,
                "row_xtxv_dense": 8 * rows * cols + 16 * cols, "row_xtxv_sparse": csr + 16 * cols,
                "row_xtxV2_dense": 8 * rows * cols + 4 * 8 * cols}
        for name, nb in algo.items():
            us = e[name + "_us"]
            e[name + "_gbs"] = nb / (us * 1e-6) / 1e9
            e[name + "_frac"] = nb / (peak_gbs * 1e9) / (us * 1e-6)
        out["cell_magg_row"].append(e)
        del X, Y, Z, Xs, sides
    m = 20_000
    U = torch.rand((m, 100), generator=g, dtype=torch.float64, device=device) + 0.1
    Vf = torch.rand((m, 100), generator=g, dtype=torch.float64, device=device) + 0.1
    xlog = [("add", "t0", "d", 1e-15), ("log", "t1", "t0"), ("mul", "t2", "a", "t1")]
    # the rate of the chain's logarithm alone: log over a streamed array (the Cell kernel), cells per second
    L = torch.rand(20_000_000, generator=g, dtype=torch.float64, device=device) + 0.5
    log_us = t_us(lambda: fo.fused_cell([("log", "t0", "a")], "t0", L.view(20_000, 1000), out=one))
    log_rate = L.numel() / (log_us * 1e-6)
    del L
    out["log_cells_per_s"] = log_rate
    for sp in (1.0, 0.1, 0.01, 0.001, 0.0001):
        Xs = _device_csr(fo, m, m, sp, g, device, chunk_rows=2000)
        us = t_us(lambda: fo.fused_outer(xlog, "t2", Xs, U, Vf, out=one))
        tiled = Xs.nnz >= 0.15 * m * m            # the schedule the library picks (stored share of X)
        terms = {"hbm": (12 * Xs.nnz + 4 * (m + 1) + 2 * 8 * m * 100) / (peak_gbs * 1e9) * 1e6,
                 "log": Xs.nnz / log_rate * 1e6}
        if tiled:
            terms["fp64_tiles"] = 2.0 * m * m * 100 / (fp64_tflops * 1e12) * 1e6
        else:
            terms["l2_gather"] = Xs.nnz * 800 / (l2_gather_gbs * 1e9) * 1e6
        binding = max(terms, key=terms.get)
        out["outer"].append({"sparsity": sp, "nnz": Xs.nnz, "us": us, "nnz_per_s": Xs.nnz / (us * 1e-6),
                             "schedule": "tiled" if tiled else "per stored cell",
                             "bound_terms_us": terms, "binding_term": binding,
                             "frac_of_binding_term": terms[binding] / us})
        del Xs
    return out


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index, period=0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for n, bit in names.items():
                    if mask & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


def physical_gpu_index(local_index):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


# ---------------------------------------------------------------------- oracle legs
def oracle_step(np_inputs, shapes):
    """One pass of the CPU checker over (a sample of) the five workloads; returns per-op seconds."""
    import oracle
    h = np_inputs
    t = {}
    t0 = time.perf_counter()
    r = {"cell": oracle.sum_xyz(h["cell.X"], h["cell.Y"], h["cell.Z"])}
    t["cell"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    r["magg"] = oracle.magg_xy_xz_xx(h["magg.X"], h["magg.Y"], h["magg.Z"])
    t["magg"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    r["row_dense"] = oracle.row_chain_dense(h["row_dense.X"], h["row_dense.v"], h["row_dense.w"])
    t["row_dense"] = time.perf_counter() - t0
    s = shapes["row_csr"]
    X4 = dict(rows=s["rows"], cols=s["cols"], rowptr=h["row_csr.rowptr"], colidx=h["row_csr.colidx"],
              vals=h["row_csr.vals"])
    t0 = time.perf_counter()
    r["row_csr"] = oracle.row_chain_csr(X4, h["row_csr.v"], h["row_csr.w"])
    t["row_csr"] = time.perf_counter() - t0
    s = shapes["outer"]
    X5 = dict(rows=s["rows"], cols=s["cols"], rowptr=h["outer.rowptr"], colidx=h["outer.colidx"],
              vals=h["outer.vals"])
    t0 = time.perf_counter()
    r["outer"] = oracle.outer_wsloss_masked(X5, h["outer.U"], h["outer.V"])
    t["outer"] = time.perf_counter() - t0
    return t, r


def oracle_single_thread(np_inputs, shapes):
    """Cell and Outer legs of the checker with the numeric libraries held to one thread."""
    import oracle
    h = np_inputs
    try:
        from threadpoolctl import threadpool_limits
        limit = threadpool_limits(limits=1)
    except Exception:
        limit = None
    try:
        t = {}
        t0 = time.perf_counter()
        oracle.sum_xyz(h["cell.X"], h["cell.Y"], h["cell.Z"])
        t["cell"] = time.perf_counter() - t0
        s = shapes["outer"]
        X5 = dict(rows=s["rows"], cols=s["cols"], rowptr=h["outer.rowptr"], colidx=h["outer.colidx"],
                  vals=h["outer.vals"])
        t0 = time.perf_counter()
        oracle.outer_wsloss_masked(X5, h["outer.U"], h["outer.V"])
        t["outer"] = time.perf_counter() - t0
    finally:
        if limit is not None:
            limit.restore_original_limits()
    return t


REL_TOL = 1e-10           # relative tolerance for fp64 aggregates and elementwise outputs
ABS_FLOOR = 1e-15         # times the sum of the magnitudes of a sum's terms (sums that cancel)


def abs_scales(h, shapes, panel=100_000):
    """Sum of the magnitudes of the terms of every result of the five operators (plain numpy, row
    panels): the denominator of a sum's condition number."""
    import oracle
    sc = {"cell": np.array([np.sum(np.abs(h["cell.X"] * h["cell.Y"] * h["cell.Z"]))])}
    X, Y, Z = h["magg.X"], h["magg.Y"], h["magg.Z"]
    acc = np.zeros(3)
    for r0 in range(0, X.shape[0], panel):
        x, y, z = X[r0:r0 + panel], Y[r0:r0 + panel], Z[r0:r0 + panel]
        acc += [np.abs(x * y).sum(), np.abs(x * z).sum(), (x * x).sum()]
    sc["magg"] = acc
    X, v, w = h["row_dense.X"], np.abs(h["row_dense.v"]), h["row_dense.w"]
    acc = np.zeros(X.shape[1])
    for r0 in range(0, X.shape[0], panel):
        ax = np.abs(X[r0:r0 + panel])
        acc += ax.T @ (np.abs(w[r0:r0 + panel]) * (ax @ v))
    sc["row_dense"] = acc
    s4 = shapes["row_csr"]
    X4 = dict(rows=s4["rows"], cols=s4["cols"], rowptr=h["row_csr.rowptr"], colidx=h["row_csr.colidx"],
              vals=np.abs(h["row_csr.vals"]))
    sc["row_csr"] = np.asarray(oracle.row_chain_csr(X4, np.abs(h["row_csr.v"]), np.abs(h["row_csr.w"])))
    sc["outer"] = None            # every term (a - d)^2 is non-negative: the sum is its own scale
    return sc


def parity_report(results, refs, scales):
    """GPU results against the checker's, per operator: largest relative error, condition number
    of the worst-conditioned element, and how many elements met the tolerance only through the
    floor for cancelling sums.  ok: every element within REL_TOL, or within the floor."""
    rep, ok_all = {}, True
    for k in OPS:
        if k not in refs or k not in results:
            continue
        g = np.asarray(results[k], dtype=np.float64).reshape(-1)
        r = np.asarray(refs[k], dtype=np.float64).reshape(-1)
        err = np.abs(g - r)
        rel = err / np.maximum(np.abs(r), 1e-300)
        sc = np.abs(r) if scales.get(k) is None else np.asarray(scales[k], dtype=np.float64).reshape(-1)
        strict = err <= REL_TOL * np.abs(r)
        floor = err <= ABS_FLOOR * sc
        ok = bool(np.all(strict | floor))
        rep[k] = {"max_rel_err": float(rel.max()), "cond_max": float(np.max(sc / np.maximum(np.abs(r), 1e-300))),
                  "floor_used": int(np.count_nonzero(~strict & floor)), "elements": int(r.size), "ok": ok}
        ok_all = ok_all and ok
    rep["tolerance"] = "|gpu - ref| <= %g |ref|, or <= %g x sum of |terms| for sums that cancel" % (REL_TOL, ABS_FLOOR)
    rep["ok"] = ok_all
    return rep


def cpu_model():
    try:
        for ln in open("/proc/cpuinfo"):
            if ln.startswith("model name"):
                return ln.split(":", 1)[1].strip()
    except Exception:
        pass
    return "unknown"


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return 1


def sample_description(shapes):
    return ("rows scaled: magg %dx%d, row_dense %dx%d, row_csr %dx%d@%.3g, outer %dx%d rank %d@%.3g "
            "(row panel, all of V); cell full size" % (
                shapes["magg"]["rows"], shapes["magg"]["cols"], shapes["row_dense"]["rows"],
                shapes["row_dense"]["cols"], shapes["row_csr"]["rows"], shapes["row_csr"]["cols"],
                shapes["row_csr"]["density"], shapes["outer"]["rows"], shapes["outer"]["cols"],
                shapes["outer"]["rank"], shapes["outer"]["density"]))


def numpy_inputs(host):
    return {k: t.numpy() for k, t in host.items()}


def run_reference(args):
    """The CPU checker, as it stands, on bounded samples; host cores only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    shapes = scaled(FULL, args.ref_frac)
    # the Outer sample is a panel of rows against all of V
    shapes["outer"]["cols"] = FULL["outer"]["cols"]
    host = make_host_inputs(shapes, pinned=False)
    nbytes = algorithmic_bytes(shapes, host)
    total = sum(nbytes.values())
    h = numpy_inputs(host)
    for _ in range(args.warmup):
        oracle_step(h, shapes)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(h, shapes)
    dt = time.perf_counter() - t0
    value = total * args.steps / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic (seeded, in-repo generator)",
        "config": {"workload": "all five fused operators, bounded sample of the full-size configs",
                   "sample": sample_description(shapes)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                         "sample": sample_description(shapes)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def max_over_ranks(values, device=None):
    """Element-wise maximum of `values` over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64,
                     device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def row_sample(host, shapes, frac):
    """The first `frac` of the rows of every workload (views of the host arrays; the
    Outer sample is a row panel against all of V; the Cell workload stays whole)."""
    import torch
    sh = {k: dict(v) for k, v in shapes.items()}
    h = dict(host)
    for op in ("magg", "row_dense"):
        r = max(8, int(round(shapes[op]["rows"] * frac)))
        sh[op]["rows"] = r
        for k in list(h):
            if k.startswith(op + ".") and h[k].shape[0] == shapes[op]["rows"]:
                h[k] = h[k][:r]
    for op in ("row_csr", "outer"):
        r = max(8, int(round(shapes[op]["rows"] * frac)))
        sh[op]["rows"] = r
        rp = h[op + ".rowptr"][:r + 1]
        nnz = int(rp[-1])
        h[op + ".rowptr"] = rp
        h[op + ".colidx"] = h[op + ".colidx"][:nnz]
        h[op + ".vals"] = h[op + ".vals"][:nnz]
        if op == "row_csr":
            h["row_csr.w"] = h["row_csr.w"][:r]
        else:
            h["outer.U"] = h["outer.U"][:r]
    return h, sh


# ---------------------------------------------------------------------- main arm
def run_ours(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the fused operators have no CPU path")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    import paper_1801_00829_b200 as fo
    fo.load_library()

    shapes = scaled(FULL, args.frac) if args.frac != 1.0 else {k: dict(v) for k, v in FULL.items()}
    if args.frac != 1.0:
        shapes["outer"]["cols"] = max(8, int(round(FULL["outer"]["cols"] * args.frac)))
        if args.full_outer:
            shapes["outer"] = dict(FULL["outer"])
    t_gen = time.perf_counter()
    host = make_host_inputs(shapes, pinned=True)
    t_gen = time.perf_counter() - t_gen
    nbytes = algorithmic_bytes(shapes, host)
    total_bytes = sum(nbytes.values())
    dev = alloc_device(host, device)
    upload(host, dev)
    torch.cuda.synchronize()
    step = Step(fo, shapes, dev)
    if args.ops:
        step.enabled = set(args.ops.split(","))
        assert step.enabled <= set(OPS), "unknown op in --ops"
    if args.interp:
        fo.force_interpreter(True)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: K steps between two events
    for _ in range(args.warmup):
        step.all()
    barrier()
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in OPS]
          for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    launches0 = step.launches
    barrier()
    e0.record()
    for k in range(args.steps):
        step.all(ev[k])
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms_total = e0.elapsed_time(e1)
    gpu_launches = step.launches - launches0
    per_op_ms = {name: ([ev[k][i][0].elapsed_time(ev[k][i][1]) for k in range(args.steps)]
                        if name in step.enabled else [float("nan")])
                 for i, name in enumerate(OPS)}
    results = {k: v.cpu().numpy().copy() for k, v in step.out.items()}
    status = fo.device_status(device)

    # ---- end to end: host buffers -> device -> five calls -> results back on the host
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    h2d = sum(t.numel() * t.element_size() for t in host.values())
    host_out = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True) for k, v in step.out.items()}
    d2h = sum(t.numel() * t.element_size() for t in host_out.values())

    def e2e_once():
        upload(host, dev)
        step.all()
        for k2, v2 in step.out.items():
            host_out[k2].copy_(v2, non_blocking=True)

    e2e_once()
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for _ in range(e2e_steps):
        e2e_once()
    f1.record()
    barrier()
    ms_e2e = f0.elapsed_time(f1)

    # ---- max over ranks
    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], device if world > 1 else None)

    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    peak_gbs = float(peaks.get("hbm_gbs", 6650.0))
    peak_kind = "measured" if "hbm_gbs" in peaks else "fallback"

    total_bytes = sum(nbytes[n] for n in step.enabled)
    ms_step = ms_total / args.steps
    value = world * total_bytes / (ms_step * 1e-3) / 1e9
    e2e_value = world * total_bytes / (ms_e2e / e2e_steps * 1e-3) / 1e9
    per_op = {}
    for name in OPS:
        ms = statistics.mean(per_op_ms[name])
        gbs = nbytes[name] / (ms * 1e-3) / 1e9
        per_op[name] = {"ms": ms, "ms_min": min(per_op_ms[name]), "ms_median": statistics.median(per_op_ms[name]),
                        "bytes": nbytes[name], "gbs": gbs, "frac_of_" + peak_kind: gbs / peak_gbs,
                        "frac_of_nominal_8000": gbs / 8000.0}
    nnz4, nnz5 = int(host["row_csr.vals"].numel()), int(host["outer.vals"].numel())
    per_op["row_csr"]["nnz_per_s"] = nnz4 / (per_op["row_csr"]["ms"] * 1e-3)
    per_op["outer"]["nnz_per_s"] = nnz5 / (per_op["outer"]["ms"] * 1e-3)
    dominant = max(sorted(step.enabled), key=lambda n: per_op[n]["ms"])
    units = {"cell": shapes["cell"]["rows"] * shapes["cell"]["cols"],
             "magg": shapes["magg"]["rows"] * shapes["magg"]["cols"],
             "row_dense": shapes["row_dense"]["rows"], "row_csr": nnz4, "outer": nnz5}
    per_unit = NCU_DRAM_BYTES_PER_UNIT.get(dominant)
    traffic = per_unit * units[dominant] if per_unit is not None and args.frac == 1.0 else None
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": per_op[dominant]["gbs"], "peak": peak_gbs,
                "peak_kind": peak_kind, "unit": "GB/s", "frac": per_op[dominant]["gbs"] / peak_gbs,
                "traffic": traffic, "algorithmic_bytes": nbytes[dominant]}
    roofline_per_op = {n: {"bound": "hbm", "achieved": per_op[n]["gbs"], "peak": peak_gbs, "unit": "GB/s",
                           "frac": per_op[n]["gbs"] / peak_gbs, "algorithmic_bytes": nbytes[n]}
                       for n in OPS if n in step.enabled}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded, in-repo generator)",
        "config": {"workload": "all five fused operators at full size: cell 1000x1000x3, magg 1e6x100x3, "
                               "row dense 1e6x1000, row csr 1e7x1000@0.01, outer 1e5x1e5@0.001 rank 100"
                               if args.frac == 1.0 else "five fused operators, rows scaled by %g" % args.frac,
                   "shapes": shapes, "nnz": {"row_csr": nnz4, "outer": nnz5},
                   "l2": "inputs larger than L2: 12 GB stream through between two uses of any array",
                   "multi_gpu": "replicas only"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps},
        "gpu_launches": gpu_launches,
        "roofline": roofline,
        "roofline_per_op": roofline_per_op,
        "per_op": per_op,
        "device_status": status,
        "results": {k: [float(x) for x in v.reshape(-1)[:3]] for k, v in results.items()},
        "input_generation_s": t_gen,
    }

    if not args.no_variants and step.enabled == set(OPS):
        line["variants"] = time_variants(fo, step, shapes)
        probes = machine_probes(fo, step, shapes)
        line["probes"] = probes
        for n in roofline_per_op:
            roofline_per_op[n]["frac_of_stream_sum"] = per_op[n]["gbs"] / probes["stream_sum_gbs"]
        # Outer: the slowest of compulsory bytes / HBM, gathered V rows / L2 gather rate, FMAs / fp64 rate.
        # The gather rate is quoted three ways: the per-lane-load probe, the bulk-copy probe (another
        # access shape), and what the hardware's L2-to-SM path carries at most (64 bytes per clock and SM)
        rank5 = shapes["outer"]["rank"]
        sm_mhz = float(peaks.get("sm_max_mhz", 1965.0))
        probes["l2_to_sm_port_gbs"] = probes["sm_count"] * 64 * sm_mhz * 1e6 / 1e9
        probes["l2_to_sm_port"] = "%d SMs x 64 B per clock x %.0f MHz" % (probes["sm_count"], sm_mhz)
        gather_bytes = nnz5 * rank5 * 8
        terms = {"hbm": nbytes["outer"] / (peak_gbs * 1e9) * 1e3,
                 "l2_gather": gather_bytes / (probes["l2_gather_gbs"] * 1e9) * 1e3,
                 "fp64_fma": 2.0 * nnz5 * rank5 / (probes["fp64_fma_tflops"] * 1e12) * 1e3}
        binding = max(terms, key=terms.get)
        roofline_per_op["outer"].update({
            "bound_terms_ms": terms, "binding_term": binding,
            "frac_of_binding_term": terms[binding] / per_op["outer"]["ms"],
            "l2_gather_ms_by_bulk_copy_probe": gather_bytes / (probes["bulk_gather_all_rows_gbs"] * 1e9) * 1e3,
            "l2_gather_ms_at_port_limit": gather_bytes / (probes["l2_to_sm_port_gbs"] * 1e9) * 1e3,
            "frac_of_port_limit": gather_bytes / (probes["l2_to_sm_port_gbs"] * 1e9) * 1e3 / per_op["outer"]["ms"]})
        # the paper's cost model (Section 4.3: write time + max(read time, compute time)) fed with
        # this machine's measured rates: predicted time of each fused operator and of the plan of
        # basic operators it replaces, next to the measured time
        gf = probes["fp64_fma_tflops"] * 1e3
        cm = {}
        for n in OPS:
            kw = dict(shapes[n])
            if n == "row_csr":
                kw["nnz"] = nnz4
            if n == "outer":
                kw["nnz"] = nnz5
            kw = {k2: v2 for k2, v2 in kw.items() if k2 in ("rows", "cols", "nnz", "rank")}
            fused = fo.plan_cost([fo.operator_sizes(n, **kw)], peak_gbs, peak_gbs, gf) * 1e3
            unfused = fo.plan_cost(fo.unfused_plan_sizes(n, **kw), peak_gbs, peak_gbs, gf) * 1e3
            cm[n] = {"predicted_fused_ms": fused, "predicted_unfused_ms": unfused,
                     "measured_ms": per_op[n]["ms"], "measured_over_predicted": per_op[n]["ms"] / fused}
        line["cost_model"] = cm
        if args.frac == 1.0 and world == 1:
            line["size_sweep"] = size_sweep(fo, device)
            line["cell_phases"] = cell_phases(fo, device)
        if args.paper_suite and world == 1:
            line["paper_suite"] = paper_suite(fo, device, peak_gbs=peak_gbs, fp64_tflops=probes["fp64_fma_tflops"],
                                              l2_gather_gbs=probes["l2_gather_gbs"])

    # ---- CPU baseline: the checker on a bounded sample, rank 0 at N = 1 only; at full size its
    # results are also what the GPU results of the timed steps are checked against
    parity_ok = True
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        chost, cshapes = row_sample(host, shapes, args.cpu_frac)
        cbytes = algorithmic_bytes(cshapes, chost)
        cnp = numpy_inputs(chost)
        runs = []
        for _ in range(max(1, args.cpu_runs)):
            t0 = time.perf_counter()
            ct, cres = oracle_step(cnp, cshapes)
            runs.append((time.perf_counter() - t0, ct))
        cdt, ct = min(runs, key=lambda x: x[0])
        line["cpu_baseline"] = {
            "value": sum(cbytes.values()) / cdt / 1e9, "unit": UNIT, "cores": host_threads(),
            "kind": "oracle", "sample": "first %g of the rows of the bench inputs: %s" % (
                args.cpu_frac, sample_description(cshapes)),
            "seconds": cdt, "runs": len(runs), "seconds_all_runs": [r[0] for r in runs],
            "per_op_gbs": {k: cbytes[k] / ct[k] / 1e9 for k in OPS},
            "cpu_model": cpu_model(), "nproc": os.cpu_count(),
        }
        # one thread, configs 1 and 5 (Outer on a sixteenth of the sample's rows)
        shost, sshapes = row_sample(chost, cshapes, 1.0 / 16)
        sbytes = algorithmic_bytes(sshapes, shost)
        st = oracle_single_thread(numpy_inputs(shost), sshapes)
        line["cpu_baseline"]["single_thread_gbs"] = {k: sbytes[k] / st[k] / 1e9 for k in st}
        line["cpu_baseline"]["single_thread_sample"] = "cell full size; outer %d rows x %d" % (
            sshapes["outer"]["rows"], sshapes["outer"]["cols"])
        if args.cpu_frac == 1.0 and step.enabled == set(OPS):
            line["parity"] = parity_report(results, cres, abs_scales(cnp, cshapes))
        else:       # only the Cell workload is whole in a sample
            line["parity"] = parity_report({"cell": results["cell"]}, {"cell": cres["cell"]}, {"cell": None})
            line["parity"]["note"] = "sampled CPU run: only the Cell workload is compared"
        parity_ok = line["parity"]["ok"]
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0 if parity_ok else 3


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--frac", type=float, default=1.0, help="scale the row counts (debugging)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-frac", type=float, default=1.0, help="sample of the workloads the CPU baseline runs")
    ap.add_argument("--cpu-runs", type=int, default=2, help="runs of the CPU baseline (the best one is reported)")
    ap.add_argument("--ref-frac", type=float, default=0.01, help="sample per step of --impl reference")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-variants", action="store_true", help="skip the untimed-step variant measurements")
    ap.add_argument("--full-outer", action="store_true", help="keep the Outer workload at full size under --frac")
    ap.add_argument("--ops", default="", help="comma-separated subset of the five operators (profiling)")
    ap.add_argument("--paper-suite", action="store_true", default=True,
                    help="time the paper's operator micro-benchmarks at their own sizes too (the default; about a minute)")
    ap.add_argument("--no-paper-suite", dest="paper_suite", action="store_false")
    ap.add_argument("--interp", action="store_true", help="run Cell / MAgg chains through the interpreter")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
