"""The five benchmark workloads at full size, in the launch configuration bench.py
times, against the CPU checker: every output element where the checker is fast
enough, sampled outputs plus size-independent properties elsewhere."""
import math
import os
import sys

import numpy as np
import pytest

import datagen
import oracle
from util import assert_close, to_dev

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


@pytest.fixture(scope="module")
def fo():
    import torch
    assert torch.cuda.is_available()
    import paper_1801_00829_b200 as fo_
    fo_.load_library()
    return fo_


def test_cell_full_size(fo):
    w = datagen.cell_workload()                       # 1000 x 1000, seed 0
    got = fo.fused_cell(bench.XYZ, "t1", to_dev(w["X"]), [("cell", to_dev(w["Y"])), ("cell", to_dev(w["Z"]))])
    assert_close(got.cpu().numpy(), [oracle.sum_xyz(w["X"], w["Y"], w["Z"])])
    for agg in ("row", "col"):
        ref = oracle.cell(bench.XYZ, "t1", w["X"], [("cell", w["Y"]), ("cell", w["Z"])], agg=agg)
        g = fo.fused_cell(bench.XYZ, "t1", to_dev(w["X"]), [("cell", to_dev(w["Y"])), ("cell", to_dev(w["Z"]))],
                          agg=agg)
        assert_close(g.cpu().numpy(), ref, what="cell %s" % agg)


def test_magg_full_size(fo):
    w = datagen.magg_workload()                       # 1e6 x 100, seed 1
    ref = oracle.magg_xy_xz_xx(w["X"], w["Y"], w["Z"])
    absref = np.array([np.abs(w["X"] * w["Y"]).sum(), np.abs(w["X"] * w["Z"]).sum(), ref[2]])
    got = fo.fused_magg(bench.MAGG3, ["t0", "t1", "t2"], to_dev(w["X"]),
                        [("cell", to_dev(w["Y"])), ("cell", to_dev(w["Z"]))])
    # no element of a full-size result needs the floor for cancelling sums
    assert_close(got.cpu().numpy(), ref, absscale=absref, what="magg full size", max_floor=0)


def test_row_dense_full_size(fo):
    import torch
    rows, cols = 1_000_000, 1000
    w = datagen.row_dense_workload(rows, cols)        # seed 2
    Xd, vd, wd = to_dev(w["X"]), to_dev(w["v"]), to_dev(w["w"])
    got = fo.fused_row(bench.WD, "t0", Xd, vd, [("row", wd)]).cpu().numpy()
    ref = oracle.row_chain_dense(w["X"], w["v"], w["w"])
    # |X|^T (w * (|X| |v|)) would cost two more passes over 8 GB: a bound from the
    # second moments does as the cancellation scale (every |term| is O(w |x| |d|))
    scale = np.full(cols, float(rows) * 0.5 * math.sqrt(cols))
    assert_close(got, ref, absscale=scale, what="row dense full size", max_floor=0)
    assert fo.device_status() == 0
    # sampled rows of the per-row output, one by one
    t = fo.fused_row(bench.WD, "t0", Xd, vd, [("row", wd)], agg="row").cpu().numpy()
    for i in (0, 1, 7, 8, 12345, 500_000, 999_991, 999_999):
        ti = float(w["w"][i]) * float(np.sum(w["X"][i].astype(np.longdouble) * w["v"]))
        assert abs(t[i] - ti) <= 1e-10 * max(abs(ti), 1e-15 * float(np.abs(w["X"][i]) @ np.abs(w["v"])) * 1e5)
    # size-independent property: sum_j v_j q_j = sum_i w_i (X_i . v)^2
    lhs = float(np.sum(got.astype(np.longdouble) * w["v"]))
    rhs = float(np.sum((t.astype(np.longdouble) ** 2) / np.maximum(w["w"], 1e-300)))
    assert abs(lhs - rhs) <= 1e-9 * abs(rhs)
    del Xd
    torch.cuda.empty_cache()


def test_row_csr_full_size(fo):
    w = datagen.row_csr_workload()                    # 1e7 x 1000 @ 0.01, seed 3
    X = {k: w[k] for k in ("rows", "cols", "rowptr", "colidx", "vals")}
    ref = oracle.row_chain_csr(X, w["v"], w["w"])
    scale = oracle.row_chain_csr(dict(X, vals=np.abs(w["vals"])), np.abs(w["v"]), w["w"])
    Xd = fo.CSR(w["rows"], w["cols"], to_dev(w["rowptr"]), to_dev(w["colidx"]), to_dev(w["vals"]))
    got = fo.fused_row(bench.WD, "t0", Xd, to_dev(w["v"]), [("row", to_dev(w["w"]))]).cpu().numpy()
    assert_close(got, ref, absscale=scale, what="row csr full size", max_floor=0)


def test_outer_full_size(fo):
    w = datagen.outer_workload()                      # 1e5 x 1e5 @ 0.001, rank 100, seed 4
    rows = w["rows"]
    Xd = fo.CSR(rows, w["cols"], to_dev(w["rowptr"]), to_dev(w["colidx"]), to_dev(w["vals"]))
    Ud, Vd = to_dev(w["U"]), to_dev(w["V"])
    got = fo.fused_outer(bench.WSLOSS, "t3", Xd, Ud, Vd).item()
    per_cell = fo.fused_outer(bench.WSLOSS, "t3", Xd, Ud, Vd, agg="none").cpu().numpy()
    # the checker on row panels (its nnz x rank intermediates would not fit in one go)
    total = []
    panel = 10_000
    for r0 in range(0, rows, panel):
        a, b = int(w["rowptr"][r0]), int(w["rowptr"][r0 + panel])
        sub = dict(rows=panel, cols=w["cols"], rowptr=(w["rowptr"][r0:r0 + panel + 1] - a).astype(np.int32),
                   colidx=w["colidx"][a:b], vals=w["vals"][a:b])
        total.append(oracle.outer_wsloss_masked(sub, w["U"][r0:r0 + panel], w["V"]))
        if r0 in (0, 50_000, 90_000):                 # sampled panels, cell by cell
            ref_cells = oracle.outer(bench.WSLOSS, "t3", sub, w["U"][r0:r0 + panel], w["V"], agg="none",
                                     mode="masked")
            assert_close(per_cell[a:b], ref_cells, what="outer cells of panel %d" % r0)
    ref = math.fsum(total)
    assert_close([got], [ref], what="outer full size")
    # full_agg equals the sum of its own per-cell values
    assert abs(got - math.fsum(per_cell.tolist())) <= 1e-11 * abs(got)
