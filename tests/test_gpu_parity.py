"""CUDA library vs. the CPU checker, element by element, on the same seeded inputs.

Sizes here are the ones the checker finishes in seconds; they still span several
tiles and ragged tails.  Tolerance: see tests/util.py (relative 1e-10).
"""
import numpy as np
import pytest

import datagen
import oracle
from datagen.workloads import csr_to_dense
from util import assert_close, csr_to_dev, host_csr, to_dev

pytestmark = pytest.mark.gpu

XYZ = [("mul", "t0", "a", "side0"), ("mul", "t1", "t0", "side1")]
MAGG3 = [("mul", "t0", "a", "side0"), ("mul", "t1", "a", "side1"), ("mul", "t2", "a", "a")]
WD = [("mul", "t0", "side0", "d")]
WSLOSS = [("ne", "t0", "a", 0.0), ("sub", "t1", "a", "d"), ("mul", "t2", "t1", "t1"),
          ("mul", "t3", "t0", "t2")]


@pytest.fixture(scope="module")
def fo():
    import torch
    assert torch.cuda.is_available()
    import paper_1801_00829_b200 as fo_
    fo_.load_library()
    return fo_


def dev_sides(sides):
    return [(acc, to_dev(arr)) for acc, arr in sides]


# ------------------------------------------------------------------ Cell
@pytest.mark.parametrize("chain,out,scalars", [
    ([("mul", "t0", "a", 1e-6), ("mul", "t1", "t0", "side1"), ("add", "t2", "side0", "t1")], "t2", []),
    ([("mul", "t3", "s0", "a"), ("mul", "t1", "side1", "t3"), ("add", "t0", "t1", "side0")], "t0", [0.25]),
])
@pytest.mark.parametrize("rows,cols", [(3000, 20), (257, 100), (64, 1000)])
def test_cell_scaled_add_chain_equals_interpreter_bitwise(fo, chain, out, scalars, rows, cols):
    """The cell-wise operator of Section 2.2 (I + 1e-6 * U * r: a matrix side, a column-vector side, no
    aggregation) runs as straight-line code; same bits as the interpreter, same values as the checker."""
    U = datagen.normal(61, 0, rows * cols).reshape(rows, cols)
    I = datagen.normal(61, 2, rows * cols).reshape(rows, cols)
    r = datagen.normal(61, 3, rows)
    for sides_h in ([("cell", I), ("row", r)], [("cell", I), ("cell", I)]):
        sides_d = [(a, to_dev(x)) for a, x in sides_h]
        for agg in ("none", "full"):
            try:
                fo.force_interpreter(False)
                fast = fo.fused_cell(chain, out, to_dev(U), sides_d, scalars, agg=agg).cpu().numpy()
                fo.force_interpreter(True)
                slow = fo.fused_cell(chain, out, to_dev(U), sides_d, scalars, agg=agg).cpu().numpy()
            finally:
                fo.force_interpreter(False)
            assert fast.tobytes() == slow.tobytes()
            ref = oracle.cell(chain, out, U, sides_h, scalars, agg=agg)
            c = scalars[0] if scalars else 1e-6
            second = sides_h[1][1][:, None] if sides_h[1][0] == "row" else sides_h[1][1]
            tabs = np.abs(I) + np.abs(U * c * second)
            assert_close(fast, np.asarray(ref), absscale=tabs if agg == "none" else float(tabs.sum()))


@pytest.mark.parametrize("cols", [1, 2, 5, 10, 20, 32, 33, 63, 64, 65])
def test_cell_narrow_rows_with_vector_sides(fo, cols):
    """Rows of at most 64 columns share a warp in the row-wise Cell kernel: every aggregation, the three
    side kinds (a column vector and a row vector keep the call off the flat kernel), strided inputs."""
    rows, ld = 4099, cols + 2
    flat = datagen.normal(51, 0, rows * ld + 1)
    Y = datagen.normal(51, 2, rows * cols).reshape(rows, cols)
    rvec = datagen.normal(51, 3, rows)
    cvec = datagen.normal(51, 4, cols)
    chain = [("mul", "t0", "a", "side0"), ("fma", "t1", "t0", "side1", "side2"), ("mul", "t2", "t1", "s0")]
    for off in (0, 1):
        Xh = flat[off:off + rows * ld].reshape(rows, ld)[:, :cols]
        Xd = to_dev(flat)[off:off + rows * ld].view(rows, ld)[:, :cols]
        sides_h = [("cell", Y), ("row", rvec), ("col", cvec)]
        sides_d = [("cell", to_dev(Y)), ("row", to_dev(rvec)), ("col", to_dev(cvec))]
        tabs = (np.abs(Xh * Y) * np.abs(rvec)[:, None] + np.abs(cvec)[None, :]) * 1.5
        for agg in ("none", "row", "full"):
            ref = oracle.cell(chain, "t2", Xh, sides_h, [1.5], agg=agg)
            got = fo.fused_cell(chain, "t2", Xd, sides_d, [1.5], agg=agg)
            scale = {"none": tabs, "row": tabs.sum(axis=1), "full": float(tabs.sum())}[agg]
            assert_close(got.cpu().numpy(), np.asarray(ref), absscale=scale, what="cell narrow %d %s off=%d" % (cols, agg, off))
    # several aggregates in one scan over the same layout
    ref = oracle.magg(MAGG3, ["t0", "t1", "t2"], Xh, [("cell", Y), ("cell", Y)])
    got = fo.fused_magg(MAGG3, ["t0", "t1", "t2"], Xd, [("cell", to_dev(Y)), ("cell", to_dev(Y))])
    assert_close(got.cpu().numpy(), ref, absscale=np.array([np.abs(Xh * Y).sum(), np.abs(Xh * Y).sum(), (Xh * Xh).sum()]))
    assert fo.device_status() == 0


@pytest.mark.parametrize("rows,cols", [(1000, 1000), (1, 1), (1, 7), (5, 1), (33, 65), (257, 129),
                                       (1024, 1), (1, 1024), (3, 1025), (2047, 3), (64, 2048)])
def test_cell_full_xyz(fo, rows, cols):
    w = datagen.cell_workload(rows, cols, seed=0)
    ref = oracle.sum_xyz(w["X"], w["Y"], w["Z"])
    got = fo.fused_cell(XYZ, "t1", to_dev(w["X"]), dev_sides([("cell", w["Y"]), ("cell", w["Z"])]))
    assert_close(got.cpu().numpy(), [ref], what="cell full %dx%d" % (rows, cols))


def test_cell_full_is_bit_reproducible(fo):
    w = datagen.cell_workload(777, 333, seed=5)
    args = (XYZ, "t1", to_dev(w["X"]), dev_sides([("cell", w["Y"]), ("cell", w["Z"])]))
    a = fo.fused_cell(*args).cpu().numpy()
    for _ in range(3):
        assert fo.fused_cell(*args).cpu().numpy().tobytes() == a.tobytes()


@pytest.mark.parametrize("agg", ["full", "row", "col", "none"])
@pytest.mark.parametrize("rows,cols", [(300, 200), (37, 1001), (129, 5), (8, 513), (1, 1)])
def test_cell_aggs_with_all_side_kinds(fo, agg, rows, cols):
    X = datagen.normal(7, 0, rows * cols).reshape(rows, cols)
    Y = datagen.normal(7, 2, rows * cols).reshape(rows, cols)
    rv = datagen.normal(7, 3, rows)
    cv = datagen.normal(7, 4, cols)
    chain = [("mul", "t0", "a", "s0"), ("mul", "t1", "t0", "side1"),
             ("add", "t2", "side0", "t1"), ("sub", "t3", "t2", "side2")]
    sides = [("cell", Y), ("row", rv), ("col", cv)]
    ref = oracle.cell(chain, "t3", X, sides, [0.25], agg=agg)
    absref = oracle.cell([("abs", "t0", "a"), ("abs", "t1", "side0"), ("abs", "t2", "side1"),
                          ("abs", "t3", "side2"), ("mul", "t4", "t0", 0.25), ("mul", "t5", "t4", "t2"),
                          ("add", "t6", "t5", "t1"), ("add", "t7", "t6", "t3")], "t7", X, sides,
                         agg=agg)
    got = fo.fused_cell(chain, "t3", to_dev(X), dev_sides(sides), [0.25], agg=agg)
    assert_close(got.cpu().numpy(), ref, absscale=absref, what="cell %s" % agg)


@pytest.mark.parametrize("agg", ["full", "row", "col", "none"])
def test_cell_strided_and_unaligned_inputs(fo, agg):
    import torch
    rows, cols, ld = 45, 70, 77
    base = datagen.uniform(3, 0, rows * ld + 1, 0.5, 1.5)
    basey = datagen.uniform(3, 2, rows * ld + 1, 0.5, 1.5)
    for off in (0, 1):                      # off = 1: base pointer only 8-byte aligned
        Xh = base[off:off + rows * ld].reshape(rows, ld)[:, :cols]
        Yh = basey[off:off + rows * ld].reshape(rows, ld)[:, :cols]
        Xd = to_dev(base)[off:off + rows * ld].view(rows, ld)[:, :cols]
        Yd = to_dev(basey)[off:off + rows * ld].view(rows, ld)[:, :cols]
        assert Xd.stride(0) == ld
        chain = [("mul", "t0", "a", "side0")]
        ref = oracle.cell(chain, "t0", Xh, [("cell", Yh)], agg=agg)
        got = fo.fused_cell(chain, "t0", Xd, [("cell", Yd)], agg=agg)
        assert_close(got.cpu().numpy(), ref, what="strided off=%d %s" % (off, agg))
    # contiguous but 8-byte-aligned base: the flat kernel must not be chosen
    n = 5000
    xd = to_dev(datagen.uniform(3, 4, n + 1))
    ref = oracle.cell([("sq", "t0", "a")], "t0", xd[1:].cpu().numpy().reshape(1, n))
    got = fo.fused_cell([("sq", "t0", "a")], "t0", xd[1:].view(1, n))
    assert_close(got.cpu().numpy(), [ref])
    torch.cuda.synchronize()


def test_cell_every_opcode(fo):
    rows, cols = 64, 96
    X = datagen.uniform(11, 0, rows * cols, 0.25, 4.0).reshape(rows, cols)
    Y = datagen.uniform(11, 2, rows * cols, -2.0, 2.0).reshape(rows, cols)
    Y[::7, ::5] = 0.0
    sides = [("cell", Y)]
    unary = ["mov", "neg", "abs", "sqrt", "exp", "log", "sq"]
    binary = ["add", "sub", "mul", "div", "min", "max", "eq", "ne", "lt", "le", "gt", "ge"]
    for op in unary:
        ch = [(op, "t0", "a")]
        ref = oracle.cell(ch, "t0", X, sides, agg="none")
        got = fo.fused_cell(ch, "t0", to_dev(X), dev_sides(sides), agg="none")
        assert_close(got.cpu().numpy(), ref, what=op)
    for op in binary:
        ch = [(op, "t0", "a", "side0")]
        if op == "div":
            ch = [("add", "t1", "side0", 3.0), ("div", "t0", "a", "t1")]
        ref = oracle.cell(ch, "t0", X, sides, agg="none")
        got = fo.fused_cell(ch, "t0", to_dev(X), dev_sides(sides), agg="none")
        assert_close(got.cpu().numpy(), ref, what=op)
    ch = [("pow", "t0", "a", 1.7)]
    assert_close(fo.fused_cell(ch, "t0", to_dev(X), agg="none").cpu().numpy(),
                 oracle.cell(ch, "t0", X, agg="none"), what="pow")
    ch = [("sel", "t0", "side0", "a", -1.0)]
    assert_close(fo.fused_cell(ch, "t0", to_dev(X), dev_sides(sides), agg="none").cpu().numpy(),
                 oracle.cell(ch, "t0", X, sides, agg="none"), what="sel")
    ch = [("fma", "t0", "a", "side0", 0.5)]
    assert_close(fo.fused_cell(ch, "t0", to_dev(X), dev_sides(sides), agg="none").cpu().numpy(),
                 oracle.cell(ch, "t0", X, sides, agg="none"), absscale=np.abs(X * Y) + 0.5, what="fma")
    # equality on exactly equal values
    ch = [("eq", "t0", "a", "a"), ("ne", "t1", "a", "a"), ("add", "t2", "t0", "t1")]
    assert fo.fused_cell(ch, "t2", to_dev(X)).item() == float(rows * cols)


def test_cell_long_chain_with_register_reuse(fo):
    rows, cols = 100, 64
    X = datagen.uniform(13, 0, rows * cols, 0.5, 1.5).reshape(rows, cols)
    sides = [("cell", datagen.uniform(13, 2 + k, rows * cols, 0.5, 1.5).reshape(rows, cols))
             for k in range(4)]
    chain = []
    # 30 steps cycling through all eight temporaries
    chain.append(("mul", "t0", "a", "side0"))
    for k in range(1, 30):
        src = "side%d" % (k % 4)
        chain.append((("add", "mul", "sub")[k % 3], "t%d" % (k % 8), "t%d" % ((k - 1) % 8), src))
    chain.append(("mul", "t1", "t%d" % (29 % 8), "s0"))
    ref = oracle.cell(chain, "t1", X, sides, [0.5])
    got = fo.fused_cell(chain, "t1", to_dev(X), dev_sides(sides), [0.5])
    absref = oracle.cell(chain + [("abs", "t2", "t1")], "t2", X, sides, [0.5])
    assert_close(got.cpu().numpy(), [ref], absscale=absref)


def test_cell_empty(fo):
    import torch
    X = torch.zeros((0, 5), dtype=torch.float64, device="cuda")
    assert fo.fused_cell([("sq", "t0", "a")], "t0", X).item() == 0.0
    assert fo.fused_cell([("sq", "t0", "a")], "t0", X, agg="col").cpu().tolist() == [0.0] * 5


# ------------------------------------------------------------------ MAgg
@pytest.mark.parametrize("rows,cols", [(20000, 100), (999, 7), (1, 3)])
def test_magg_three_aggregates(fo, rows, cols):
    w = datagen.magg_workload(rows, cols, seed=1)
    ref = oracle.magg_xy_xz_xx(w["X"], w["Y"], w["Z"])
    absref = oracle.magg_xy_xz_xx(np.abs(w["X"]), np.abs(w["Y"]), np.abs(w["Z"]))
    got = fo.fused_magg(MAGG3, ["t0", "t1", "t2"], to_dev(w["X"]),
                        dev_sides([("cell", w["Y"]), ("cell", w["Z"])]))
    assert_close(got.cpu().numpy(), ref, absscale=absref, what="magg")


@pytest.mark.parametrize("k", [1, 2, 5, 8])
def test_magg_k_outputs_match_single_cells(fo, k):
    rows, cols = 513, 40
    X = datagen.normal(21, 0, rows * cols).reshape(rows, cols)
    Y = datagen.normal(21, 2, rows * cols).reshape(rows, cols)
    rv = datagen.uniform(21, 3, rows)
    chain = [("mul", "t0", "a", "side0")]
    outs = ["t0"]
    for j in range(1, k):
        chain.append(("fma", "t%d" % j, "t%d" % (j - 1), "side1", float(j)))
        outs.append("t%d" % j)
    sides = [("cell", Y), ("row", rv)]
    ref = oracle.magg(chain, outs, X, sides)
    absref = oracle.magg(chain + [("abs", "t%d" % j, "t%d" % j) for j in range(k)], outs, X, sides)
    got = fo.fused_magg(chain, outs, to_dev(X), dev_sides(sides))
    assert_close(got.cpu().numpy(), ref, absscale=absref + rows * cols * k)
    for j in range(k):       # fused multi-aggregate == each aggregate on its own
        single = fo.fused_cell(chain, outs[j], to_dev(X), dev_sides(sides))
        assert_close(single.cpu().numpy(), [ref[j]], absscale=absref[j] + rows * cols * k)


# ------------------------------------------------------------------ Row
def row_abs_scale(X, v, w):
    return np.abs(X).T @ (np.abs(w) * (np.abs(X) @ np.abs(v)))


@pytest.mark.parametrize("rows,cols", [(2000, 1000), (501, 64), (37, 10), (100, 1024), (9, 2),
                                       (1, 128), (300, 257), (64, 999), (5, 1), (333, 512), (200, 1026),
                                       (77, 2048), (50, 3000), (21, 4100), (19, 8192), (18, 8191)])
def test_row_dense_col_t(fo, rows, cols):
    w = datagen.row_dense_workload(rows, cols, seed=2)
    ref = oracle.row_chain_dense(w["X"], w["v"], w["w"])
    got = fo.fused_row(WD, "t0", to_dev(w["X"]), to_dev(w["v"]), [("row", to_dev(w["w"]))])
    assert_close(got.cpu().numpy(), ref, absscale=row_abs_scale(w["X"], w["v"], w["w"]),
                 what="row dense %dx%d" % (rows, cols))
    assert fo.device_status() == 0


def test_row_dense_many_tiles_per_cta_and_reproducible(fo):
    rows, cols = 20011, 1000         # > 148 * 8 * 3 rows: every ring slot is reused, ragged last tile
    w = datagen.row_dense_workload(rows, cols, seed=22)
    ref = oracle.row_chain_dense(w["X"], w["v"], w["w"])
    args = (WD, "t0", to_dev(w["X"]), to_dev(w["v"]), [("row", to_dev(w["w"]))])
    got = fo.fused_row(*args).cpu().numpy()
    assert_close(got, ref, absscale=row_abs_scale(w["X"], w["v"], w["w"]))
    assert fo.fused_row(*args).cpu().numpy().tobytes() == got.tobytes()
    assert fo.device_status() == 0


@pytest.mark.parametrize("agg", ["col_t", "row", "full"])
def test_row_dense_variants_strided_unaligned(fo, agg):
    rows, cols, ld = 333, 120, 130
    flat = datagen.normal(2, 0, rows * ld + 1)
    v = datagen.normal(2, 2, cols)
    wv = datagen.uniform(2, 3, rows)
    chain = [("mul", "t0", "side0", "d"), ("add", "t1", "t0", "s0")]
    for off in (0, 1):
        Xh = flat[off:off + rows * ld].reshape(rows, ld)[:, :cols]
        Xd = to_dev(flat)[off:off + rows * ld].view(rows, ld)[:, :cols]
        ref = oracle.row(chain, "t1", Xh, v, [("row", wv)], [0.125], agg=agg)
        scale = {"col_t": np.abs(Xh).T @ (wv * (np.abs(Xh) @ np.abs(v)) + 0.125),
                 "row": None, "full": float(np.sum(wv * (np.abs(Xh) @ np.abs(v)) + 0.125))}[agg]
        got = fo.fused_row(chain, "t1", Xd, to_dev(v), [("row", to_dev(wv))], [0.125], agg=agg)
        assert_close(got.cpu().numpy(), ref, absscale=scale, what="row %s off=%d" % (agg, off))
    # no weight: t(X) %*% (X %*% v)
    Xh = flat[:rows * ld].reshape(rows, ld)[:, :cols]
    ref = oracle.row([], "d", Xh, v, agg="col_t")
    got = fo.fused_row([], "d", to_dev(flat)[:rows * ld].view(rows, ld)[:, :cols], to_dev(v))
    assert_close(got.cpu().numpy(), ref, absscale=row_abs_scale(Xh, v, np.ones(rows)))


@pytest.mark.parametrize("cols", [1, 2, 3, 4, 5, 8, 10, 13, 16, 17, 24, 31, 32])
def test_row_dense_narrow_rows_all_variants(fo, cols):
    """At most 32 columns: a thread takes whole rows.  Every aggregation, a chain that goes through the
    interpreter, contiguous and strided / 8-byte-aligned inputs."""
    rows, ld = 70001, cols + 3
    flat = datagen.normal(31, 0, rows * ld + 1)
    v = datagen.normal(31, 2, cols)
    wv = datagen.uniform(31, 3, rows)
    chain = [("mul", "t0", "side0", "d"), ("add", "t1", "t0", "s0")]
    for layout in ("contiguous", "strided", "offset"):
        if layout == "contiguous":
            Xh = np.ascontiguousarray(flat[:rows * cols].reshape(rows, cols))
            Xd = to_dev(Xh)
        else:
            off = 0 if layout == "strided" else 1
            Xh = flat[off:off + rows * ld].reshape(rows, ld)[:, :cols]
            Xd = to_dev(flat)[off:off + rows * ld].view(rows, ld)[:, :cols]
        tabs = wv * (np.abs(Xh) @ np.abs(v)) + 0.125
        for agg in ("col_t", "row", "full", "none"):
            ref = oracle.row(chain, "t1", Xh, v, [("row", wv)], [0.125], agg=agg)
            got = fo.fused_row(chain, "t1", Xd, to_dev(v), [("row", to_dev(wv))], [0.125], agg=agg)
            scale = {"col_t": np.abs(Xh).T @ tabs, "row": tabs, "full": float(np.sum(tabs)),
                     "none": tabs[:, None] * np.abs(Xh)}[agg]
            assert_close(got.cpu().numpy(), ref, absscale=scale, what="narrow %d cols %s %s" % (cols, layout, agg))
    # the weighted chain evaluated inline, and bit-reproducible
    ref = oracle.row_chain_dense(Xh, v, wv)
    a = fo.fused_row(WD, "t0", Xd, to_dev(v), [("row", to_dev(wv))]).cpu().numpy()
    assert_close(a, ref, absscale=row_abs_scale(Xh, v, wv))
    assert fo.fused_row(WD, "t0", Xd, to_dev(v), [("row", to_dev(wv))]).cpu().numpy().tobytes() == a.tobytes()
    assert fo.device_status() == 0


@pytest.mark.parametrize("rows,cols", [(1000, 1000), (333, 120), (257, 129), (64, 18), (5, 1), (1, 7), (90, 4096),
                                       (40, 8191)])
def test_row_dense_no_agg_and_col_agg(fo, rows, cols):
    w = datagen.row_dense_workload(rows, cols, seed=2)
    chain = [("mul", "t0", "side0", "d"), ("add", "t1", "t0", "s0")]
    sides_h, sides_d = [("row", w["w"])], [("row", to_dev(w["w"]))]
    ref = oracle.row(chain, "t1", w["X"], w["v"], sides_h, [0.25], agg="none")
    got = fo.fused_row(chain, "t1", to_dev(w["X"]), to_dev(w["v"]), sides_d, [0.25], agg="none")
    assert tuple(got.shape) == (rows, cols)
    tabs = (w["w"] * (np.abs(w["X"]) @ np.abs(w["v"])) + 0.25)[:, None] * np.abs(w["X"])
    assert_close(got.cpu().numpy(), ref, absscale=tabs, what="row dense no_agg")
    refc = oracle.row(chain, "t1", w["X"], w["v"], sides_h, [0.25], agg="col")
    gotc = fo.fused_row(chain, "t1", to_dev(w["X"]), to_dev(w["v"]), sides_d, [0.25], agg="col")
    assert_close(gotc.cpu().numpy(), refc, absscale=tabs.sum(axis=0), what="row dense col_agg")
    # an output that starts 8 bytes off a 16-byte boundary
    import torch
    buf = torch.empty(rows * cols + 1, dtype=torch.float64, device="cuda")
    out = buf[1:].view(rows, cols)
    fo.fused_row(chain, "t1", to_dev(w["X"]), to_dev(w["v"]), sides_d, [0.25], agg="none", out=out)
    assert_close(out.cpu().numpy(), ref, absscale=tabs, what="row dense no_agg, unaligned out")
    assert fo.device_status() == 0


@pytest.mark.parametrize("rows,cols,density", [(20000, 1000, 0.01), (5000, 64, 0.2), (300, 4000, 0.001), (17, 9, 0.5),
                                               (2000, 800, 0.1), (100, 50, 0.0)])
def test_row_csr_no_agg_and_col_agg(fo, rows, cols, density):
    w = datagen.row_csr_workload(rows, cols, density, seed=3)
    Xh = host_csr(w)
    sides_h, sides_d = [("row", w["w"])], [("row", to_dev(w["w"]))]
    ref = oracle.row(WD, "t0", Xh, w["v"], sides_h, agg="none")
    got = fo.fused_row(WD, "t0", csr_to_dev(w), to_dev(w["v"]), sides_d, agg="none")
    assert tuple(got.shape) == (len(w["vals"]),)
    absX = dict(Xh, vals=np.abs(w["vals"]))
    tabs = oracle.row(WD, "t0", absX, np.abs(w["v"]), sides_h, agg="none")
    assert_close(got.cpu().numpy(), ref, absscale=tabs, what="row csr no_agg")
    refc = oracle.row(WD, "t0", Xh, w["v"], sides_h, agg="col")
    gotc = fo.fused_row(WD, "t0", csr_to_dev(w), to_dev(w["v"]), sides_d, agg="col")
    assert_close(gotc.cpu().numpy(), refc, absscale=oracle.row(WD, "t0", absX, np.abs(w["v"]), sides_h, agg="col"),
                 what="row csr col_agg")
    assert fo.device_status() == 0


@pytest.mark.parametrize("rows,cols,density", [(100000, 1000, 0.01), (5000, 64, 0.2), (300, 4000, 0.001),
                                               (17, 9, 0.5), (1000, 1000, 0.0),
                                               # mean row lengths 36, 80 and 200: 8, 16 and 32 lanes per row
                                               (3000, 600, 0.06), (2000, 800, 0.1), (1500, 2000, 0.1)])
def test_row_csr_col_t(fo, rows, cols, density):
    w = datagen.row_csr_workload(rows, cols, density, seed=3)
    Xh = host_csr(w)
    ref = oracle.row_chain_csr(Xh, w["v"], w["w"])
    absX = dict(Xh, vals=np.abs(w["vals"]))
    scale = oracle.row_chain_csr(absX, np.abs(w["v"]), w["w"])
    got = fo.fused_row(WD, "t0", csr_to_dev(w), to_dev(w["v"]), [("row", to_dev(w["w"]))])
    assert_close(got.cpu().numpy(), ref, absscale=scale, what="row csr")


@pytest.mark.parametrize("agg", ["row", "full"])
@pytest.mark.parametrize("density", [0.02, 0.05, 0.12, 0.5])
def test_row_csr_other_aggs_and_dense_agreement(fo, agg, density):
    rows, cols = 2500, 300
    w = datagen.row_csr_workload(rows, cols, density, seed=33)
    Xh = host_csr(w)
    ref = oracle.row(WD, "t0", Xh, w["v"], [("row", w["w"])], agg=agg)
    got = fo.fused_row(WD, "t0", csr_to_dev(w), to_dev(w["v"]), [("row", to_dev(w["w"]))], agg=agg)
    absX = dict(Xh, vals=np.abs(w["vals"]))
    scale = oracle.row(WD, "t0", absX, np.abs(w["v"]), [("row", w["w"])], agg=agg)
    assert_close(got.cpu().numpy(), ref, absscale=scale)
    # the dense kernel on the same matrix agrees too
    Xd = csr_to_dense(rows, cols, w["rowptr"], w["colidx"], w["vals"])
    got_d = fo.fused_row(WD, "t0", to_dev(Xd), to_dev(w["v"]), [("row", to_dev(w["w"]))], agg=agg)
    assert_close(got_d.cpu().numpy(), ref, absscale=scale)


# ------------------------------------------------------------------ Outer
def outer_case(rows, cols, rank, density, seed=4):
    w = datagen.outer_workload(rows, cols, rank, density, seed)
    return w, host_csr(w)


@pytest.mark.parametrize("rows,cols,rank,density", [
    (2000, 3000, 100, 0.01), (300, 200, 1, 0.1), (300, 200, 16, 0.1), (300, 200, 17, 0.1),
    (257, 129, 33, 0.2), (100, 90, 128, 0.3), (64, 50, 256, 0.3), (500, 400, 7, 0.0),
    (40, 30, 100, 1.0)])
def test_outer_full_agg(fo, rows, cols, rank, density):
    w, Xh = outer_case(rows, cols, rank, density)
    ref = oracle.outer_wsloss_masked(Xh, w["U"], w["V"])
    got = fo.fused_outer(WSLOSS, "t3", csr_to_dev(w), to_dev(w["U"]), to_dev(w["V"]))
    assert_close(got.cpu().numpy(), [ref], what="outer full rank %d" % rank)
    if rows * cols <= 1_000_000:
        assert_close(got.cpu().numpy(), [oracle.outer_wsloss_dense(Xh, w["U"], w["V"])])


@pytest.mark.parametrize("agg", ["none", "right", "left"])
@pytest.mark.parametrize("rank", [5, 100, 200])
def test_outer_other_aggs(fo, agg, rank):
    w, Xh = outer_case(700, 900, rank, 0.02, seed=14)
    chain = [("ne", "t0", "a", 0.0), ("mul", "t1", "t0", "d")]          # (X != 0) * (U V^T), Eq. 1
    ref = oracle.outer(chain, "t1", Xh, w["U"], w["V"], agg=agg, mode="masked")
    got = fo.fused_outer(chain, "t1", csr_to_dev(w), to_dev(w["U"]), to_dev(w["V"]), agg=agg)
    absU, absV = np.abs(w["U"]), np.abs(w["V"])
    scale = oracle.outer(chain, "t1", Xh, absU, absV, agg=agg, mode="masked")
    assert_close(got.cpu().numpy(), ref, absscale=scale, what="outer %s" % agg)


def test_outer_explicit_zeros_unaligned_and_reproducible(fo):
    w, Xh = outer_case(400, 300, 10, 0.05, seed=24)
    w["vals"][::3] = 0.0                 # stored zeros stay stored
    Xh = host_csr(w)
    ref = oracle.outer_wsloss_masked(Xh, w["U"], w["V"])
    ref_nomask = oracle.outer(WSLOSS[1:3], "t2", Xh, w["U"], w["V"], mode="masked")
    assert ref_nomask > ref
    Xd = csr_to_dev(w)
    got = fo.fused_outer(WSLOSS, "t3", Xd, to_dev(w["U"]), to_dev(w["V"]))
    assert_close(got.cpu().numpy(), [ref])
    got2 = fo.fused_outer(WSLOSS[1:3], "t2", Xd, to_dev(w["U"]), to_dev(w["V"]))
    assert_close(got2.cpu().numpy(), [ref_nomask])
    # U, V with a padded leading dimension and an 8-byte-aligned base
    Up = to_dev(np.pad(w["U"], ((0, 0), (0, 3))).reshape(-1))
    Vp = to_dev(np.concatenate([[0.0], np.pad(w["V"], ((0, 0), (0, 1))).reshape(-1)]))
    Ud = Up.view(400, 13)[:, :10]
    Vd = Vp[1:].view(300, 11)[:, :10]
    got3 = fo.fused_outer(WSLOSS, "t3", Xd, Ud, Vd)
    assert_close(got3.cpu().numpy(), [ref])
    assert fo.fused_outer(WSLOSS, "t3", Xd, to_dev(w["U"]), to_dev(w["V"])).cpu().numpy().tobytes() \
        == got.cpu().numpy().tobytes()


def test_outer_log_chain(fo):
    # sum(X * log(U V^T + eps)), Fig. 1(d)
    w = datagen.outer_workload(500, 400, 20, 0.05, seed=34)
    U, V = np.abs(w["U"]) + 0.01, np.abs(w["V"]) + 0.01
    Xh = host_csr(w)
    chain = [("add", "t0", "d", "s0"), ("log", "t1", "t0"), ("mul", "t2", "a", "t1")]
    ref = oracle.outer(chain, "t2", Xh, U, V, [1e-15], mode="masked")
    got = fo.fused_outer(chain, "t2", csr_to_dev(w), to_dev(U), to_dev(V), [1e-15])
    assert_close(got.cpu().numpy(), [ref])


@pytest.fixture
def outer_schedule(fo):
    """Sets the schedule knob of fused_outer for one test and clears it afterwards."""
    def choose(name):
        fo.tune("outer.kernel", name)
    yield choose
    fo.tune("outer.kernel", None)


@pytest.mark.parametrize("rows,cols,rank,density", [
    (64, 64, 8, 1.0), (200, 300, 100, 1.0), (129, 257, 100, 0.3), (130, 70, 128, 0.5), (1000, 90, 34, 0.2),
    (65, 1000, 10, 0.9)])
@pytest.mark.parametrize("agg", ["full", "none"])
def test_outer_dense_schedule(fo, rows, cols, rank, density, agg):
    """Densely stored main inputs run the tiled schedule (every tile of U V^T formed on
    the tensor cores, stored cells sample it): against the dense-mode checker, which
    forms U V^T outright, and against the per-cell schedule on the same input."""
    w, Xh = outer_case(rows, cols, rank, density, seed=44)
    w["vals"][::5] = 0.0                  # stored zeros are visited like any stored cell
    Xh = host_csr(w)
    Xd, Ud, Vd = csr_to_dev(w), to_dev(w["U"]), to_dev(w["V"])
    ref = oracle.outer(WSLOSS, "t3", Xh, w["U"], w["V"], agg=agg, mode="dense")
    got = fo.fused_outer(WSLOSS, "t3", Xd, Ud, Vd, agg=agg).cpu().numpy()        # picks the tiled schedule itself
    assert_close(got, ref, what="outer tiled %s" % agg)
    try:
        fo.tune("outer.kernel", "dense")
        forced = fo.fused_outer(WSLOSS, "t3", Xd, Ud, Vd, agg=agg).cpu().numpy()
        fo.tune("outer.kernel", "pipe")
        per_cell = fo.fused_outer(WSLOSS, "t3", Xd, Ud, Vd, agg=agg).cpu().numpy()
    finally:
        fo.tune("outer.kernel", None)
    assert forced.tobytes() == got.tobytes()
    assert_close(per_cell, ref, what="outer per cell %s" % agg)
    # a generic chain (interpreted) through the same schedule
    gen = [("sub", "t1", "a", "d"), ("abs", "t2", "t1"), ("add", "t3", "t2", 0.25)]
    assert_close(fo.fused_outer(gen, "t3", Xd, Ud, Vd, agg=agg).cpu().numpy(),
                 oracle.outer(gen, "t3", Xh, w["U"], w["V"], agg=agg, mode="dense"), what="outer tiled generic")


@pytest.mark.parametrize("schedule", ["bulk", "pipe", "direct", "dense"])
def test_outer_every_schedule_on_a_sparse_input(fo, outer_schedule, schedule):
    w, Xh = outer_case(700, 900, 100, 0.02, seed=15)
    w["rowptr"] = w["rowptr"].copy()
    Xd, Ud, Vd = csr_to_dev(w), to_dev(w["U"]), to_dev(w["V"])
    outer_schedule(schedule)
    assert fo.device_status() == 0
    for agg in ("full", "none"):
        ref = oracle.outer(WSLOSS, "t3", Xh, w["U"], w["V"], agg=agg, mode="masked")
        got = fo.fused_outer(WSLOSS, "t3", Xd, Ud, Vd, agg=agg).cpu().numpy()
        assert_close(got, ref, what="outer %s %s" % (schedule, agg))
        again = fo.fused_outer(WSLOSS, "t3", Xd, Ud, Vd, agg=agg).cpu().numpy()
        assert again.tobytes() == got.tobytes()
    assert fo.device_status() == 0               # no bounded wait ran out


@pytest.mark.parametrize("rows,cols,rank,density", [
    (257, 129, 34, 0.2), (100, 90, 2, 0.3), (64, 5000, 108, 0.01), (5000, 64, 100, 0.3), (3, 40, 64, 1.0),
    (1, 1, 100, 1.0), (400, 300, 100, 0.0), (300, 200, 128, 0.2), (150, 100, 120, 0.3)])
def test_outer_bulk_copy_schedule_shapes(fo, outer_schedule, rows, cols, rank, density):
    """The schedule that lands factor rows with bulk copies: short rows, rows longer than a
    stage, rows without cells, a single cell, ranks down to one 16-byte piece per row."""
    w, Xh = outer_case(rows, cols, rank, density, seed=16)
    Xd, Ud, Vd = csr_to_dev(w), to_dev(w["U"]), to_dev(w["V"])
    outer_schedule("bulk")
    for agg in ("full", "none") if len(w["vals"]) else ("full",):     # (no cells: nothing to write per cell)
        ref = oracle.outer(WSLOSS, "t3", Xh, w["U"], w["V"], agg=agg, mode="masked")
        got = fo.fused_outer(WSLOSS, "t3", Xd, Ud, Vd, agg=agg).cpu().numpy()
        assert_close(got, ref, what="outer bulk %s rank %d" % (agg, rank))
    assert fo.device_status() == 0


@pytest.mark.parametrize("agg", ["full", "none", "right", "left"])
@pytest.mark.parametrize("rank", [10, 100])
def test_outer_side_inputs(fo, agg, rank):
    """Dense side inputs of the Outer template (Table 1): a matrix read at (i, j), a column
    vector at i, a row vector at j, in one chain; against the checker's masked and dense modes."""
    w, Xh = outer_case(300, 260, rank, 0.05, seed=54)
    m, n = w["rows"], w["cols"]
    S = datagen.uniform(54, 5, m * n, -1.0, 1.0).reshape(m, n)
    r = datagen.uniform(54, 6, m, 0.5, 2.0)
    c = datagen.uniform(54, 7, n, -2.0, 2.0)
    chain = [("sub", "t0", "a", "d"), ("mul", "t1", "t0", "side0"), ("add", "t2", "t1", "side2"),
             ("mul", "t3", "t2", "side1")]                         # ((a - d) * S_ij + c_j) * r_i
    sides_h = [("cell", S), ("row", r), ("col", c)]
    sides_d = [("cell", to_dev(S)), ("row", to_dev(r)), ("col", to_dev(c))]
    ref = oracle.outer(chain, "t3", Xh, w["U"], w["V"], agg=agg, mode="masked", sides=sides_h)
    got = fo.fused_outer(chain, "t3", csr_to_dev(w), to_dev(w["U"]), to_dev(w["V"]), agg=agg,
                         sides=sides_d).cpu().numpy()
    absch = [("sub", "t0", "a", "d"), ("abs", "t0", "t0"), ("mul", "t1", "t0", "side0"), ("add", "t2", "t1", "side2"),
             ("mul", "t3", "t2", "side1")]
    scale = oracle.outer(absch, "t3", Xh, np.abs(w["U"]), np.abs(w["V"]), agg=agg, mode="masked",
                         sides=[("cell", np.abs(S)), ("row", r), ("col", np.abs(c))])
    assert_close(got, ref, absscale=np.abs(scale) + 1e-300, what="outer sides %s" % agg)
    if agg in ("full", "none"):
        assert_close(got, oracle.outer(chain, "t3", Xh, w["U"], w["V"], agg=agg, mode="dense", sides=sides_h),
                     absscale=np.abs(scale) + 1e-300, what="outer sides, dense mode")
    # a side the chain does not read changes nothing: the staged schedule runs, same bits as without sides
    if agg != "left":
        plain = fo.fused_outer(WSLOSS, "t3", csr_to_dev(w), to_dev(w["U"]), to_dev(w["V"]), agg=agg).cpu().numpy()
        unused = fo.fused_outer(WSLOSS, "t3", csr_to_dev(w), to_dev(w["U"]), to_dev(w["V"]), agg=agg,
                                sides=sides_d[:1]).cpu().numpy()
        assert plain.tobytes() == unused.tobytes()


def test_nonzero_count_of_elementwise_results(fo):
    """out_nnz: the number of non-zero values of a no_agg result - the nnz a sparse output
    would store - equals the checker's count exactly (Cell over dense and CSR, Outer)."""
    import torch
    nnz = torch.full((1,), -1, dtype=torch.int64, device="cuda")
    # Cell over CSR: the chain zeroes about half the stored cells, and X stores zeros of its own
    w, Xh = outer_case(900, 700, 4, 0.05, seed=64)
    w["vals"][::7] = 0.0
    Xh = host_csr(w)
    Y = datagen.normal(64, 9, w["rows"] * w["cols"]).reshape(w["rows"], w["cols"])
    chain = [("gt", "t0", "side0", 0.0), ("mul", "t1", "a", "t0")]                 # a * (Y > 0)
    ref = oracle.cell(chain, "t1", Xh, [("cell", Y)], agg="none")
    got = fo.fused_cell(chain, "t1", csr_to_dev(w), [("cell", to_dev(Y))], agg="none", out_nnz=nnz).cpu().numpy()
    assert_close(got, ref, what="cell csr none")
    assert nnz.item() == oracle.count_nonzero(ref) and 0 < nnz.item() < len(ref)
    # Cell over a dense input, ragged size
    Xd = datagen.normal(64, 10, 501 * 333).reshape(501, 333)
    chain = [("max", "t0", "a", 0.0)]                                              # relu: about half are zero
    ref = oracle.cell(chain, "t0", Xd, agg="none")
    got = fo.fused_cell(chain, "t0", to_dev(Xd), agg="none", out_nnz=nnz).cpu().numpy()
    assert got.tobytes() == ref.tobytes()
    assert nnz.item() == oracle.count_nonzero(ref)
    # Outer no_agg: (a != 0) * d keeps the stored zeros of X at zero
    chain = [("ne", "t0", "a", 0.0), ("mul", "t1", "t0", "d")]
    ref = oracle.outer(chain, "t1", Xh, w["U"], w["V"], agg="none", mode="masked")
    got = fo.fused_outer(chain, "t1", csr_to_dev(w), to_dev(w["U"]), to_dev(w["V"]), agg="none",
                         out_nnz=nnz).cpu().numpy()
    assert_close(got, ref, what="outer none")
    assert nnz.item() == oracle.count_nonzero(ref) == np.count_nonzero(w["vals"])
    # an empty result counts zero; an aggregating variant refuses the count
    empty = dict(rows=5, cols=6, rowptr=np.zeros(6, np.int32), colidx=np.zeros(0, np.int32), vals=np.zeros(0))
    fo.fused_cell([("mov", "t0", "a")], "t0", csr_to_dev(empty), agg="none", out_nnz=nnz,
                  out=torch.zeros(1, dtype=torch.float64, device="cuda"))       # (nothing is written to it)
    assert nnz.item() == 0
    with pytest.raises(fo.FusedOpsError):
        fo.fused_cell(chain[:1], "t0", to_dev(Xd), agg="full", out_nnz=nnz)


# ------------------------------------------------------------------ specialised vs interpreted chains
@pytest.mark.parametrize("name,chain,outs,nsides", [
    ("mul2", [("mul", "t0", "a", "side0")], ["t0"], 1),
    ("mul3", XYZ, ["t1"], 2),
    ("mul3-renamed", [("mul", "t5", "a", "side0"), ("mul", "t2", "t5", "side1")], ["t2"], 2),
    ("sq", [("mul", "t0", "a", "a")], ["t0"], 0),
    ("sq-op", [("sq", "t3", "a")], ["t3"], 2),
    ("magg2", [("mul", "t0", "a", "side0"), ("mul", "t1", "a", "side1")], ["t0", "t1"], 2),
    ("magg3", MAGG3, ["t0", "t1", "t2"], 2),
])
def test_specialised_chains_equal_interpreter_bitwise(fo, name, chain, outs, nsides):
    rows, cols = 700, 300
    w = datagen.magg_workload(rows, cols, seed=41)
    sides_h = [("cell", w["Y"]), ("cell", w["Z"])][:nsides]
    X, sides = to_dev(w["X"]), dev_sides(sides_h)
    ref = oracle.magg(chain, outs, w["X"], sides_h)
    absref = oracle.magg(chain + [("abs", o, o) for o in outs], outs, w["X"], sides_h)
    try:
        fo.force_interpreter(False)
        fast = fo.fused_magg(chain, outs, X, sides).cpu().numpy()
        fo.force_interpreter(True)
        slow = fo.fused_magg(chain, outs, X, sides).cpu().numpy()
    finally:
        fo.force_interpreter(False)
    assert fast.tobytes() == slow.tobytes(), name
    assert_close(fast, ref, absscale=absref, what=name)
    if len(outs) == 1:
        for agg in ("row", "col", "none"):
            r = oracle.cell(chain, outs[0], w["X"], sides_h, agg=agg)
            a = oracle.cell(chain + [("abs", outs[0], outs[0])], outs[0], w["X"], sides_h, agg=agg)
            try:
                fo.force_interpreter(False)
                f1 = fo.fused_cell(chain, outs[0], X, sides, agg=agg).cpu().numpy()
                fo.force_interpreter(True)
                f2 = fo.fused_cell(chain, outs[0], X, sides, agg=agg).cpu().numpy()
            finally:
                fo.force_interpreter(False)
            assert f1.tobytes() == f2.tobytes(), (name, agg)
            assert_close(f1, r, absscale=a, what="%s %s" % (name, agg))


@pytest.mark.parametrize("name,chain,out,scalars", [
    ("wsloss", WSLOSS, "t3", []),
    ("wsloss-commuted", [("sub", "t0", "a", "d"), ("sq", "t5", "t0"), ("ne", "t1", "a", 0.0),
                         ("mul", "t0", "t5", "t1")], "t0", []),
    ("xlogd", [("add", "t0", "d", "s0"), ("log", "t1", "t0"), ("mul", "t2", "a", "t1")], "t2", [2.5]),
    ("xlogd-imm", [("add", "t0", 2.5, "d"), ("log", "t1", "t0"), ("mul", "t2", "t1", "a")], "t2", []),
    ("maskdot", [("ne", "t0", "a", 0.0), ("mul", "t1", "t0", "d")], "t1", []),
    ("maskdot-commuted", [("ne", "t3", "a", 0.0), ("mul", "t1", "d", "t3")], "t1", []),
    ("not-inline", [("sub", "t0", "a", "d"), ("abs", "t1", "t0")], "t1", []),
])
@pytest.mark.parametrize("agg", ["full", "none", "right"])
def test_outer_inline_chains_equal_interpreter_bitwise(fo, name, chain, out, scalars, agg):
    w = datagen.outer_workload(300, 257, 20, 0.05, seed=77)
    U, V = w["U"], w["V"]
    X, Ud, Vd = csr_to_dev(w), to_dev(U), to_dev(V)
    try:
        fo.force_interpreter(False)
        fast = fo.fused_outer(chain, out, X, Ud, Vd, scalars, agg=agg).cpu().numpy()
        fo.force_interpreter(True)
        slow = fo.fused_outer(chain, out, X, Ud, Vd, scalars, agg=agg).cpu().numpy()
    finally:
        fo.force_interpreter(False)
    assert fast.tobytes() == slow.tobytes(), (name, agg)
    ref = oracle.outer(chain, out, host_csr(w), U, V, scalars, mode="masked", agg=agg)
    assert_close(fast, np.asarray(ref).reshape(fast.shape), what="%s %s" % (name, agg))
