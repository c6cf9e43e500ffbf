"""Row template with matrix-valued row intermediates (fused_row_b1) against the
CPU checker: t(X) (X V), the inner loop of Eq. 2, generic two-chain programs with
every side kind, both output variants, every compiled kernel shape, ragged tiles,
strided and unaligned inputs.  Tolerance: tests/util.py (relative 1e-10).
"""
import os

import numpy as np
import pytest

import datagen
import oracle
from util import assert_close, csr_to_dev, host_csr, to_dev

pytestmark = pytest.mark.gpu

MLR_PRE = [("mul", "t0", "side0", "d")]
MLR_POST = [("mul", "t0", "side0", "d"), ("mul", "t1", "side0", "rowsum"), ("sub", "t2", "t0", "t1")]


@pytest.fixture(scope="module")
def fo():
    import torch
    assert torch.cuda.is_available()
    import paper_1801_00829_b200 as fo_
    fo_.load_library()
    return fo_


@pytest.fixture(params=["fma", "mma"])
def path(request):
    """Runs a test once on the multiply-add kernels and once with the tensor-core
    kernels preferred (they take over wherever their layout fits)."""
    import paper_1801_00829_b200 as fo_
    fo_.tune("b1.mma", "0" if request.param == "fma" else "1")
    yield request.param
    fo_.tune("b1.mma", None)


def mm_scale(X, V):
    aX = np.abs(X)
    return aX.T @ (aX @ np.abs(V))


def mlr_scale(X, V, P):
    aX = np.abs(X)
    Q = P * (aX @ np.abs(V))
    return aX.T @ (Q + P * Q.sum(axis=1, keepdims=True))


# (rows, cols, k): k = 1..32, narrow and wide rows, odd sizes, ragged last tiles
SHAPES = [(2000, 1000, 2), (5000, 100, 2), (3001, 100, 4), (3000, 100, 8), (2500, 100, 16), (1501, 100, 32),
          (777, 64, 3), (513, 200, 5), (1000, 512, 16), (600, 1024, 8), (300, 2048, 4), (150, 4096, 2),
          (97, 31, 7), (64, 2, 1), (50001, 10, 2), (40001, 10, 4), (30000, 16, 4), (25000, 8, 8), (9999, 7, 3), (20000, 16, 2), (900, 102, 9), (700, 160, 20), (500, 500, 12), (650, 1000, 8), (800, 64, 32), (300, 230, 17), (1, 10, 2), (5, 1, 3), (1200, 256, 32), (40, 999, 2), (333, 250, 24)]


@pytest.mark.parametrize("rows,cols,k", SHAPES)
def test_b1_mmchain(fo, path, rows, cols, k):
    w = datagen.row_b1_workload(rows, cols, k, seed=5)
    ref = oracle.mmchain(w["X"], w["V"])
    got = fo.fused_row_b1(None, None, [], "d", to_dev(w["X"]), to_dev(w["V"]), agg="col_t")
    assert tuple(got.shape) == (cols, k)
    assert_close(got.cpu().numpy(), ref, absscale=mm_scale(w["X"], w["V"]), what="mmchain %dx%d k=%d" % (rows, cols, k))
    assert fo.device_status() == 0


@pytest.mark.parametrize("rows,cols,k", SHAPES)
def test_b1_mlogreg(fo, path, rows, cols, k):
    w = datagen.row_b1_workload(rows, cols, k, seed=6)
    X, V, P = w["X"], w["V"], w["P"]
    ref = oracle.mlogreg_inner(X, V, P)
    got = fo.fused_row_b1(MLR_PRE, "t0", MLR_POST, "t2", to_dev(X), to_dev(V), [("cell", to_dev(P))], agg="col_t")
    assert_close(got.cpu().numpy(), ref, absscale=mlr_scale(X, V, P), what="mlogreg %dx%d k=%d" % (rows, cols, k))
    # the row intermediates themselves
    refT = oracle.row_b1(MLR_PRE, "t0", MLR_POST, "t2", X, V, [("cell", P)], agg="none")
    gotT = fo.fused_row_b1(MLR_PRE, "t0", MLR_POST, "t2", to_dev(X), to_dev(V), [("cell", to_dev(P))], agg="none")
    aD = np.abs(X) @ np.abs(V)
    Q = P * aD
    assert_close(gotT.cpu().numpy(), refT, absscale=Q + P * Q.sum(axis=1, keepdims=True), what="mlogreg T")
    assert fo.device_status() == 0


@pytest.mark.parametrize("rows,cols,k", [(1000, 100, 3), (700, 1000, 2), (400, 300, 8), (90, 64, 32), (30000, 10, 3),
                                         (20000, 5, 8)])
def test_b1_generic_chains_all_side_kinds(fo, path, rows, cols, k):
    # T_ic = (d * rvec_c + cvec_i * P_ic) * s0 - exp(-|rowsum|),  rowsum = sum_c P_ic * d
    w = datagen.row_b1_workload(rows, cols, k, seed=7)
    X, V, P = w["X"], w["V"], w["P"]
    cvec = datagen.normal(7, 9, rows)
    rvec = datagen.normal(7, 10, k)
    pre = [("mul", "t0", "side2", "d")]
    post = [("mul", "t0", "d", "side0"), ("mul", "t1", "side1", "side2"), ("add", "t2", "t0", "t1"),
            ("mul", "t3", "t2", "s0"), ("abs", "t4", "rowsum"), ("neg", "t5", "t4"), ("exp", "t6", "t5"),
            ("sub", "t7", "t3", "t6")]
    sides_h = [("col", rvec), ("row", cvec), ("cell", P)]
    sides_d = [(a, to_dev(x)) for a, x in sides_h]
    for agg in ("none", "col_t"):
        ref = oracle.row_b1(pre, "t0", post, "t7", X, V, sides_h, [1.5], agg=agg)
        got = fo.fused_row_b1(pre, "t0", post, "t7", to_dev(X), to_dev(V), sides_d, [1.5], agg=agg)
        aD = np.abs(X) @ np.abs(V)
        tscale = (aD * np.abs(rvec)[None, :] + np.abs(cvec)[:, None] * P) * 1.5 + 1.0
        scale = tscale if agg == "none" else np.abs(X).T @ tscale
        assert_close(got.cpu().numpy(), ref, absscale=scale, what="generic %s" % agg)
    # a second chain without a first one: T = d * d
    ref = oracle.row_b1(None, None, [("sq", "t0", "d")], "t0", X, V, agg="col_t")
    got = fo.fused_row_b1(None, None, [("sq", "t0", "d")], "t0", to_dev(X), to_dev(V), agg="col_t")
    assert_close(got.cpu().numpy(), ref, absscale=np.abs(X).T @ (np.abs(X) @ np.abs(V)) ** 2)
    assert fo.device_status() == 0


def test_b1_inline_and_interpreted_chains_agree_bitwise(fo, path):
    # the Eq. 2 chains are evaluated inline; the same arithmetic written with an extra
    # (no-op) step goes through the interpreter and must give the same bits
    rows, cols, k = 4000, 100, 4
    w = datagen.row_b1_workload(rows, cols, k, seed=8)
    args = (to_dev(w["X"]), to_dev(w["V"]), [("cell", to_dev(w["P"]))])
    a = fo.fused_row_b1(MLR_PRE, "t0", MLR_POST, "t2", *args, agg="col_t").cpu().numpy()
    post2 = MLR_POST + [("mov", "t3", "t2")]
    b = fo.fused_row_b1(MLR_PRE, "t0", post2, "t3", *args, agg="col_t").cpu().numpy()
    assert a.tobytes() == b.tobytes()
    # repeated calls: same bits
    c = fo.fused_row_b1(MLR_PRE, "t0", MLR_POST, "t2", *args, agg="col_t").cpu().numpy()
    assert a.tobytes() == c.tobytes()


@pytest.mark.parametrize("shape", ["1,8,2", "2,4,2", "4,2,2", "1,4,4", "2,2,4", "1,2,8"])
def test_b1_every_compiled_shape(fo, shape):
    nch, r, kl = (int(x) for x in shape.split(","))
    k = kl if kl > 2 else 2
    rows, cols = 3000 + r - 1, 200
    w = datagen.row_b1_workload(rows, cols, k, seed=9)
    fo.tune("b1.shape", shape)
    fo.tune("b1.mma", "0")
    try:
        for kk in (k, 2 * k):
            ww = w if kk == k else datagen.row_b1_workload(rows, cols, kk, seed=9)
            X, V, P = ww["X"], ww["V"], ww["P"]
            ref = oracle.mlogreg_inner(X, V, P)
            got = fo.fused_row_b1(MLR_PRE, "t0", MLR_POST, "t2", to_dev(X), to_dev(V), [("cell", to_dev(P))])
            assert_close(got.cpu().numpy(), ref, absscale=mlr_scale(X, V, P), what="shape %s k=%d" % (shape, kk))
    finally:
        fo.tune("b1.shape", None)
        fo.tune("b1.mma", None)
    assert fo.device_status() == 0


def test_b1_strided_unaligned_inputs(fo, path):
    rows, cols, ld, k, ldv = 333, 120, 130, 3, 5
    flat = datagen.normal(5, 0, rows * ld + 1)
    Vflat = datagen.normal(5, 2, cols * ldv)
    Pflat = datagen.uniform(5, 3, rows * 4 + 1)
    Vh = Vflat.reshape(cols, ldv)[:, :k]
    Vd = to_dev(Vflat).view(cols, ldv)[:, :k]
    for off in (0, 1):
        Xh = flat[off:off + rows * ld].reshape(rows, ld)[:, :cols]
        Xd = to_dev(flat)[off:off + rows * ld].view(rows, ld)[:, :cols]
        Ph = Pflat[off:off + rows * 4].reshape(rows, 4)[:, :k]
        Pd = to_dev(Pflat)[off:off + rows * 4].view(rows, 4)[:, :k]
        ref = oracle.mlogreg_inner(Xh, Vh, Ph)
        got = fo.fused_row_b1(MLR_PRE, "t0", MLR_POST, "t2", Xd, Vd, [("cell", Pd)])
        assert_close(got.cpu().numpy(), ref, absscale=mlr_scale(Xh, Vh, Ph), what="strided off=%d" % off)
    assert fo.device_status() == 0


def test_b1_many_tiles_per_group(fo, path):
    # far more tiles than ring slots: every slot is refilled many times
    rows, cols, k = 60011, 100, 2
    w = datagen.row_b1_workload(rows, cols, k, seed=10)
    ref = oracle.mmchain(w["X"], w["V"])
    got = fo.fused_row_b1(None, None, [], "d", to_dev(w["X"]), to_dev(w["V"]))
    assert_close(got.cpu().numpy(), ref, absscale=mm_scale(w["X"], w["V"]))
    assert fo.device_status() == 0


def test_b1_empty_and_limits(fo):
    import torch
    dev = torch.device("cuda")
    V = to_dev(datagen.normal(5, 2, 8 * 2).reshape(8, 2))
    X0 = torch.empty((0, 8), dtype=torch.float64, device=dev)
    got = fo.fused_row_b1(None, None, [], "d", X0, V)
    assert got.cpu().numpy().tolist() == [[0.0, 0.0]] * 8
    assert tuple(fo.fused_row_b1(None, None, [], "d", X0, V, agg="none").shape) == (0, 2)
    # beyond the limits: an error code, nothing launched
    Xw = torch.zeros((4, 8), dtype=torch.float64, device=dev)
    V33 = torch.zeros((8, 33), dtype=torch.float64, device=dev)
    with pytest.raises(fo.FusedOpsError) as e:
        fo.fused_row_b1(None, None, [], "d", Xw, V33)
    assert e.value.status == -4
    with pytest.raises(fo.FusedOpsError) as e:          # "rowsum" without a first chain
        fo.fused_row_b1(None, None, [("mov", "t0", "side0")], "t0", Xw, V)
    assert e.value.status == -3
    with pytest.raises(fo.FusedOpsError) as e:          # side of the wrong shape
        fo.fused_row_b1(None, None, [("mul", "t0", "side0", "d")], "t0", Xw, V,
                        [("cell", torch.zeros((4, 3), dtype=torch.float64, device=dev))])
    assert e.value.status == -2


@pytest.mark.parametrize("rows,cols,k,density", [(20000, 1000, 2, 0.01), (5000, 100, 8, 0.1), (3000, 300, 32, 0.05),
                                                 (700, 64, 5, 0.3), (100, 1200, 3, 0.001), (33, 9, 1, 0.5),
                                                 (400, 600, 16, 0.4), (50, 40, 2, 0.0)])
def test_b1_csr_rows(fo, rows, cols, k, density):
    """The same operator over a CSR X (the listing's sparse binding), against the checker."""
    w = datagen.row_csr_workload(rows, cols, density, seed=3)
    Xh = host_csr(w)
    b = datagen.row_b1_workload(rows, cols, k, seed=5)
    V, P = b["V"], b["P"]
    absX = dict(Xh, vals=np.abs(w["vals"]))
    tabs = oracle.row_b1(None, None, [("mul", "t0", "d", "side0"), ("mul", "t1", "t0", 2.0)], "t1", absX, np.abs(V),
                         [("cell", P)], agg="none")
    habs = oracle.row_b1(None, None, [("mul", "t0", "d", "side0"), ("mul", "t1", "t0", 2.0)], "t1", absX, np.abs(V),
                         [("cell", P)], agg="col_t")
    for agg, scale in (("col_t", habs), ("none", tabs)):
        ref = oracle.row_b1(MLR_PRE, "t0", MLR_POST, "t2", Xh, V, [("cell", P)], agg=agg)
        got = fo.fused_row_b1(MLR_PRE, "t0", MLR_POST, "t2", csr_to_dev(w), to_dev(V), [("cell", to_dev(P))], agg=agg)
        assert_close(got.cpu().numpy(), ref, absscale=scale, what="b1 csr mlogreg %s" % agg)
    # t(X) (X V), and a generic chain that is not zero at D = 0 (rows without stored cells count)
    ref = oracle.row_b1(None, None, [], "d", Xh, V, agg="col_t")
    got = fo.fused_row_b1(None, None, [], "d", csr_to_dev(w), to_dev(V), agg="col_t")
    assert_close(got.cpu().numpy(), ref, absscale=oracle.row_b1(None, None, [], "d", absX, np.abs(V), agg="col_t"))
    gen = [("add", "t0", "d", 1.0), ("mul", "t1", "t0", "rowsum")]
    genpre = [("abs", "t0", "d")]
    ref = oracle.row_b1(genpre, "t0", gen, "t1", Xh, V, agg="none")
    got = fo.fused_row_b1(genpre, "t0", gen, "t1", csr_to_dev(w), to_dev(V), agg="none")
    aD = oracle.row_b1(None, None, [], "d", absX, np.abs(V), agg="none")
    assert_close(got.cpu().numpy(), ref, absscale=(aD + 1.0) * aD.sum(axis=1, keepdims=True) + 1e-300)
    assert fo.device_status() == 0


@pytest.mark.parametrize("cols,k", [(10, 2), (7, 4), (16, 3), (3, 8)])
def test_b1_narrow_rows_strided_unaligned(fo, cols, k):
    """At most 16 columns: a thread takes whole rows; strided and 8-byte-aligned inputs, and the switch back
    to the wide kernels gives the same values within tolerance."""
    rows, ld = 30011, cols + 3
    flat = datagen.normal(41, 0, rows * ld + 1)
    V = datagen.normal(41, 2, cols * k).reshape(cols, k)
    P = datagen.uniform(41, 3, rows * k).reshape(rows, k) / (k + 1)
    for off in (0, 1):
        Xh = flat[off:off + rows * ld].reshape(rows, ld)[:, :cols]
        Xd = to_dev(flat)[off:off + rows * ld].view(rows, ld)[:, :cols]
        for agg in ("col_t", "none"):
            ref = oracle.row_b1(MLR_PRE, "t0", MLR_POST, "t2", Xh, V, [("cell", P)], agg=agg)
            got = fo.fused_row_b1(MLR_PRE, "t0", MLR_POST, "t2", Xd, to_dev(V), [("cell", to_dev(P))], agg=agg)
            Q = P * (np.abs(Xh) @ np.abs(V))
            tabs = Q + P * Q.sum(axis=1, keepdims=True)
            assert_close(got.cpu().numpy(), ref, absscale=tabs if agg == "none" else np.abs(Xh).T @ tabs,
                         what="b1 narrow %dx%d off=%d %s" % (cols, k, off, agg))
    fo.tune("b1.narrow", "0")
    try:
        wide = fo.fused_row_b1(MLR_PRE, "t0", MLR_POST, "t2", Xd, to_dev(V), [("cell", to_dev(P))]).cpu().numpy()
    finally:
        fo.tune("b1.narrow", None)
    assert_close(wide, oracle.mlogreg_inner(Xh, V, P), absscale=mlr_scale(Xh, V, P))
    assert fo.device_status() == 0
