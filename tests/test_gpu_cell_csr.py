"""Cell and MAgg over a CSR main input (the sparse-safe binding): the chain runs on the stored
cells only, sides are read at each stored cell's position.  Checked against the CPU checker's
own sparse-safe evaluation, element by element."""
import numpy as np
import pytest

import datagen
import oracle
from util import assert_close, csr_to_dev, host_csr, to_dev

pytestmark = pytest.mark.gpu

XYZ = [("mul", "t0", "a", "side0"), ("mul", "t1", "t0", "side1")]
# every side kind and a scalar: (a * Y_ij + r_i) * c_j - s0
MIXED = [("mul", "t0", "a", "side0"), ("add", "t1", "t0", "side1"), ("mul", "t2", "t1", "side2"),
         ("sub", "t3", "t2", "s0")]


@pytest.fixture(scope="module")
def fo():
    import paper_1801_00829_b200 as m
    m.load_library()
    return m


def case(rows, cols, density, seed):
    w = datagen.row_csr_workload(rows, cols, density, seed=seed)
    rng = np.random.default_rng(seed)
    Y = rng.standard_normal((rows, cols))
    Z = rng.standard_normal((rows, cols))
    r = rng.standard_normal(rows)
    c = rng.standard_normal(cols)
    return w, Y, Z, r, c


# mean row lengths 2, 25 and 150: two, eight and thirty-two lanes per row
@pytest.mark.parametrize("rows,cols,density", [(3000, 500, 0.004), (3000, 500, 0.05), (700, 500, 0.3),
                                               (33, 7, 0.5), (1, 1, 1.0)])
@pytest.mark.parametrize("agg", ["full", "row", "col", "none"])
def test_cell_csr_every_side_kind(fo, rows, cols, density, agg):
    w, Y, Z, r, c = case(rows, cols, density, seed=51)
    Xh = host_csr(w)
    sides_h = [("cell", Y), ("row", r), ("col", c)]
    ref = oracle.cell(MIXED, "t3", Xh, sides_h, [0.25], agg=agg)
    scale = oracle.cell(MIXED + [("abs", "t3", "t3")], "t3", Xh,
                        [("cell", np.abs(Y)), ("row", np.abs(r)), ("col", np.abs(c))], [-0.25], agg=agg)
    sides = [(k, to_dev(v)) for k, v in sides_h]
    got = fo.fused_cell(MIXED, "t3", csr_to_dev(w), sides, [0.25], agg=agg).cpu().numpy()
    assert_close(got, np.asarray(ref).reshape(got.shape), absscale=np.asarray(scale).reshape(got.shape),
                 what="cell csr %s" % agg)


@pytest.mark.parametrize("agg", ["full", "row", "none"])
def test_cell_csr_specialised_chain_equals_interpreter_bitwise(fo, agg):
    w, Y, Z, r, c = case(4000, 300, 0.03, seed=52)
    X, sides = csr_to_dev(w), [("cell", to_dev(Y)), ("cell", to_dev(Z))]
    try:
        fo.force_interpreter(False)
        fast = fo.fused_cell(XYZ, "t1", X, sides, agg=agg).cpu().numpy()
        again = fo.fused_cell(XYZ, "t1", X, sides, agg=agg).cpu().numpy()
        fo.force_interpreter(True)
        slow = fo.fused_cell(XYZ, "t1", X, sides, agg=agg).cpu().numpy()
    finally:
        fo.force_interpreter(False)
    assert fast.tobytes() == slow.tobytes() == again.tobytes()
    ref = oracle.cell(XYZ, "t1", host_csr(w), [("cell", Y), ("cell", Z)], agg=agg)
    scale = oracle.cell(XYZ, "t1", host_csr(w), [("cell", np.abs(Y)), ("cell", np.abs(Z))], agg=agg)
    assert_close(fast, np.asarray(ref).reshape(fast.shape), absscale=np.asarray(scale).reshape(fast.shape))


def test_cell_csr_zero_preserving_chain_equals_dense_kernel(fo):
    from datagen.workloads import csr_to_dense
    w, Y, Z, r, c = case(600, 257, 0.1, seed=53)
    Xd = csr_to_dense(600, 257, w["rowptr"], w["colidx"], w["vals"])
    sides = [("cell", to_dev(Y)), ("cell", to_dev(Z))]
    for agg in ("full", "row", "col"):
        sparse = fo.fused_cell(XYZ, "t1", csr_to_dev(w), sides, agg=agg).cpu().numpy()
        dense = fo.fused_cell(XYZ, "t1", to_dev(Xd), sides, agg=agg).cpu().numpy()
        scale = oracle.cell(XYZ, "t1", np.abs(Xd), [("cell", np.abs(Y)), ("cell", np.abs(Z))], agg=agg)
        assert_close(sparse, dense, absscale=np.asarray(scale).reshape(dense.shape), what=agg)


@pytest.mark.parametrize("k", [2, 3, 5, 8])
def test_magg_csr(fo, k):
    w, Y, Z, r, c = case(5000, 200, 0.05, seed=54)
    chain = [("mul", "t0", "a", "side0"), ("mul", "t1", "a", "side1"), ("mul", "t2", "a", "a"),
             ("add", "t3", "t0", "side2"), ("abs", "t4", "a"), ("sub", "t5", "t1", "t2"),
             ("max", "t6", "a", "side0"), ("mov", "t7", "a")][:max(k, 3)]
    outs = ["t%d" % i for i in range(k)]
    sides_h = [("cell", Y), ("cell", Z), ("col", c)]
    ref = oracle.magg(chain, outs, host_csr(w), sides_h)
    absref = oracle.magg(chain + [("abs", o, o) for o in outs], outs, host_csr(w), sides_h)
    got = fo.fused_magg(chain, outs, csr_to_dev(w), [(a, to_dev(v)) for a, v in sides_h]).cpu().numpy()
    assert_close(got, ref, absscale=absref, what="magg csr k=%d" % k)


def test_cell_csr_empty_matrix_and_empty_rows(fo):
    import torch
    dev = torch.device("cuda", 0)
    rowptr = torch.tensor([0, 0, 2, 2, 2, 3], dtype=torch.int32, device=dev)
    colidx = torch.tensor([1, 3, 0], dtype=torch.int32, device=dev)
    vals = torch.tensor([2.0, 0.0, -4.0], dtype=torch.float64, device=dev)       # one stored zero
    X = fo.CSR(5, 4, rowptr, colidx, vals)
    chain = [("add", "t0", "a", 1.0)]            # not zero-preserving: stored cells only
    assert fo.fused_cell(chain, "t0", X, agg="full").cpu().tolist() == [1.0]
    assert fo.fused_cell(chain, "t0", X, agg="row").cpu().tolist() == [0.0, 4.0, 0.0, 0.0, -3.0]
    assert fo.fused_cell(chain, "t0", X, agg="col").cpu().tolist() == [-3.0, 3.0, 0.0, 1.0]
    assert fo.fused_cell(chain, "t0", X, agg="none").cpu().tolist() == [3.0, 1.0, -3.0]
    E = fo.CSR(3, 4, torch.zeros(4, dtype=torch.int32, device=dev),
               torch.zeros(0, dtype=torch.int32, device=dev), torch.zeros(0, dtype=torch.float64, device=dev))
    assert fo.fused_cell(chain, "t0", E, agg="full").cpu().tolist() == [0.0]
    assert fo.fused_cell(chain, "t0", E, agg="row").cpu().tolist() == [0.0, 0.0, 0.0]
    assert fo.fused_cell(chain, "t0", E, agg="col").cpu().tolist() == [0.0] * 4
    assert fo.fused_magg(chain + [("mov", "t1", "a")], ["t0", "t1"], E).cpu().tolist() == [0.0, 0.0]


@pytest.mark.parametrize("rows,cols,dx,dy", [(3000, 1000, 0.1, 0.1), (500, 64, 0.3, 0.5), (100, 4000, 0.01, 0.02),
                                             (33, 17, 0.5, 0.0), (2000, 300, 0.02, 0.9)])
def test_cell_csr_sparse_sides(fo, rows, cols, dx, dy):
    """A sparse driver with sparse side inputs (Section 5.2, "Cell Operations" over sparse data)."""
    import datagen
    rp, ci, xv = datagen.csr_bernoulli(21, 0, rows, cols, dx, 0.5, 1.5)
    X = dict(rows=rows, cols=cols, rowptr=rp, colidx=ci, vals=xv)
    rp2, ci2, yv = datagen.csr_bernoulli(21, 4, rows, cols, dy, -1.0, 1.0)
    Y = dict(rows=rows, cols=cols, rowptr=rp2, colidx=ci2, vals=yv)
    rp3, ci3, zv = datagen.csr_bernoulli(21, 8, rows, cols, 0.5, -1.0, 1.0)
    Z = dict(rows=rows, cols=cols, rowptr=rp3, colidx=ci3, vals=zv)
    W = datagen.normal(21, 12, rows * cols).reshape(rows, cols)
    Xd, Yd_, Zd_ = csr_to_dev(X), csr_to_dev(Y), csr_to_dev(Z)
    xyz = [("mul", "t0", "a", "side0"), ("mul", "t1", "t0", "side1")]
    absX = dict(X, vals=np.abs(xv))
    absY = dict(Y, vals=np.abs(yv))
    absZ = dict(Z, vals=np.abs(zv))
    for agg in ("full", "row", "col", "none"):
        ref = oracle.cell(xyz, "t1", X, [("cell", Y), ("cell", Z)], agg=agg)
        got = fo.fused_cell(xyz, "t1", Xd, [("cell", Yd_), ("cell", Zd_)], agg=agg)
        scale = oracle.cell(xyz, "t1", absX, [("cell", absY), ("cell", absZ)], agg=agg)
        assert_close(got.cpu().numpy(), ref, absscale=scale, what="sparse sides %s" % agg)
    # sparse and dense sides mixed, a chain that is not zero-preserving in the sparse side, MAgg
    chain = [("add", "t0", "side0", 1.0), ("mul", "t1", "a", "t0"), ("mul", "t2", "a", "side1")]
    ref = oracle.magg(chain, ["t1", "t2"], X, [("cell", Y), ("cell", W)])
    got = fo.fused_magg(chain, ["t1", "t2"], Xd, [("cell", Yd_), ("cell", to_dev(W))])
    scale = oracle.magg([("abs", "t3", "side0"), ("add", "t0", "t3", 1.0), ("mul", "t1", "a", "t0"),
                         ("abs", "t4", "side1"), ("mul", "t2", "a", "t4")], ["t1", "t2"], absX,
                        [("cell", Y), ("cell", W)])
    assert_close(got.cpu().numpy(), ref, absscale=scale, what="sparse sides magg")
    # a dense main input refuses a sparse side
    with pytest.raises(fo.FusedOpsError) as e:
        fo.fused_cell(xyz, "t1", to_dev(W), [("cell", Yd_), ("cell", to_dev(W))])
    assert e.value.status == -4
