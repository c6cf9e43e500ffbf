"""Host-side checks of the C ABI that need no GPU: the library builds, loads and
exports every function the headers under include/ declare; workspace sizes are plain
arithmetic; invalid arguments are refused with the documented status before
anything touches the device."""
import ctypes as C
import glob
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

import paper_1801_00829_b200.binding as B  # noqa: E402


@pytest.fixture(scope="module")
def lib():
    return B.load_library()


def declared_functions():
    names = []
    for header in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))):
        text = open(header).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"^(?:int|size_t|const char \*)\s*(\w+)\s*\(", text, flags=re.M)
    return names


def test_header_functions_are_exported(lib):
    names = declared_functions()
    assert set(names) == set(B.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings(lib):
    seen = set()
    for code in range(0, -9, -1):
        s = lib.fo_status_string(code).decode()
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 9
    assert lib.fo_status_string(-99).decode() == "unknown status"


def dense_mat(rows, cols, ld=None, ptr=0x1000):
    m = B.fo_mat()
    m.kind = 0
    m.dense.rows, m.dense.cols, m.dense.ld, m.dense.data = rows, cols, ld or cols, ptr
    return m


HEAD = 16384        # control words at the head of every workspace


def test_workspace_sizes(lib):
    m = dense_mat(1000, 1000)
    full = lib.fused_cell_workspace_bytes(C.byref(m), 3)
    assert full >= HEAD + 8 and full % 8 == 0
    assert lib.fused_cell_workspace_bytes(C.byref(m), 1) == HEAD           # row_agg: control words only
    col = lib.fused_cell_workspace_bytes(C.byref(m), 2)
    assert col >= HEAD + 1000 * 8 and (col - HEAD) % (1000 * 8) == 0
    assert lib.fused_cell_workspace_bytes(C.byref(m), 9) == 0
    assert lib.fused_magg_workspace_bytes(C.byref(m), 3) == HEAD + (full - HEAD) * 3
    assert lib.fused_magg_workspace_bytes(C.byref(m), 9) == 0
    r = lib.fused_row_workspace_bytes(C.byref(m), 4)
    assert r >= HEAD + 148 * 1000 * 8
    assert lib.fused_row_workspace_bytes(C.byref(m), 0) == HEAD          # no_agg: control words only
    assert lib.fused_row_workspace_bytes(C.byref(m), 2) == r             # col_agg holds what col_t_agg holds
    assert lib.fused_row_workspace_bytes(C.byref(m), 9) == 0
    x = B.fo_csr()
    x.rows, x.cols, x.nnz = 10, 10, 5
    assert lib.fused_outer_workspace_bytes(C.byref(x), 100, 3) >= HEAD + 8
    assert lib.fused_outer_workspace_bytes(C.byref(x), 257, 3) == 0


def call_cell(lib, steps, output, m, sides=(), n_scalars=0, agg=3, ws=0x10000, ws_bytes=1 << 24,
              out=0x2000):
    ch, keep = B.make_chain(steps, output)
    sarr = (B.fo_side * max(1, len(sides)))(*sides)
    sc = (C.c_double * 8)()
    return lib.fused_cell(C.byref(ch), C.byref(m), sarr, len(sides), sc, n_scalars, agg,
                          C.c_void_p(out), None, C.c_void_p(ws), ws_bytes, None)


def side(rows, cols, access, ptr=0x3000):
    s = B.fo_side()
    s.m.rows, s.m.cols, s.m.ld, s.m.data = rows, cols, cols, ptr
    s.access = access
    return s


def test_cell_argument_errors(lib):
    m = dense_mat(10, 10)
    ok_chain = [("mul", "t0", "a", "a")]
    assert call_cell(lib, ok_chain, "t0", m, out=0) == -1                        # FO_ERR_NULL
    assert call_cell(lib, ok_chain, "t0", dense_mat(10, 10, ld=5)) == -2         # ld < cols
    assert call_cell(lib, ok_chain, "t0", m, agg=7) == -4                        # unknown variant
    assert call_cell(lib, [("mul", "t0", "a", "t1")], "t0", m) == -3             # use before definition
    assert call_cell(lib, [("mul", "t0", "a", "d")], "t0", m) == -3              # no dot product in Cell
    assert call_cell(lib, [("mul", "t0", "a", "side0")], "t0", m) == -3          # side not passed
    assert call_cell(lib, [("mul", "t0", "a", "s0")], "t0", m) == -3             # scalar not passed
    assert call_cell(lib, ok_chain, "t5", m) == -3                               # undefined output
    assert call_cell(lib, ok_chain, "t0", m, sides=[side(9, 10, 0)]) == -2       # side shape
    assert call_cell(lib, ok_chain, "t0", m, sides=[side(10, 1, 2)]) == -2       # row vector expected
    assert call_cell(lib, ok_chain, "t0", m, ws=0) == -5                         # no workspace
    assert call_cell(lib, ok_chain, "t0", m, ws=0x10008) == -5                   # misaligned
    assert call_cell(lib, ok_chain, "t0", m, ws_bytes=16) == -5                  # too small
    bad = B.fo_mat()
    bad.kind = 5
    assert call_cell(lib, ok_chain, "t0", bad) == -2


def test_sparse_side_is_refused_outside_the_sparse_driver_kernels(lib):
    y = B.fo_csr()
    y.rows, y.cols, y.nnz = 10, 10, 5
    y.rowptr, y.colidx, y.vals = 0x5000, 0x6000, 0x7000
    sd = (B.fo_side * 1)()
    sd[0].access = 0
    sd[0].sparse = C.addressof(y)
    ch, keep = B.make_chain([("mul", "t0", "a", "side0")], "t0")
    sc = (C.c_double * 8)()
    m = dense_mat(10, 10)
    assert lib.fused_cell(C.byref(ch), C.byref(m), sd, 1, sc, 0, 3, C.c_void_p(0x2000), None,
                          C.c_void_p(0x10000), 1 << 24, None) == -4
    # over a CSR main input: the side must have the main input's shape and be read at the cell
    x = B.fo_mat()
    x.kind = 1
    x.csr.rows, x.csr.cols, x.csr.nnz = 10, 12, 5
    x.csr.rowptr, x.csr.colidx, x.csr.vals = 0x5000, 0x6000, 0x7000
    assert lib.fused_cell(C.byref(ch), C.byref(x), sd, 1, sc, 0, 3, C.c_void_p(0x2000), None,
                          C.c_void_p(0x10000), 1 << 24, None) == -2


def test_chain_limits(lib):
    m = dense_mat(4, 4)
    long_chain = [("add", "t0", "a", 1.0)] + [("add", "t0", "t0", 1.0)] * 31
    ch, keep = B.make_chain(long_chain, "t0")
    assert ch.n_ops == 32
    too_long = long_chain + [("add", "t0", "t0", 1.0)]
    assert call_cell(lib, too_long, "t0", m) == -3
    ch, keep = B.make_chain([("mov", "t0", "a")], "t0")
    keep[0].opcode = 200
    sarr = (B.fo_side * 1)()
    sc = (C.c_double * 8)()
    assert lib.fused_cell(C.byref(ch), C.byref(m), sarr, 0, sc, 0, 3, C.c_void_p(0x2000), None,
                          C.c_void_p(0x10000), 1 << 24, None) == -3
    # a count of non-zero results needs an elementwise result
    ok, keep_ok = B.make_chain([("mov", "t0", "a")], "t0")
    assert lib.fused_cell(C.byref(ok), C.byref(m), sarr, 0, sc, 0, 3, C.c_void_p(0x2000), C.c_void_p(0x4000),
                          C.c_void_p(0x10000), 1 << 24, None) == -4


def test_row_and_outer_argument_errors(lib):
    ch, keep = B.make_chain([("mul", "t0", "side0", "d")], "t0")
    m = dense_mat(10, 10000)
    sarr = (B.fo_side * 1)(side(10, 1, 1))
    sc = (C.c_double * 8)()

    def row(mat, agg=4, sides=sarr, ns=1, chain=ch, v=0x4000):
        return lib.fused_row(C.byref(chain), C.byref(mat), C.c_void_p(v), sides, ns, sc, 0, agg,
                             C.c_void_p(0x2000), C.c_void_p(0x10000), 1 << 30, None)

    assert row(m) == -4                                   # too wide for the single-pass kernel
    assert row(dense_mat(10, 100), agg=5) == -4           # the B1 variants belong to fused_row_b1
    assert row(dense_mat(10, 100), agg=9) == -4           # no such variant
    assert row(dense_mat(10, 100), v=0) == -1
    bad_side = (B.fo_side * 1)(side(10, 100, 0))
    assert row(dense_mat(10, 100), sides=bad_side) == -2  # Row sides are read at the row index
    ch2, keep2 = B.make_chain([("mul", "t0", "a", "d")], "t0")
    assert row(dense_mat(10, 100), chain=ch2, ns=0) == -3  # no main value in Row

    x = B.fo_csr()
    x.rows, x.cols, x.nnz = 10, 12, 5
    x.rowptr, x.colidx, x.vals = 0x5000, 0x6000, 0x7000
    u, v = B.fo_dense(), B.fo_dense()
    u.rows, u.cols, u.ld, u.data = 10, 4, 4, 0x8000
    v.rows, v.cols, v.ld, v.data = 12, 4, 4, 0x9000
    ch3, keep3 = B.make_chain([("sub", "t0", "a", "d")], "t0")

    no_sides = (B.fo_side * 1)()

    def outer(xx=x, uu=u, vv=v, agg=3, chain=ch3, sides=no_sides, ns=0, nnz=None):
        return lib.fused_outer(C.byref(chain), C.byref(xx), C.byref(uu), C.byref(vv), sides, ns, sc, 0, agg,
                               C.c_void_p(0x2000), nnz, C.c_void_p(0x10000), 1 << 24, None)

    v2 = B.fo_dense()
    v2.rows, v2.cols, v2.ld, v2.data = 12, 5, 5, 0x9000
    assert outer(vv=v2) == -2                             # rank mismatch
    u2 = B.fo_dense()
    u2.rows, u2.cols, u2.ld, u2.data = 11, 4, 4, 0x8000
    assert outer(uu=u2) == -2                             # U.rows != X.rows
    assert outer(agg=7) == -4                             # no such variant
    x2 = B.fo_csr()
    x2.rows, x2.cols, x2.nnz = 10, 12, 1 << 31
    x2.rowptr, x2.colidx, x2.vals = 0x5000, 0x6000, 0x7000
    assert outer(xx=x2) == -4
    # side inputs of the Outer template: dense, at most three, shaped like X under their access kind
    ch4, keep4 = B.make_chain([("mul", "t0", "d", "side0")], "t0")
    assert outer(chain=ch4) == -3                          # the chain names a side that is not passed
    assert outer(chain=ch4, sides=(B.fo_side * 1)(side(10, 1, 1)), ns=1, agg=7) == -4
    assert outer(chain=ch4, sides=(B.fo_side * 1)(side(10, 12, 1)), ns=1) == -2     # a column vector is rows x 1
    assert outer(chain=ch4, sides=(B.fo_side * 1)(side(1, 10, 2)), ns=1) == -2      # a row vector is 1 x cols
    assert outer(chain=ch4, sides=(B.fo_side * 4)(*[side(10, 1, 1)] * 4), ns=4) == -4
    assert outer(nnz=C.c_void_p(0x4000)) == -4             # a count needs the no_agg variant


def test_row_b1_argument_errors(lib):
    # every error is found on the host, before anything is launched (no GPU here)
    pre, k1 = B.make_chain([("mul", "t0", "side0", "d")], "t0")
    post, k2 = B.make_chain([("mul", "t0", "side0", "rowsum")], "t0", rowsum_side=1)
    ident, k3 = B.make_chain([], "d")
    sc = (C.c_double * 8)()

    def dense(rows, cols, ld=None, data=0x9000):
        d = B.fo_dense()
        d.rows, d.cols, d.ld, d.data = rows, cols, ld or cols, data
        return d

    def call(mat, bmat, agg=6, sides=None, ns=0, prec=None, postc=ident, ws_bytes=1 << 30):
        sarr = sides if sides is not None else (B.fo_side * 1)()
        return lib.fused_row_b1(C.byref(prec) if prec is not None else None, C.byref(postc), C.byref(mat),
                                C.byref(bmat), sarr, ns, sc, 0, agg, C.c_void_p(0x2000),
                                C.c_void_p(0x10000), ws_bytes, None)

    m = dense_mat(10, 100)
    assert call(m, dense(100, 33)) == -4                    # more than 32 classes
    assert call(m, dense(99, 2)) == -2                      # B.rows != X.cols
    assert call(m, dense(100, 2), agg=4) == -4              # not a B1 variant
    assert call(dense_mat(10, 5000), dense(5000, 2)) == -4  # too wide
    assert call(dense_mat(10, 2000), dense(2000, 16)) == -4  # n * k beyond the output tile
    assert call(m, dense(100, 2), ws_bytes=1024) == -5
    one = (B.fo_side * 1)(side(10, 2, 0))
    bad = (B.fo_side * 1)(side(10, 3, 0))
    assert call(m, dense(100, 2), sides=bad, ns=1, prec=pre, postc=post) == -2   # cell side must be rows x k
    assert call(m, dense(100, 2), sides=one, ns=1, prec=None, postc=post) == -3  # row sum without a first chain
    x = B.fo_mat()
    x.kind = 1
    x.csr.rows, x.csr.cols, x.csr.nnz = 10, 100, 1 << 31
    x.csr.rowptr, x.csr.colidx, x.csr.vals = 0x5000, 0x6000, 0x7000
    assert call(x, dense(100, 2)) == -4                     # CSR main input: nnz must fit 31 bits
    x.csr.nnz, x.csr.cols = 50, 2000
    assert call(x, dense(2000, 8)) == -4                    # CSR main input: n * k beyond the shared tiles
    # workspace: one n x k tile per CTA and per group of CTAs for col_agg_B1_T, the head alone otherwise
    assert lib.fused_row_b1_workspace_bytes(C.byref(m), 2, 5) == 16384
    assert lib.fused_row_b1_workspace_bytes(C.byref(m), 2, 6) > 16384 + 148 * 100 * 2 * 8
    assert lib.fused_row_b1_workspace_bytes(C.byref(m), 0, 6) == 0


def test_make_chain_rejects_bad_text():
    with pytest.raises(ValueError):
        B.make_chain([("frobnicate", "t0", "a")], "t0")
    with pytest.raises(ValueError):
        B.make_chain([("add", "t0", "a")], "t0")
    with pytest.raises(ValueError):
        B.make_chain([("add", "x0", "a", "a")], "t0")
    with pytest.raises(ValueError):
        B.make_chain([("add", "t0", 1.0, 2.0)], "t0")
    with pytest.raises(ValueError):
        B.make_chain([("mov", "t0", "a")], 1.0)


def test_cost_model_worked_example():
    """Section 4.3: reading a 100M x 10 dense matrix at 32 GB/s takes 0.25 s."""
    from paper_1801_00829_b200 import algorithmic_bytes, ideal_seconds
    golden = open(os.path.join(ROOT, "tests", "golden", "cost_model_example.txt")).read()
    vals = dict(l.split("=") for l in golden.split() if "=" in l)
    nbytes = int(vals["rows"]) * int(vals["cols"]) * 8
    assert abs(ideal_seconds(nbytes, float(vals["gb_per_s"])) - float(vals["seconds"])) < 1e-12
    assert algorithmic_bytes("cell", rows=1000, cols=1000, n_inputs=3) == 24_000_008
    assert algorithmic_bytes("row_dense", rows=10**6, cols=1000) == 8 * 10**9 + 8 * 10**6 + 16000


def test_chain_describe_writes_the_arithmetic_not_the_temporaries():
    import paper_1801_00829_b200 as fo
    from paper_1801_00829_b200.binding import FusedOpsError
    wsloss = [("ne", "t0", "a", 0.0), ("sub", "t1", "a", "d"), ("mul", "t2", "t1", "t1"), ("mul", "t3", "t0", "t2")]
    renamed = [("ne", "t7", "a", 0.0), ("sub", "t0", "a", "d"), ("sq", "t0", "t0"), ("mul", "t1", "t7", "t0")]
    a = fo.chain_describe(wsloss, "t3", use="outer")
    b = fo.chain_describe(renamed, "t1", use="outer")
    assert a == b == "mul(ne(r0,k8),mul(sub(r0,r1),sub(r0,r1)))"       # Eq. 1; sq(x) reads mul(x,x)
    assert fo.chain_describe([("mul", "t0", "a", "side0"), ("mul", "t1", "t0", "side1")], "t1",
                             use="cell", n_sides=2) == "mul(mul(r0,r1),r2)"
    assert fo.chain_describe([("mul", "t0", "side0", "d")], "t0", use="row", n_sides=1) == "mul(r1,r0)"
    assert fo.chain_describe([("add", "t0", "d", "s0"), ("log", "t1", "t0"), ("mul", "t2", "a", "t1")], "t2",
                             use="outer", scalars=[1e-15]) == "mul(r0,log(add(r1,k0)))"
    # several outputs, and an output that is an input
    magg = [("mul", "t0", "a", "side0"), ("mul", "t1", "a", "a")]
    assert fo.chain_describe(magg, ["t0", "t1"], use="cell", n_sides=1, k=1) == "mul(r0,r0)"
    assert fo.chain_describe([], "a", use="cell") == "r0"
    with pytest.raises(FusedOpsError):
        fo.chain_describe(magg, ["t0", "t1"], use="cell", n_sides=1, k=2)
    with pytest.raises(FusedOpsError):
        fo.chain_describe([("mul", "t0", "a", "side3")], "t0", use="cell", n_sides=1)


def test_cost_model_form_and_plans():
    # Section 4.3: C = sum over operators of T_w + max(T_r, T_c)
    from paper_1801_00829_b200 import operator_cost, operator_sizes, plan_cost, unfused_plan_sizes
    # the worked example is the read term of an I/O-bound operator with nothing to write
    assert abs(operator_cost(1e9 * 8, 0, 0, 32, 32, 1) - 0.25) < 1e-12
    # compute-bound: the larger of read and compute counts, the write time adds
    assert abs(operator_cost(8e9, 16e9, 230.4e9 * 2, 32, 32, 230.4) - (0.5 + 2.0)) < 1e-12
    # a fused Cell operator reads its three inputs once; the unfused plan also writes and
    # re-reads two intermediates: 3 reads against 5 reads + 2 writes of m*n doubles
    kw = dict(rows=1000, cols=1000)
    r, w, f = operator_sizes("cell", **kw)
    assert (r, w) == (24_000_000, 8)
    ops = unfused_plan_sizes("cell", **kw)
    assert sum(o[0] for o in ops) == 5 * 8_000_000 and sum(o[1] for o in ops) == 2 * 8_000_000 + 8
    fused = plan_cost([(r, w, f)], 32, 32, 230.4)
    unfused = plan_cost(ops, 32, 32, 230.4)
    assert abs(unfused / fused - 7.0 / 3.0) < 1e-3          # bandwidth-bound on both sides
    # the Row chain: fusion removes the second scan of X, the model's factor of two (Section 5.2)
    kw = dict(rows=10 ** 6, cols=1000)
    fused = plan_cost([operator_sizes("row_dense", **kw)], 32, 32, 230.4)
    unfused = plan_cost(unfused_plan_sizes("row_dense", **kw), 32, 32, 230.4)
    assert 1.99 < unfused / fused < 2.01
    # the Outer operator: the unfused plan's cost does not depend on the number of stored
    # cells, the fused one's is proportional to it - orders of magnitude at low density
    kw = dict(rows=20000, cols=20000, rank=100)
    hi = plan_cost(unfused_plan_sizes("outer", nnz=40000, **kw), 32, 32, 230.4)
    lo = plan_cost([operator_sizes("outer", nnz=40000, **kw)], 32, 32, 230.4)
    assert hi / lo > 1000
