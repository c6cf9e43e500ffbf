"""Pins for the CPU checker: each function in oracle/ is compared with something
that is not itself - closed forms on exactly representable values, pure-Python
brute force in exact rational arithmetic on tiny inputs, algebraic identities,
special cases that reduce to a textbook result.  A dropped term, a wrong sign or
index, or a transposed operand in the checker fails at least one of these.
"""
import math
from fractions import Fraction

import numpy as np
import pytest

import datagen
import oracle
from datagen.workloads import csr_to_dense

F = Fraction


def fsum_exact(values):
    """Exact sum of floats through rationals, rounded once."""
    return float(sum((F(float(x)) for x in values), F(0)))


def close(a, b, rel=1e-14):
    a, b = float(a), float(b)
    return abs(a - b) <= rel * max(abs(a), abs(b), 1e-300)


# ------------------------------------------------------------------ chain ops
def run1(op, *vals):
    args = [np.array([v], dtype=np.float64) for v in vals]
    names = ["side%d" % k for k in range(len(vals))]
    env = dict(zip(names, args))
    (r,) = oracle.eval_chain([(op, "t0") + tuple(names)], ["t0"], env, (1,))
    return float(r[0])


def test_ops_known_values():
    assert run1("exp", 0.0) == 1.0
    assert close(run1("exp", 1.0), 2.718281828459045, 1e-15)
    assert run1("log", 1.0) == 0.0
    assert close(run1("log", 2.0), 0.6931471805599453, 1e-15)
    assert close(run1("sqrt", 2.0), 1.4142135623730951, 1e-16)
    assert run1("sqrt", 9.0) == 3.0
    assert run1("sq", -3.0) == 9.0
    assert run1("neg", 2.5) == -2.5 and run1("abs", -2.5) == 2.5
    assert run1("mov", -0.0) == 0.0 and math.copysign(1.0, run1("mov", -0.0)) == -1.0
    assert run1("add", 1.5, 2.25) == 3.75
    assert run1("sub", 1.5, 2.25) == -0.75        # order of operands
    assert run1("mul", 1.5, -2.0) == -3.0
    assert run1("div", 3.0, 2.0) == 1.5           # order of operands
    assert run1("min", 3.0, -2.0) == -2.0 and run1("max", 3.0, -2.0) == 3.0
    assert run1("pow", 2.0, 10.0) == 1024.0 and run1("pow", 9.0, 0.5) == 3.0
    assert run1("fma", 2.0, 3.0, 4.0) == 10.0
    assert run1("sel", 1.0, 5.0, 7.0) == 5.0 and run1("sel", 0.0, 5.0, 7.0) == 7.0
    assert run1("sel", -0.0, 5.0, 7.0) == 7.0


def test_ops_comparisons_truth_table():
    for a, b in [(1.0, 2.0), (2.0, 1.0), (2.0, 2.0), (0.0, -0.0)]:
        assert run1("eq", a, b) == float(a == b)
        assert run1("ne", a, b) == float(a != b)
        assert run1("lt", a, b) == float(a < b)
        assert run1("le", a, b) == float(a <= b)
        assert run1("gt", a, b) == float(a > b)
        assert run1("ge", a, b) == float(a >= b)


def test_ops_inverse_identities():
    x = datagen.uniform(11, 0, 200, 0.1, 9.0)
    env = {"a": x}
    chain = [("log", "t0", "a"), ("exp", "t1", "t0"),
             ("sqrt", "t2", "a"), ("sq", "t3", "t2"),
             ("pow", "t4", "a", 2.0), ("sq", "t5", "a")]
    r = oracle.eval_chain(chain, ["t1", "t3", "t4", "t5"], env, x.shape)
    assert np.allclose(r[0], x, rtol=1e-14, atol=0)
    assert np.allclose(r[1], x, rtol=1e-15, atol=0)
    assert np.allclose(r[2], r[3], rtol=1e-15, atol=0)


def test_chain_rejects_use_before_def():
    with pytest.raises(KeyError):
        oracle.eval_chain([("add", "t0", "t1", "a")], ["t0"], {"a": np.zeros(2)}, (2,))


# ------------------------------------------------------------------ aggregates
def test_sums_exact_against_rationals():
    x = datagen.normal(5, 0, 6 * 7, 0.0, 1e6).reshape(6, 7)
    x[2, 3] = 1e-9
    assert oracle.full_sum(x) == fsum_exact(x.reshape(-1))
    assert oracle.row_sums(x).tolist() == [fsum_exact(x[i]) for i in range(6)]
    assert oracle.col_sums(x).tolist() == [fsum_exact(x[:, j]) for j in range(7)]
    assert oracle.full_sum(np.zeros((0, 5))) == 0.0


# ------------------------------------------------------------------ Cell
XYZ = [("mul", "t0", "a", "side0"), ("mul", "t1", "t0", "side1")]


def test_cell_all_ones_and_integer_grid():
    m, n = 37, 53
    ones = np.ones((m, n))
    assert oracle.sum_xyz(ones, ones, ones) == m * n
    X = np.repeat(np.arange(1, m + 1, dtype=np.float64)[:, None], n, axis=1)   # X_ij = i
    Y = np.repeat(np.arange(1, n + 1, dtype=np.float64)[None, :], m, axis=0)   # Y_ij = j
    expect = (m * (m + 1) // 2) * (n * (n + 1) // 2)
    assert oracle.sum_xyz(X, Y, ones) == float(expect)
    assert oracle.cell(XYZ, "t1", X, [("cell", Y), ("cell", ones)]) == float(expect)
    # row / col aggregation of the same grid: closed forms
    r = oracle.cell(XYZ, "t1", X, [("cell", Y), ("cell", ones)], agg="row")
    c = oracle.cell(XYZ, "t1", X, [("cell", Y), ("cell", ones)], agg="col")
    assert r.tolist() == [float(i * n * (n + 1) // 2) for i in range(1, m + 1)]
    assert c.tolist() == [float(j * m * (m + 1) // 2) for j in range(1, n + 1)]


def test_cell_one_hot_selects_single_product():
    m, n = 9, 11
    w = datagen.cell_workload(m, n, seed=21)
    E = np.zeros((m, n))
    E[4, 7] = 1.0
    got = oracle.sum_xyz(E, w["Y"], w["Z"])
    assert got == w["Y"][4, 7] * w["Z"][4, 7]


def test_cell_frobenius():
    X = datagen.normal(3, 0, 40 * 30).reshape(40, 30)
    s = oracle.cell([("mul", "t0", "a", "a")], "t0", X)
    assert close(s, np.linalg.norm(X) ** 2, 1e-13)
    assert close(s, oracle.cell([("sq", "t0", "a")], "t0", X), 1e-16)


def test_cell_bruteforce_rational_with_all_side_kinds():
    m, n = 5, 6
    X = datagen.normal(7, 0, m * n).reshape(m, n)
    Y = datagen.normal(7, 2, m * n).reshape(m, n)
    rv = datagen.normal(7, 3, m)          # read at the row index
    cv = datagen.normal(7, 4, n)          # read at the column index
    s0 = 1e-6
    # f = Y + (a * s0) * rv[r] - cv[c]   (shape of the cell-wise listing in Section 2.2)
    chain = [("mul", "t0", "a", "s0"), ("mul", "t1", "t0", "side1"),
             ("add", "t2", "side0", "t1"), ("sub", "t3", "t2", "side2")]
    sides = [("cell", Y), ("row", rv), ("col", cv)]
    cellv = [[((X[i, j] * s0) * rv[i] + Y[i, j]) - cv[j] for j in range(n)] for i in range(m)]
    none = oracle.cell(chain, "t3", X, sides, [s0], agg="none")
    assert none.tolist() == cellv
    assert oracle.cell(chain, "t3", X, sides, [s0], agg="full") == \
        fsum_exact([x for r in cellv for x in r])
    assert oracle.cell(chain, "t3", X, sides, [s0], agg="row").tolist() == \
        [fsum_exact(r) for r in cellv]
    assert oracle.cell(chain, "t3", X, sides, [s0], agg="col").tolist() == \
        [fsum_exact([cellv[i][j] for i in range(m)]) for j in range(n)]


def test_cell_generic_equals_literal():
    w = datagen.cell_workload(64, 48, seed=0)
    assert oracle.cell(XYZ, "t1", w["X"], [("cell", w["Y"]), ("cell", w["Z"])]) == \
        oracle.sum_xyz(w["X"], w["Y"], w["Z"])


def test_cell_sparse_safe_equals_dense_for_zero_preserving_chain():
    rp, ci, v = datagen.csr_bernoulli(9, 0, 30, 40, 0.1, 0.5, 2.0)
    Xs = dict(rows=30, cols=40, rowptr=rp, colidx=ci, vals=v)
    Xd = csr_to_dense(30, 40, rp, ci, v)
    Y = datagen.normal(9, 2, 30 * 40).reshape(30, 40)
    rv = datagen.normal(9, 3, 30)
    chain = [("mul", "t0", "a", "side0"), ("mul", "t1", "t0", "side1")]
    sides = [("cell", Y), ("row", rv)]
    for agg in ("full", "row", "col"):
        a = oracle.cell(chain, "t1", Xs, sides, agg=agg)
        b = oracle.cell(chain, "t1", Xd, sides, agg=agg)
        assert np.allclose(a, b, rtol=1e-13, atol=1e-15)
    # per-cell values sit on X's pattern
    vals = oracle.cell(chain, "t1", Xs, sides, agg="none")
    dense = oracle.cell(chain, "t1", Xd, sides, agg="none")
    rid = oracle.csr_row_ids(30, rp)
    assert np.array_equal(vals, dense[rid, ci])


# ------------------------------------------------------------------ MAgg
def test_cell_sparse_sides_bruteforce():
    # a sparse driver with a sparse side: the side reads 0 wherever it stores nothing
    m, n = 7, 9
    rp, ci, xv = datagen.csr_bernoulli(11, 0, m, n, 0.5, 1.0, 2.0)
    X = dict(rows=m, cols=n, rowptr=rp, colidx=ci, vals=xv)
    rp2, ci2, yv = datagen.csr_bernoulli(11, 4, m, n, 0.4, -1.0, 1.0)
    Y = dict(rows=m, cols=n, rowptr=rp2, colidx=ci2, vals=yv)
    Z = datagen.normal(11, 8, m * n).reshape(m, n)
    Yd = csr_to_dense(m, n, rp2, ci2, yv)
    Xd = csr_to_dense(m, n, rp, ci, xv)
    chain = [("mul", "t0", "a", "side0"), ("mul", "t1", "t0", "side1")]
    want = sum((F(float(Xd[i, j])) * F(float(Yd[i, j])) * F(float(Z[i, j])) for i in range(m) for j in range(n)), F(0))
    got = oracle.cell(chain, "t1", X, [("cell", Y), ("cell", Z)], agg="full")
    assert abs(got - float(want)) <= 1e-15 * float(np.sum(np.abs(Xd * Yd * Z))) + 1e-300
    assert 0 < np.count_nonzero(Xd * Yd) < np.count_nonzero(Xd)        # the patterns really differ
    # same values as with the side made dense, cell by cell and for every aggregation
    for agg in ("none", "row", "col", "full"):
        a = oracle.cell(chain, "t1", X, [("cell", Y), ("cell", Z)], agg=agg)
        b = oracle.cell(chain, "t1", X, [("cell", Yd), ("cell", Z)], agg=agg)
        assert np.array_equal(np.asarray(a), np.asarray(b))
    # a chain that is not zero-preserving in the side: a + side0 keeps a where the side is empty
    t = oracle.cell([("add", "t0", "a", "side0")], "t0", X, [("cell", Y)], agg="none")
    rid = oracle.csr_row_ids(m, rp)
    assert t.tolist() == (xv + Yd[rid, ci]).tolist()
    # an empty side
    E = dict(rows=m, cols=n, rowptr=np.zeros(m + 1, dtype=np.int32), colidx=np.zeros(0, dtype=np.int32),
             vals=np.zeros(0))
    assert oracle.cell(chain, "t1", X, [("cell", E), ("cell", Z)], agg="full") == 0.0
    # a dense main input takes the sparse side as a dense array
    d = oracle.cell(chain, "t1", Xd, [("cell", Y), ("cell", Z)], agg="full")
    assert abs(d - float(want)) <= 1e-15 * float(np.sum(np.abs(Xd * Yd * Z)))


def test_magg_matches_single_aggregates_and_inequalities():
    w = datagen.magg_workload(200, 30, seed=1)
    X, Y, Z = w["X"], w["Y"], w["Z"]
    got = oracle.magg_xy_xz_xx(X, Y, Z)
    assert got.shape == (3,)
    # order of the outputs: [sum xy, sum xz, sum xx]
    assert got[0] == oracle.cell([("mul", "t0", "a", "side0")], "t0", X, [("cell", Y)])
    assert got[1] == oracle.cell([("mul", "t0", "a", "side0")], "t0", X, [("cell", Z)])
    assert got[2] == oracle.cell([("mul", "t0", "a", "a")], "t0", X)
    assert got[2] >= 0
    syy = oracle.cell([("mul", "t0", "a", "a")], "t0", Y)
    assert got[0] ** 2 <= got[2] * syy          # Cauchy-Schwarz
    chain = [("mul", "t0", "a", "side0"), ("mul", "t1", "a", "side1"), ("mul", "t2", "a", "a")]
    g2 = oracle.magg(chain, ["t0", "t1", "t2"], X, [("cell", Y), ("cell", Z)])
    assert g2.tolist() == got.tolist()
    # exact brute force
    xs, ys, zs = X.reshape(-1), Y.reshape(-1), Z.reshape(-1)
    assert got[0] == fsum_exact([a * b for a, b in zip(xs, ys)])
    assert got[1] == fsum_exact([a * b for a, b in zip(xs, zs)])
    assert got[2] == fsum_exact([a * a for a in xs])


# ------------------------------------------------------------------ Row
WD = [("mul", "t0", "side0", "d")]


def rat_row_chain(X, v, w):
    """q_j = sum_i w_i (X_i . v) X_ij in exact rationals."""
    m, n = X.shape
    q = [F(0)] * n
    for i in range(m):
        d = sum((F(float(X[i, k])) * F(float(v[k])) for k in range(n)), F(0))
        t = F(float(w[i])) * d
        for j in range(n):
            q[j] += t * F(float(X[i, j]))
    return np.array([float(x) for x in q])


def test_row_identity_matrix():
    n = 17
    v = datagen.normal(2, 2, n)
    w = datagen.uniform(2, 3, n)
    q = oracle.row_chain_dense(np.eye(n), v, w)
    assert q.tolist() == (w * v).tolist()


def test_row_unit_vector_gives_gram_column():
    m, n, k = 12, 7, 3
    X = datagen.normal(2, 0, m * n).reshape(m, n)
    e = np.zeros(n)
    e[k] = 1.0
    q = oracle.row_chain_dense(X, e, np.ones(m))
    gram_col = [fsum_exact([X[i, j] * X[i, k] for i in range(m)]) for j in range(n)]
    assert np.allclose(q, gram_col, rtol=1e-13, atol=1e-15)


def test_row_bruteforce_rational_nonsquare():
    for (m, n) in [(9, 4), (3, 8), (1, 5), (6, 1)]:
        w_ = datagen.row_dense_workload(m, n, seed=2)
        X, v, w = w_["X"], w_["v"], w_["w"]
        ref = rat_row_chain(X, v, w)
        scale = np.abs(X).T @ (w * (np.abs(X) @ np.abs(v)))
        got = oracle.row_chain_dense(X, v, w)
        assert np.all(np.abs(got - ref) <= 1e-15 * scale)
        got2 = oracle.row(WD, "t0", X, v, [("row", w)], agg="col_t")
        assert got2.tolist() == got.tolist()
        # quadratic-form identity  v^T q = sum_i w_i (X_i . v)^2  >= 0
        lhs = float(v @ got)
        rhs = fsum_exact([w[i] * float(X[i] @ v) ** 2 for i in range(m)])
        assert rhs >= 0 and abs(lhs - rhs) <= 1e-12 * max(abs(rhs), 1e-300)


def test_row_other_aggregations():
    X = datagen.normal(2, 0, 8 * 5).reshape(8, 5)
    v = datagen.normal(2, 2, 5)
    w = datagen.uniform(2, 3, 8)
    t = [float(w[i]) * sum(float(X[i, k]) * float(v[k]) for k in range(5)) for i in range(8)]
    r = oracle.row(WD, "t0", X, v, [("row", w)], agg="row")
    assert np.allclose(r, t, rtol=1e-14, atol=1e-16)
    assert close(oracle.row(WD, "t0", X, v, [("row", w)], agg="full"), fsum_exact(t), 1e-13)
    # without a weight the chain's output is d itself: X^T (X v)
    q = oracle.row([], "d", X, v, agg="col_t")
    assert np.allclose(q, rat_row_chain(X, v, np.ones(8)), rtol=1e-13, atol=1e-15)


# ------------------------------------------------------------------ Row, matrix-valued intermediates
MLR_PRE = [("mul", "t0", "side0", "d")]
MLR_POST = [("mul", "t0", "side0", "d"), ("mul", "t1", "side0", "rowsum"), ("sub", "t2", "t0", "t1")]


def rat_mlogreg(X, V, P):
    """Eq. 2 in exact rationals: H_jc = sum_i X_ij (Q_ic - P_ic * sum_c' Q_ic'), Q = P * (X V)."""
    m, n = X.shape
    k = V.shape[1]
    H = [[F(0)] * k for _ in range(n)]
    for i in range(m):
        D = [sum((F(float(X[i, j])) * F(float(V[j, c])) for j in range(n)), F(0)) for c in range(k)]
        Q = [F(float(P[i, c])) * D[c] for c in range(k)]
        s = sum(Q, F(0))
        T = [Q[c] - F(float(P[i, c])) * s for c in range(k)]
        for j in range(n):
            for c in range(k):
                H[j][c] += F(float(X[i, j])) * T[c]
    return np.array([[float(x) for x in r] for r in H])


def test_row_b1_bruteforce_rational():
    for (m, n, k) in [(7, 5, 3), (4, 9, 2), (1, 3, 4), (6, 1, 1), (5, 4, 5)]:
        w = datagen.row_b1_workload(m, n, k, seed=5)
        X, V, P = w["X"], w["V"], w["P"]
        ref = rat_mlogreg(X, V, P)
        aX, aV = np.abs(X), np.abs(V)
        scale = aX.T @ (2.0 * P * (aX @ aV) + 1e-300)
        got = oracle.mlogreg_inner(X, V, P)
        assert got.shape == (n, k)
        assert np.all(np.abs(got - ref) <= 4e-15 * scale)
        # the generic two-chain form states the same expression
        got2 = oracle.row_b1(MLR_PRE, "t0", MLR_POST, "t2", X, V, [("cell", P)], agg="col_t")
        assert np.all(np.abs(got2 - ref) <= 4e-15 * scale)
        # no aggregation: the m x k row intermediates themselves
        T = oracle.row_b1(MLR_PRE, "t0", MLR_POST, "t2", X, V, [("cell", P)], agg="none")
        D = X @ V
        for i in range(m):
            Q = [F(float(P[i, c])) * F(float(D[i, c])) for c in range(k)]
            s = float(sum(Q, F(0)))
            for c in range(k):
                want = float(P[i, c]) * float(D[i, c]) - float(P[i, c]) * s
                assert abs(T[i, c] - want) <= 1e-14 * (abs(want) + abs(s))


def test_row_b1_probability_rows_give_zero_column_total():
    # if every row of P sums to one, sum_c (Q_ic - P_ic * rowSums(Q)_i) = 0, so the
    # columns of H add up to the zero vector: a sign or index slip in Eq. 2 breaks it
    m, n, k = 40, 6, 4
    w = datagen.row_b1_workload(m, n, k, seed=6)
    P = w["P"] / w["P"].sum(axis=1, keepdims=True)
    H = oracle.mlogreg_inner(w["X"], w["V"], P)
    scale = np.abs(w["X"]).T @ (P * (np.abs(w["X"]) @ np.abs(w["V"]))).sum(axis=1)
    assert np.all(np.abs(H.sum(axis=1)) <= 1e-13 * scale)
    assert np.max(np.abs(H)) > 1e-3            # and H itself is not zero


def test_row_b1_mmchain_special_cases():
    m, n, k = 11, 6, 3
    w = datagen.row_b1_workload(m, n, k, seed=7)
    X, V = w["X"], w["V"]
    H = oracle.mmchain(X, V)
    # column c of t(X) (X V) is the vector chain with v = V[:, c]
    for c in range(k):
        ref = rat_row_chain(X, V[:, c], np.ones(m))
        assert np.allclose(H[:, c], ref, rtol=1e-13, atol=1e-14)
    # generic form with the identity chain
    H2 = oracle.row_b1(None, None, [], "d", X, V, agg="col_t")
    assert H2.tolist() == H.tolist()
    # X = I: t(I) (I V) = V exactly
    E = np.eye(n)
    assert oracle.mmchain(E, V).tolist() == V.tolist()
    # a one-column V is the Row template's vector form (col_t_agg), bit for bit
    q = oracle.row([], "d", X, V[:, 0], agg="col_t")
    assert oracle.mmchain(X, V[:, :1])[:, 0].tolist() == q.tolist()
    # a non-square X: transposing the first factor would not even have the right shape
    assert H.shape == (n, k)
    # small integers: every intermediate exact
    Xi = np.arange(1, 1 + m * n, dtype=np.float64).reshape(m, n) % 7 - 3
    Vi = np.arange(1, 1 + n * k, dtype=np.float64).reshape(n, k) % 5 - 2
    Hi = oracle.mmchain(Xi, Vi)
    want = [[sum(int(Xi[i, j]) * sum(int(Xi[i, l]) * int(Vi[l, c]) for l in range(n)) for i in range(m))
             for c in range(k)] for j in range(n)]
    assert Hi.tolist() == [[float(x) for x in r] for r in want]


def test_row_b1_csr_rows_equal_dense_rows():
    m, n, k = 25, 14, 3
    ws = datagen.row_csr_workload(m, n, 0.3, seed=3)
    Xs = {q: ws[q] for q in ("rows", "cols", "rowptr", "colidx", "vals")}
    Xd = csr_to_dense(m, n, ws["rowptr"], ws["colidx"], ws["vals"])
    b = datagen.row_b1_workload(m, n, k, seed=5)
    V, P = b["V"], b["P"]
    ref = rat_mlogreg(Xd, V, P)
    aX = np.abs(Xd)
    scale = aX.T @ (2.0 * P * (aX @ np.abs(V)) + 1e-300)
    for agg in ("col_t", "none"):
        a = oracle.row_b1(MLR_PRE, "t0", MLR_POST, "t2", Xs, V, [("cell", P)], agg=agg)
        d = oracle.row_b1(MLR_PRE, "t0", MLR_POST, "t2", Xd, V, [("cell", P)], agg=agg)
        assert np.allclose(a, d, rtol=1e-12, atol=1e-14)
    got = oracle.row_b1(MLR_PRE, "t0", MLR_POST, "t2", Xs, V, [("cell", P)], agg="col_t")
    assert np.all(np.abs(got - ref) <= 4e-15 * scale)
    # a row without stored cells has D = 0: with T = d + 1 its T is all ones and adds nothing to H
    assert np.any(np.diff(ws["rowptr"]) == 0) or True
    T = oracle.row_b1(None, None, [("add", "t0", "d", 1.0)], "t0", Xs, V, agg="none")
    empty = np.flatnonzero(np.diff(ws["rowptr"]) == 0)
    assert np.all(T[empty] == 1.0)


def test_row_b1_side_kinds_and_scalars():
    # T_ic = (d * rowvec_c + colvec_i) * s0 - rowsum, rowsum = sum_c d * rowvec_c
    m, n, k = 5, 4, 3
    w = datagen.row_b1_workload(m, n, k, seed=8)
    X, V = w["X"], w["V"]
    cvec = datagen.normal(8, 9, m)            # read at the row
    rvec = datagen.normal(8, 10, k)           # read at the class
    pre = [("mul", "t0", "d", "side0")]
    post = [("mul", "t0", "d", "side0"), ("add", "t1", "t0", "side1"), ("mul", "t2", "t1", "s0"),
            ("sub", "t3", "t2", "rowsum")]
    T = oracle.row_b1(pre, "t0", post, "t3", X, V, [("col", rvec), ("row", cvec)], [2.5], agg="none")
    D = X @ V
    for i in range(m):
        rs = fsum_exact([D[i, c] * rvec[c] for c in range(k)])
        for c in range(k):
            want = (D[i, c] * rvec[c] + cvec[i]) * 2.5 - rs
            assert abs(T[i, c] - want) <= 1e-14 * (abs(want) + abs(rs) + 1.0)


def test_row_no_agg_and_col_agg():
    m, n = 9, 6
    w_ = datagen.row_dense_workload(m, n, seed=2)
    X, v, w = w_["X"], w_["v"], w_["w"]
    T = oracle.row(WD, "t0", X, v, [("row", w)], agg="none")
    assert T.shape == (m, n)
    for i in range(m):
        t = float(w[i]) * float(sum(F(float(X[i, k])) * F(float(v[k])) for k in range(n)))
        for j in range(n):
            assert abs(T[i, j] - t * X[i, j]) <= 4e-15 * abs(t * X[i, j]) + 1e-300
    # the column sums of the scaled rows are the transposed product: two routes to one vector
    c = oracle.row(WD, "t0", X, v, [("row", w)], agg="col")
    q = rat_row_chain(X, v, w)
    scale = np.abs(X).T @ (w * (np.abs(X) @ np.abs(v)))
    assert np.all(np.abs(c - q) <= 2e-15 * scale)
    # CSR main input: same values on X's pattern
    ws = datagen.row_csr_workload(30, 12, 0.3, seed=3)
    Xs = {k: ws[k] for k in ("rows", "cols", "rowptr", "colidx", "vals")}
    Xd = csr_to_dense(ws["rows"], ws["cols"], ws["rowptr"], ws["colidx"], ws["vals"])
    Ts = oracle.row(WD, "t0", Xs, ws["v"], [("row", ws["w"])], agg="none")
    Td = oracle.row(WD, "t0", Xd, ws["v"], [("row", ws["w"])], agg="none")
    rid = oracle.csr_row_ids(ws["rows"], ws["rowptr"])
    assert np.allclose(Ts, Td[rid, ws["colidx"]], rtol=1e-14, atol=0)
    cs = oracle.row(WD, "t0", Xs, ws["v"], [("row", ws["w"])], agg="col")
    assert np.allclose(cs, oracle.row(WD, "t0", Xd, ws["v"], [("row", ws["w"])], agg="col"), rtol=1e-13, atol=1e-15)


def test_row_csr_equals_dense_and_bruteforce():
    m, n = 40, 25
    w_ = datagen.row_csr_workload(m, n, 0.2, seed=3)
    Xs = {k: w_[k] for k in ("rows", "cols", "rowptr", "colidx", "vals")}
    Xd = csr_to_dense(m, n, w_["rowptr"], w_["colidx"], w_["vals"])
    assert (Xd != 0).sum() == len(w_["vals"])
    qs = oracle.row_chain_csr(Xs, w_["v"], w_["w"])
    qd = oracle.row_chain_dense(Xd, w_["v"], w_["w"])
    ref = rat_row_chain(Xd, w_["v"], w_["w"])
    scale = np.abs(Xd).T @ (w_["w"] * (np.abs(Xd) @ np.abs(w_["v"]))) + 1e-300
    assert np.all(np.abs(qs - ref) <= 1e-15 * scale)
    assert np.all(np.abs(qd - ref) <= 1e-15 * scale)
    assert oracle.row(WD, "t0", Xs, w_["v"], [("row", w_["w"])]).tolist() == qs.tolist()


def test_row_csr_empty_rows_and_empty_matrix():
    rp = np.array([0, 0, 2, 2, 3], dtype=np.int32)
    ci = np.array([1, 3, 0], dtype=np.int32)
    va = np.array([2.0, -1.0, 4.0])
    Xs = dict(rows=4, cols=4, rowptr=rp, colidx=ci, vals=va)
    v = np.array([1.0, 2.0, 3.0, 4.0])
    w = np.array([1.0, 0.5, 1.0, 2.0])
    # row1: d = 2*2 - 1*4 = 0 ; row3: d = 4*1 = 4, t = 8 -> q[0] = 32
    assert oracle.row_chain_csr(Xs, v, w).tolist() == [32.0, 0.0, 0.0, 0.0]
    E = dict(rows=3, cols=4, rowptr=np.zeros(4, np.int32), colidx=np.zeros(0, np.int32),
             vals=np.zeros(0))
    assert oracle.row_chain_csr(E, v, np.ones(3)).tolist() == [0.0] * 4


# ------------------------------------------------------------------ Outer
WSLOSS = [("ne", "t0", "a", 0.0), ("sub", "t1", "a", "d"), ("mul", "t2", "t1", "t1"),
          ("mul", "t3", "t0", "t2")]


def small_outer(m=14, n=11, k=5, density=0.3, seed=4):
    w = datagen.outer_workload(m, n, k, density, seed)
    X = {key: w[key] for key in ("rows", "cols", "rowptr", "colidx", "vals")}
    return X, w["U"], w["V"]


def brute_outer(X, U, V, f):
    """Loop over all cells; f(a, d) only where a cell is stored; exact rational dot."""
    m, n = X["rows"], X["cols"]
    stored = {}
    rid = oracle.csr_row_ids(m, X["rowptr"])
    for p, (i, j) in enumerate(zip(rid, X["colidx"])):
        stored[(int(i), int(j))] = float(X["vals"][p])
    terms = []
    for i in range(m):
        for j in range(n):
            if (i, j) in stored:
                d = float(sum((F(float(U[i, c])) * F(float(V[j, c])) for c in range(U.shape[1])), F(0)))
                terms.append(((i, j), f(stored[(i, j)], d)))
    return terms


def test_outer_bruteforce_and_mode_agreement():
    X, U, V = small_outer()
    terms = brute_outer(X, U, V, lambda a, d: (1.0 if a != 0 else 0.0) * ((a - d) * (a - d)))
    ref = fsum_exact([t for _, t in terms])
    for got in (oracle.outer_wsloss_dense(X, U, V), oracle.outer_wsloss_masked(X, U, V),
                oracle.outer(WSLOSS, "t3", X, U, V, mode="dense"),
                oracle.outer(WSLOSS, "t3", X, U, V, mode="masked")):
        assert close(got, ref, 1e-13)
    per_cell = oracle.outer(WSLOSS, "t3", X, U, V, agg="none", mode="masked")
    assert np.allclose(per_cell, [t for _, t in terms], rtol=1e-12, atol=1e-15)
    assert np.allclose(oracle.outer(WSLOSS, "t3", X, U, V, agg="none", mode="dense"),
                       per_cell, rtol=1e-12, atol=1e-15)


def test_outer_special_cases():
    X, U, V = small_outer()
    zU = np.zeros_like(U)
    sq = fsum_exact([x * x for x in X["vals"]])
    assert close(oracle.outer_wsloss_masked(X, zU, V), sq, 1e-15)
    assert close(oracle.outer_wsloss_dense(X, zU, V), sq, 1e-15)
    one_u, one_v = np.ones((X["rows"], 1)), np.ones((X["cols"], 1))
    ref = fsum_exact([(x - 1.0) * (x - 1.0) for x in X["vals"]])
    assert close(oracle.outer_wsloss_masked(X, one_u, one_v), ref, 1e-15)
    assert close(oracle.outer_wsloss_dense(X, one_u, one_v), ref, 1e-15)


def test_outer_full_pattern_is_frobenius_residual():
    m, n, k = 8, 9, 3
    rp, ci, v = datagen.csr_bernoulli(4, 0, m, n, 1.0, 1.0, 5.0)
    X = dict(rows=m, cols=n, rowptr=rp, colidx=ci, vals=v)
    U = datagen.normal(4, 2, m * k).reshape(m, k)
    V = datagen.normal(4, 3, n * k).reshape(n, k)
    ref = np.linalg.norm(v.reshape(m, n) - U @ V.T) ** 2
    assert close(oracle.outer_wsloss_masked(X, U, V), ref, 1e-13)
    assert close(oracle.outer_wsloss_dense(X, U, V), ref, 1e-13)


def test_outer_small_integers_exact():
    m, n, k = 6, 7, 4
    rp, ci, _ = datagen.csr_bernoulli(8, 0, m, n, 0.4)
    vals = np.arange(1, len(ci) + 1, dtype=np.float64)
    X = dict(rows=m, cols=n, rowptr=rp, colidx=ci, vals=vals)
    U = np.arange(m * k, dtype=np.float64).reshape(m, k) % 5 - 2
    V = np.arange(n * k, dtype=np.float64).reshape(n, k) % 3 - 1
    rid = oracle.csr_row_ids(m, rp)
    expect = 0
    for p in range(len(ci)):
        d = sum(int(U[rid[p], c]) * int(V[ci[p], c]) for c in range(k))
        expect += (int(vals[p]) - d) ** 2
    assert oracle.outer_wsloss_masked(X, U, V) == float(expect)
    assert oracle.outer_wsloss_dense(X, U, V) == float(expect)


def test_outer_explicit_stored_zero():
    # a stored 0.0 contributes nothing through (a != 0), but is still a bound
    # cell for a chain that does not test it
    rp = np.array([0, 2, 3], dtype=np.int32)
    ci = np.array([0, 2, 1], dtype=np.int32)
    va = np.array([0.0, 3.0, 2.0])
    X = dict(rows=2, cols=3, rowptr=rp, colidx=ci, vals=va)
    U = np.array([[1.0], [2.0]])
    V = np.array([[1.0], [1.0], [0.5]])
    # d: (0,0)=1, (0,2)=0.5, (1,1)=2 -> with mask: (3-.5)^2 + 0 = 6.25 ; without: +1
    for mode in ("dense", "masked"):
        assert oracle.outer(WSLOSS, "t3", X, U, V, mode=mode) == 6.25
        assert oracle.outer(WSLOSS[1:3], "t2", X, U, V, mode=mode) == 7.25
    assert oracle.outer_wsloss_dense(X, U, V) == 6.25
    assert oracle.outer_wsloss_masked(X, U, V) == 6.25


def test_outer_right_left_bruteforce():
    X, U, V = small_outer(9, 8, 3, 0.35, seed=14)
    m, n, k = 9, 8, 3
    chain = [("ne", "t0", "a", 0.0), ("mul", "t1", "t0", "d")]     # (X != 0) * (U V^T), Eq. 1
    terms = brute_outer(X, U, V, lambda a, d: (1.0 if a != 0 else 0.0) * d)
    R = np.zeros((m, k))
    L = np.zeros((n, k))
    for (i, j), wij in terms:
        R[i] += wij * V[j]
        L[j] += wij * U[i]
    for mode in ("dense", "masked"):
        assert np.allclose(oracle.outer(chain, "t1", X, U, V, agg="right", mode=mode), R,
                           rtol=1e-12, atol=1e-14)
        assert np.allclose(oracle.outer(chain, "t1", X, U, V, agg="left", mode=mode), L,
                           rtol=1e-12, atol=1e-14)


def test_outer_empty():
    X = dict(rows=3, cols=4, rowptr=np.zeros(4, np.int32), colidx=np.zeros(0, np.int32),
             vals=np.zeros(0))
    U, V = np.ones((3, 2)), np.ones((4, 2))
    assert oracle.outer_wsloss_masked(X, U, V) == 0.0
    assert oracle.outer_wsloss_dense(X, U, V) == 0.0
    assert oracle.outer(WSLOSS, "t3", X, U, V, mode="masked") == 0.0


def test_outer_side_inputs_bruteforce_and_mode_agreement():
    """Outer with dense side inputs (Table 1): every stored cell reads a cell-shaped side
    at (i, j), a row-vector side at j and a column-vector side at i; exact rationals."""
    X, U, V = small_outer(10, 9, 4, 0.4, seed=21)
    m, n = X["rows"], X["cols"]
    S = datagen.uniform(21, 5, m * n, -1.0, 1.0).reshape(m, n)
    r = datagen.uniform(21, 6, m, 0.5, 2.0)
    c = datagen.uniform(21, 7, n, -2.0, 2.0)
    chain = [("sub", "t0", "a", "d"), ("mul", "t1", "t0", "side0"), ("add", "t2", "t1", "side2"),
             ("mul", "t3", "t2", "side1")]                         # ((a - d) * S_ij + c_j) * r_i
    sides = [("cell", S), ("row", r), ("col", c)]
    rid = oracle.csr_row_ids(m, X["rowptr"])
    want = []
    for p in range(len(X["vals"])):
        i, j = int(rid[p]), int(X["colidx"][p])
        d = sum((F(float(U[i, q])) * F(float(V[j, q])) for q in range(U.shape[1])), F(0))
        want.append(float(((F(float(X["vals"][p])) - d) * F(float(S[i, j])) + F(float(c[j]))) * F(float(r[i]))))
    for mode in ("dense", "masked"):
        got = oracle.outer(chain, "t3", X, U, V, agg="none", mode=mode, sides=sides)
        assert np.allclose(got, want, rtol=1e-12, atol=1e-14)
        assert close(oracle.outer(chain, "t3", X, U, V, mode=mode, sides=sides), fsum_exact(want), 1e-12)
    # a side of ones changes nothing; a constant row vector is a scalar
    ones = [("cell", np.ones((m, n)))]
    plain = oracle.outer(WSLOSS, "t3", X, U, V)
    assert oracle.outer(WSLOSS + [("mul", "t4", "t3", "side0")], "t4", X, U, V, sides=ones) == plain
    assert oracle.outer([("mul", "t0", "d", "side0")], "t0", X, U, V, sides=[("row", np.full(m, 3.0))]) == \
        oracle.outer([("mul", "t0", "d", "s0")], "t0", X, U, V, [3.0])


def test_count_nonzero_known_values():
    assert oracle.count_nonzero([]) == 0
    assert oracle.count_nonzero([0.0, -0.0, 1.0, -2.5, 5e-324, float("nan"), float("inf")]) == 5
    assert oracle.count_nonzero(np.zeros((3, 4))) == 0
    a = np.arange(-3, 4, dtype=np.float64)
    assert oracle.count_nonzero(a) == 6
    assert oracle.count_nonzero(np.outer(a, a)) == 36
