"""Unfused, operator-at-a-time evaluation of the four template types on the CPU.

TEST INFRASTRUCTURE (see the package docstring).  Every step allocates its
result as a full numpy float64 array; nothing is blocked, fused or reordered.

Paper passages followed:
  Cell  - Table 1 (binding X_ij, side inputs, scalars; no/row/col/full agg) and
          the cell-wise operator listing of Section 2.2: one scalar chain per
          cell with side values read at (rix, cix) or at (rix).
  MAgg  - Table 1 and "Multi-Aggregate Operations" in Section 5.2: several
          full aggregates over shared inputs, returned as a k x 1 column.
  Row   - Fig. 1(b) / "Row Operations" in Section 5.2: X^T (w * (X v)) is the
          unfused sequence  t1 = X v ; t2 = w * t1 ; q = X^T t2.  With a side
          matrix instead of v (Table 1, the *_B1 variants; Eq. 2 and its row-wise
          listing in Section 2.2) the row intermediate is a k-vector:
          D = X V ; T = chains(D, sides, rowSums) ; H = X^T T.
  Outer - Fig. 1(d), Eq. 1 and the outer-product listing of Section 2.2: for
          every stored X_ij the scalar chain sees a = X_ij and d = U_i . V_j;
          unfused, d is the dense product U V^T masked by X's pattern.
"""
from __future__ import annotations

import numpy as np

LD = np.longdouble


# --------------------------------------------------------------------------
# basic scalar operators, each applied to whole arrays
# --------------------------------------------------------------------------
def _b(x):
    return x.astype(np.float64)


OPS = {
    # name: (arity, function)
    "mov": (1, lambda a: np.array(a, dtype=np.float64)),
    "neg": (1, lambda a: -a),
    "abs": (1, lambda a: np.abs(a)),
    "sqrt": (1, lambda a: np.sqrt(a)),
    "exp": (1, lambda a: np.exp(a)),
    "log": (1, lambda a: np.log(a)),
    "sq": (1, lambda a: a * a),
    "add": (2, lambda a, b: a + b),
    "sub": (2, lambda a, b: a - b),
    "mul": (2, lambda a, b: a * b),
    "div": (2, lambda a, b: a / b),
    "min": (2, lambda a, b: np.minimum(a, b)),
    "max": (2, lambda a, b: np.maximum(a, b)),
    "pow": (2, lambda a, b: np.power(a, b)),
    "eq": (2, lambda a, b: _b(np.equal(a, b))),
    "ne": (2, lambda a, b: _b(np.not_equal(a, b))),
    "lt": (2, lambda a, b: _b(np.less(a, b))),
    "le": (2, lambda a, b: _b(np.less_equal(a, b))),
    "gt": (2, lambda a, b: _b(np.greater(a, b))),
    "ge": (2, lambda a, b: _b(np.greater_equal(a, b))),
    "sel": (3, lambda a, b, c: np.where(np.not_equal(a, 0.0), b, c)),
    "fma": (3, lambda a, b, c: (a * b) + c),
}


def eval_chain(chain, outputs, env, shape):
    """Run the steps of `chain` one after another over arrays of `shape`.

    `env` maps operand names ("a", "d", "side0", "s0", ...) to arrays that
    broadcast to `shape` (or Python floats).  Each step's result is materialised
    as a full array of `shape` and bound to its ``dst`` name.  Returns the list
    of arrays named by `outputs`.
    """
    env = dict(env)

    def fetch(x):
        if isinstance(x, (int, float)):
            return np.float64(x)
        if x not in env:
            raise KeyError("chain reads %r before it is defined" % (x,))
        return env[x]

    for step in chain:
        name, dst, srcs = step[0], step[1], step[2:]
        arity, fn = OPS[name]
        if len(srcs) != arity:
            raise ValueError("%s takes %d operands" % (name, arity))
        with np.errstate(all="ignore"):
            res = fn(*[fetch(s) for s in srcs])
        env[dst] = np.array(np.broadcast_to(np.asarray(res, dtype=np.float64), shape))
    return [np.array(np.broadcast_to(np.asarray(fetch(o), dtype=np.float64), shape))
            for o in outputs]


# --------------------------------------------------------------------------
# aggregation operators
# --------------------------------------------------------------------------
def full_sum(t):
    """sum(T): every element, accumulated in extended precision."""
    t = np.asarray(t, dtype=np.float64)
    if t.size == 0:
        return 0.0
    return float(np.sum(t.reshape(-1), dtype=LD))


def row_sums(t):
    """rowSums(T): m-vector."""
    t = np.asarray(t, dtype=np.float64)
    return np.sum(t, axis=1, dtype=LD).astype(np.float64)


def col_sums(t):
    """colSums(T): n-vector."""
    t = np.asarray(t, dtype=np.float64)
    return np.sum(t, axis=0, dtype=LD).astype(np.float64)


def count_nonzero(values):
    """Number of entries of an elementwise result that are not zero (the nnz a sparse
    output would store; -0.0 counts as zero, NaN as non-zero): the comparison
    `values != 0`, then a count."""
    return int(np.count_nonzero(np.asarray(values, dtype=np.float64) != 0.0))


def csr_row_ids(rows, rowptr):
    """Row index of every stored cell of a CSR matrix."""
    return np.repeat(np.arange(rows, dtype=np.int64), np.diff(np.asarray(rowptr, dtype=np.int64)))


def _segment_sum(values, ids, nseg):
    """out[k] = sum of values whose id is k (np.bincount with weights)."""
    if values.size == 0:
        return np.zeros(nseg, dtype=np.float64)
    return np.bincount(ids, weights=values, minlength=nseg).astype(np.float64)


def _is_csr(x):
    return isinstance(x, dict)


# --------------------------------------------------------------------------
# Cell and MAgg templates
# --------------------------------------------------------------------------
def _cell_env_dense(X, sides, scalars):
    m, n = X.shape
    env = {"a": X}
    for k, (access, arr) in enumerate(sides):
        if _is_csr(arr):               # sparse side over a dense main input: as a dense array
            d = np.zeros((arr["rows"], arr["cols"]), dtype=np.float64)
            d[csr_row_ids(arr["rows"], arr["rowptr"]), np.asarray(arr["colidx"], dtype=np.int64)] = arr["vals"]
            arr = d
        arr = np.asarray(arr, dtype=np.float64)
        if access == "cell":
            assert arr.shape == (m, n)
            env["side%d" % k] = arr
        elif access == "row":          # column vector, read at (rix)
            assert arr.shape == (m,)
            env["side%d" % k] = arr.reshape(m, 1)
        elif access == "col":          # row vector, read at (cix)
            assert arr.shape == (n,)
            env["side%d" % k] = arr.reshape(1, n)
        else:
            raise ValueError(access)
    for k, s in enumerate(scalars):
        env["s%d" % k] = np.float64(s)
    return env


def _csr_lookup(Y, rid, cid):
    """Values of the CSR matrix Y at the cells (rid[p], cid[p]); 0.0 where Y stores
    nothing.  Cells are matched by their row-major position row * cols + col, which
    ascends through a CSR matrix (np.searchsorted on those keys)."""
    n = Y["cols"]
    ykeys = csr_row_ids(Y["rows"], Y["rowptr"]) * n + np.asarray(Y["colidx"], dtype=np.int64)
    keys = np.asarray(rid, dtype=np.int64) * n + np.asarray(cid, dtype=np.int64)
    yv = np.asarray(Y["vals"], dtype=np.float64)
    if ykeys.size == 0:
        return np.zeros(keys.shape, dtype=np.float64)
    pos = np.minimum(np.searchsorted(ykeys, keys), ykeys.size - 1)
    return np.where(ykeys[pos] == keys, yv[pos], 0.0)


def _cell_env_csr(X, sides, scalars):
    """Sparse-safe binding: one value per stored cell of the main input."""
    m, n = X["rows"], X["cols"]
    rid = csr_row_ids(m, X["rowptr"])
    cid = np.asarray(X["colidx"], dtype=np.int64)
    env = {"a": np.asarray(X["vals"], dtype=np.float64)}
    for k, (access, arr) in enumerate(sides):
        if _is_csr(arr):               # sparse side: its value at X's stored cells, 0 where it has none
            if access != "cell":
                raise ValueError("a CSR side is read at (row, column)")
            env["side%d" % k] = _csr_lookup(arr, rid, cid)
            continue
        arr = np.asarray(arr, dtype=np.float64)
        if access == "cell":
            env["side%d" % k] = arr[rid, cid]
        elif access == "row":
            env["side%d" % k] = arr[rid]
        elif access == "col":
            env["side%d" % k] = arr[cid]
        else:
            raise ValueError(access)
    for k, s in enumerate(scalars):
        env["s%d" % k] = np.float64(s)
    return env, rid, cid


def cell(chain, output, X, sides=(), scalars=(), agg="full"):
    """Cell template (Table 1): apply the scalar chain to every cell of a dense
    main input X (or, for a CSR main input, to every stored cell: the
    sparse-safe binding), then aggregate: "none" | "row" | "col" | "full".
    """
    if _is_csr(X):
        m, n = X["rows"], X["cols"]
        env, rid, cid = _cell_env_csr(X, sides, scalars)
        (t,) = eval_chain(chain, [output], env, env["a"].shape)
        if agg == "full":
            return full_sum(t)
        if agg == "row":
            return _segment_sum(t, rid, m)
        if agg == "col":
            return _segment_sum(t, cid, n)
        if agg == "none":      # same pattern as X, new values
            return t
        raise ValueError(agg)
    X = np.asarray(X, dtype=np.float64)
    env = _cell_env_dense(X, sides, scalars)
    (t,) = eval_chain(chain, [output], env, X.shape)
    if agg == "full":
        return full_sum(t)
    if agg == "row":
        return row_sums(t)
    if agg == "col":
        return col_sums(t)
    if agg == "none":
        return t
    raise ValueError(agg)


def magg(chain, outputs, X, sides=(), scalars=()):
    """MAgg template: k full aggregates over shared inputs, as a k-vector in the
    order the outputs are listed.  Unfused, each aggregate is evaluated on its
    own: its own run of the chain, its own intermediates, its own scan."""
    res = [cell(chain, o, X, sides, scalars, "full") for o in outputs]
    return np.array(res, dtype=np.float64)


# --------------------------------------------------------------------------
# Row template
# --------------------------------------------------------------------------
def _matvec(X, v):
    """t = X v  (dense: library matrix product; CSR: gather, multiply, segment-sum)."""
    if _is_csr(X):
        g = v[np.asarray(X["colidx"], dtype=np.int64)]
        p = X["vals"] * g
        return _segment_sum(p, csr_row_ids(X["rows"], X["rowptr"]), X["rows"])
    return X @ v


def _tmatvec(X, t):
    """q = X^T t."""
    if _is_csr(X):
        g = t[csr_row_ids(X["rows"], X["rowptr"])]
        p = X["vals"] * g
        return _segment_sum(p, np.asarray(X["colidx"], dtype=np.int64), X["cols"])
    return X.T @ t


def row(chain, output, X, v, sides=(), scalars=(), agg="col_t"):
    """Row template over the rows of X (dense ndarray or CSR dict).

    t1 = X v                     first scan of X
    t  = chain(d = t1, sides read at the row index, scalars)   m-vectors
    agg "col_t": q = X^T t       second scan of X, n-vector
        "row"  : t itself        m-vector
        "full" : sum(t)
        "none" : T = t * X       every row of X scaled by its t (dense: m x n; CSR:
                                 the nnz new values on X's pattern)
        "col"  : colSums(T)      the column sums of that materialised T, n-vector
    """
    m = X["rows"] if _is_csr(X) else X.shape[0]
    v = np.asarray(v, dtype=np.float64)
    t1 = _matvec(X, v)
    env = {"d": t1}
    for k, (access, arr) in enumerate(sides):
        if access != "row":
            raise ValueError("Row-template sides are read at the row index")
        arr = np.asarray(arr, dtype=np.float64)
        assert arr.shape == (m,)
        env["side%d" % k] = arr
    for k, s in enumerate(scalars):
        env["s%d" % k] = np.float64(s)
    (t,) = eval_chain(chain, [output], env, (m,))
    if agg == "col_t":
        return _tmatvec(X, t)
    if agg == "row":
        return t
    if agg == "full":
        return full_sum(t)
    if agg in ("none", "col"):
        if _is_csr(X):
            T = t[csr_row_ids(X["rows"], X["rowptr"])] * np.asarray(X["vals"], dtype=np.float64)
            if agg == "none":
                return T
            return _segment_sum(T, np.asarray(X["colidx"], dtype=np.int64), X["cols"])
        T = t.reshape(m, 1) * np.asarray(X, dtype=np.float64)
        return T if agg == "none" else col_sums(T)
    raise ValueError(agg)


def row_b1(pre, pre_out, post, post_out, X, B, sides=(), scalars=(), agg="col_t"):
    """Row template with a matrix-valued row intermediate (Table 1: the *_B1
    variants; the row-wise listing of Section 2.2 for Eq. 2; "Row Operations" in
    Section 5.2 for t(X) %*% (X %*% V)).  X is m x n, dense or CSR (the listing's
    genexecSparse binding: the same operators over the stored cells); B dense n x k.

    D  = X B                     first scan of X: m x k (the listing's vectMatMult)
    P  = pre(d = D, sides)       m x k, and  s = rowSums(P)  (vectSum); skipped
                                 when `pre` is None
    T  = post(d = D, sides, rowsum = s broadcast over the k columns)   m x k
    agg "col_t": H = X^T T       second scan of X: n x k (vectOuterMultAdd)
        "none" : T itself        m x k
    Sides: ("cell", m x k) read at (row, class), ("row", m) read at the row,
    ("col", k) read at the class.
    """
    B = np.asarray(B, dtype=np.float64)
    k = B.shape[1]
    if _is_csr(X):                 # CSR rows: one sparse matrix-vector product per class
        m, n = X["rows"], X["cols"]
        assert B.shape[0] == n
        D = np.stack([_matvec(X, np.ascontiguousarray(B[:, c])) for c in range(k)], axis=1)
    else:
        X = np.asarray(X, dtype=np.float64)
        m, n = X.shape
        assert B.shape[0] == n
        D = X @ B
    env = {"d": D}
    for j, (access, arr) in enumerate(sides):
        arr = np.asarray(arr, dtype=np.float64)
        if access == "cell":
            assert arr.shape == (m, k)
            env["side%d" % j] = arr
        elif access == "row":
            assert arr.shape == (m,)
            env["side%d" % j] = arr.reshape(m, 1)
        elif access == "col":
            assert arr.shape == (k,)
            env["side%d" % j] = arr.reshape(1, k)
        else:
            raise ValueError(access)
    for j, s in enumerate(scalars):
        env["s%d" % j] = np.float64(s)
    if pre is not None:
        (P,) = eval_chain(pre, [pre_out], env, (m, k))
        env["rowsum"] = row_sums(P).reshape(m, 1)
    (T,) = eval_chain(post, [post_out], env, (m, k))
    if agg == "col_t":
        if _is_csr(X):
            return np.stack([_tmatvec(X, np.ascontiguousarray(T[:, c])) for c in range(k)], axis=1)
        return X.T @ T
    if agg == "none":
        return T
    raise ValueError(agg)


def mmchain(X, V):
    """t(X) %*% (X %*% V) with its m x k intermediate (Section 5.2, "Row
    Operations": the matrix-matrix multiplication chain)."""
    T1 = X @ V
    return X.T @ T1


def mlogreg_inner(X, V, P):
    """Eq. 2, written out one basic operator at a time (P stands for P[,1:k],
    m x k; V is n x k):
        Q = P * (X V);   H = X^T (Q - P * rowSums(Q))
    """
    T1 = X @ V
    Q = P * T1
    s = row_sums(Q).reshape(-1, 1)
    T2 = P * s
    T3 = Q - T2
    return X.T @ T3


# --------------------------------------------------------------------------
# Outer template
# --------------------------------------------------------------------------
def outer(chain, output, X, U, V, scalars=(), agg="full", mode="masked", sides=()):
    """Outer template over the stored cells of the CSR matrix X.

    Side inputs (Table 1 binds dense side inputs to the Outer template too):
    ("cell", m x n array) read at (i, j), ("row", m-vector) read at i, ("col",
    n-vector) read at j; the chain names them "side0", "side1", ...

    mode "dense":  P = U V^T as a dense m x n array; the chain runs on every
                   cell (a = dense X, d = P); the result is kept only where X
                   has a stored cell.
    mode "masked": d[p] = U_i . V_j for every stored cell p = (i, j), as an
                   nnz-vector; the chain runs on nnz-vectors.
    agg "full":  sum of the chain's value over stored cells
        "none":  the chain's value per stored cell (nnz-vector, X's pattern)
        "right": O = W V   with W the chain's values on X's pattern (m x k)
        "left" : O = W^T U                                         (n x k)
    """
    m, n = X["rows"], X["cols"]
    U = np.asarray(U, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    rid = csr_row_ids(m, X["rowptr"])
    cid = np.asarray(X["colidx"], dtype=np.int64)
    senv = {"s%d" % k: np.float64(s) for k, s in enumerate(scalars)}
    dense_sides, cell_sides = {}, {}
    for k, (access, arr) in enumerate(sides):
        arr = np.asarray(arr, dtype=np.float64)
        if access == "cell":
            assert arr.shape == (m, n)
            dense_sides["side%d" % k], cell_sides["side%d" % k] = arr, arr[rid, cid]
        elif access == "row":
            assert arr.shape == (m,)
            dense_sides["side%d" % k], cell_sides["side%d" % k] = arr.reshape(m, 1), arr[rid]
        elif access == "col":
            assert arr.shape == (n,)
            dense_sides["side%d" % k], cell_sides["side%d" % k] = arr.reshape(1, n), arr[cid]
        else:
            raise ValueError(access)
    if mode == "dense":
        Xd = np.zeros((m, n), dtype=np.float64)
        Xd[rid, cid] = X["vals"]
        pattern = np.zeros((m, n), dtype=np.float64)
        pattern[rid, cid] = 1.0
        P = U @ V.T
        (T,) = eval_chain(chain, [output], dict(senv, a=Xd, d=P, **dense_sides), (m, n))
        Wd = np.where(pattern != 0.0, T, 0.0)
        if agg == "full":
            return full_sum(Wd)
        if agg == "none":
            return Wd[rid, cid]
        if agg == "right":
            return Wd @ V
        if agg == "left":
            return Wd.T @ U
        raise ValueError(agg)
    if mode == "masked":
        Ug = U[rid]                      # nnz x k
        Vg = V[cid]                      # nnz x k
        prod = Ug * Vg
        d = np.sum(prod, axis=1, dtype=LD).astype(np.float64) if prod.size else np.zeros(0)
        (t,) = eval_chain(chain, [output], dict(senv, a=np.asarray(X["vals"], dtype=np.float64), d=d,
                                                **cell_sides), d.shape)
        if agg == "full":
            return full_sum(t)
        if agg == "none":
            return t
        k = U.shape[1]
        if agg == "right":
            S = t[:, None] * Vg
            return np.stack([_segment_sum(S[:, c], rid, m) for c in range(k)], axis=1) \
                if k else np.zeros((m, 0))
        if agg == "left":
            S = t[:, None] * Ug
            return np.stack([_segment_sum(S[:, c], cid, n) for c in range(k)], axis=1) \
                if k else np.zeros((n, 0))
        raise ValueError(agg)
    raise ValueError(mode)


# --------------------------------------------------------------------------
# The five benchmark expressions, written out literally
# --------------------------------------------------------------------------
def sum_xyz(X, Y, Z):
    """sum(X * Y * Z) with its two intermediates (Fig. 1(a))."""
    T1 = X * Y
    T2 = T1 * Z
    return full_sum(T2)


def magg_xy_xz_xx(X, Y, Z):
    """(sum(X*Y), sum(X*Z), sum(X*X)): three separate aggregates (Fig. 1(c))."""
    T1 = X * Y
    s1 = full_sum(T1)
    T2 = X * Z
    s2 = full_sum(T2)
    T3 = X * X
    s3 = full_sum(T3)
    return np.array([s1, s2, s3], dtype=np.float64)


def row_chain_dense(X, v, w):
    """t(X) %*% (w * (X %*% v)), dense X (Fig. 1(b) with a weight vector)."""
    t1 = X @ v
    t2 = w * t1
    return X.T @ t2


def row_chain_csr(X, v, w):
    """Same expression with X in CSR."""
    t1 = _matvec(X, v)
    t2 = w * t1
    return _tmatvec(X, t2)


def outer_wsloss_dense(X, U, V):
    """sum(W * (X - U V^T)^2), W = (X != 0), all dense m x n intermediates."""
    m, n = X["rows"], X["cols"]
    Xd = np.zeros((m, n), dtype=np.float64)
    Xd[csr_row_ids(m, X["rowptr"]), np.asarray(X["colidx"], dtype=np.int64)] = X["vals"]
    P = U @ V.T
    D = Xd - P
    S = D * D
    W = (Xd != 0.0).astype(np.float64)
    M = W * S
    return full_sum(M)


def outer_wsloss_masked(X, U, V):
    """Same value from nnz-length intermediates only (U V^T is never formed)."""
    rid = csr_row_ids(X["rows"], X["rowptr"])
    cid = np.asarray(X["colidx"], dtype=np.int64)
    Ug = U[rid]
    Vg = V[cid]
    prod = Ug * Vg
    d = np.sum(prod, axis=1, dtype=LD).astype(np.float64) if prod.size else np.zeros(0)
    r = X["vals"] - d
    r2 = r * r
    wv = (X["vals"] != 0.0).astype(np.float64)
    t = wv * r2
    return full_sum(t)
