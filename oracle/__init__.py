"""CPU checker for the fused operators.  TEST INFRASTRUCTURE, NOT A PRODUCT PATH.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares no code with the CUDA library or its Python binding and
imports neither.

What it computes.  The paper's premise (Section 1, "Fusion Opportunities";
Section 2.2) is that a fused operator returns exactly what the chain of basic
operators it replaces returns.  So every function here evaluates its expression
*unfused*: one basic operator at a time over whole arrays, every intermediate
materialised as a full numpy array, all in float64.  Which sums are more
accurate than a plain float64 loop, and which are not:
  * full, row and column sums of a materialised array (``full_sum``,
    ``row_sums``, ``col_sums``) and the per-cell dot products of the Outer
    template's masked mode accumulate pairwise in numpy ``longdouble`` and are
    rounded once at the end;
  * matrix products (``X @ v``, ``X.T @ t``, ``X @ B``, ``U @ V.T``) are the
    library's float64 routine (blocked, possibly threaded: the order of its
    additions is the library's), and segmented sums over CSR rows or columns are
    ``np.bincount`` (sequential float64).  For these the checker is a second
    float64 opinion, not a more accurate one; the tests' tolerance allows for it
    (relative 1e-10, with a floor proportional to the sum of the magnitudes of
    the terms where a sum cancels).
Library primitives used as single steps: elementwise numpy ufuncs, ``@``
(matrix product), ``np.bincount`` (segmented sum), fancy-index gathers.

Pins (see tests/test_oracle_pins.py): closed forms with exactly representable
values, brute-force pure-Python loops on tiny inputs with exact rational
arithmetic, algebraic identities, and the dense-vs-masked agreement of the
Outer template.  Every function below is covered by at least one of them.

Chains.  A scalar operator chain is a list of steps ``(op, dst, a[, b[, c]])``:
``dst`` is a temporary name ``"t0".."t7"``; operands are ``"a"`` (main-input
value), ``"d"`` (Row: the row's dot product, for the B1 variants one entry of the row's
product with the side matrix; Outer: U_i . V_j), ``"rowsum"`` (B1 variants: the
row sum of the first chain), ``"sideK"``,
``"sK"`` (K-th scalar), ``"tK"`` or a Python float.  Outputs are operand names.
"""
from .ops import (
    OPS, eval_chain, full_sum, row_sums, col_sums,
    cell, magg, row, row_b1, outer,
    mmchain, mlogreg_inner,
    sum_xyz, magg_xy_xz_xx, row_chain_dense, row_chain_csr,
    outer_wsloss_dense, outer_wsloss_masked,
    csr_row_ids, count_nonzero,
)

__all__ = [
    "OPS", "eval_chain", "full_sum", "row_sums", "col_sums",
    "cell", "magg", "row", "row_b1", "outer", "mmchain", "mlogreg_inner",
    "sum_xyz", "magg_xy_xz_xx", "row_chain_dense", "row_chain_csr",
    "outer_wsloss_dense", "outer_wsloss_masked", "csr_row_ids", "count_nonzero",
]
