"""Helpers shared by the tests: tolerance checks and host<->device plumbing."""
import numpy as np

REL_TOL = 1e-10          # relative tolerance for fp64 aggregates and elementwise outputs
ABS_FLOOR = 1e-15        # times sum |terms|: floor for sums that cancel (about 9 units of roundoff)


def assert_close(got, ref, absscale=None, what="", max_floor=None):
    """|got - ref| <= REL_TOL * |ref| element by element.

    Where a sum cancels (|ref| far below the sum of the magnitudes of its terms,
    passed as `absscale`) no summation order can promise a relative error, so an
    element may instead meet ABS_FLOOR * absscale; such elements must stay rare
    (at most `max_floor` of them if given, else 2 % of the result).  Returns the
    number of elements that needed the floor.
    """
    got = np.asarray(got, dtype=np.float64).reshape(-1)
    ref = np.asarray(ref, dtype=np.float64).reshape(-1)
    assert got.shape == ref.shape, "%s: shape %s vs %s" % (what, got.shape, ref.shape)
    assert np.all(np.isfinite(got)), "%s: non-finite output" % what
    err = np.abs(got - ref)
    strict = err <= REL_TOL * np.abs(ref)
    if np.all(strict):
        return 0
    assert absscale is not None, "%s: max rel err %.3e" % (
        what, float(np.max(err / np.maximum(np.abs(ref), 1e-300))))
    absscale = np.broadcast_to(np.asarray(absscale, dtype=np.float64).reshape(-1), ref.shape)
    ok = strict | (err <= ABS_FLOOR * absscale)
    bad = np.flatnonzero(~ok)
    assert bad.size == 0, "%s: %d elements off, first %d: got %.17g ref %.17g" % (
        what, bad.size, bad[0] if bad.size else -1,
        got[bad[0]] if bad.size else 0, ref[bad[0]] if bad.size else 0)
    loose = int(np.count_nonzero(~strict))
    limit = max(1, ref.size // 50) if max_floor is None else max_floor
    assert loose <= limit, "%s: %d of %d elements needed the cancellation floor (limit %d)" % (
        what, loose, ref.size, limit)
    return loose


def to_dev(a, device="cuda"):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def csr_to_dev(w, device="cuda"):
    """Host CSR dict (rows, cols, rowptr, colidx, vals) -> binding.CSR on the device."""
    import paper_1801_00829_b200 as fo
    return fo.CSR(w["rows"], w["cols"], to_dev(w["rowptr"], device), to_dev(w["colidx"], device),
                  to_dev(w["vals"], device))


def host_csr(w):
    return {k: w[k] for k in ("rows", "cols", "rowptr", "colidx", "vals")}
