"""fused_cell_static: the entry point for callers that cannot allocate scratch.

It must give what fused_cell gives (same kernels, scratch taken from the array
built into the library instead of a caller-provided workspace), on repeated calls
that share that one array, whether this file runs alone or after every other test.
"""
import ctypes as C

import numpy as np
import pytest

import datagen
import oracle
from util import assert_close, to_dev

XYZ = [("mul", "t0", "a", "side0"), ("mul", "t1", "t0", "side1")]
GENERIC = [("sub", "t0", "a", "side0"), ("abs", "t1", "t0"), ("fma", "t2", "t1", "side1", 0.5)]


@pytest.mark.gpu
@pytest.mark.parametrize("agg", ["full", "col", "row", "none"])
@pytest.mark.parametrize("chain,output", [(XYZ, "t1"), (GENERIC, "t2")])
def test_static_scratch_matches_workspace_entry_point(agg, chain, output):
    import torch
    import paper_1801_00829_b200 as fo
    fo.load_library()
    rows, cols = 1537, 771
    w = datagen.cell_workload(rows, cols, seed=51)
    X, sides = to_dev(w["X"]), [("cell", to_dev(w["Y"])), ("cell", to_dev(w["Z"]))]
    ref = fo.fused_cell(chain, output, X, sides, agg=agg).cpu().numpy()
    assert_close(ref, oracle.cell(chain, output, w["X"], [("cell", w["Y"]), ("cell", w["Z"])], agg=agg),
                 what="workspace entry point %s" % agg)
    out = torch.empty(ref.shape, dtype=torch.float64, device="cuda")   # the caller owns the output
    for call in range(2):                                      # two calls in a row share the scratch
        out.fill_(float("nan"))
        fo.fused_cell_static(chain, output, X, sides, agg=agg, out=out)
        got = out.cpu().numpy()
        assert_close(got, ref, what="static %s call %d" % (agg, call))
        assert got.tobytes() == ref.tobytes()
    # a different shape right after, then the first one again: nothing stale is read
    w2 = datagen.cell_workload(97, 2049, seed=52)
    X2, s2 = to_dev(w2["X"]), [("cell", to_dev(w2["Y"])), ("cell", to_dev(w2["Z"]))]
    r2 = fo.fused_cell(chain, output, X2, s2, agg=agg).cpu().numpy()
    g2 = fo.fused_cell_static(chain, output, X2, s2, agg=agg).cpu().numpy()
    assert g2.tobytes() == r2.tobytes()
    fo.fused_cell_static(chain, output, X, sides, agg=agg, out=out)
    assert out.cpu().numpy().tobytes() == ref.tobytes()


@pytest.mark.gpu
@pytest.mark.parametrize("agg", ["full", "none"])
def test_static_entry_point_first_with_a_fresh_chain_compiles_and_allocates_nothing(agg):
    """The no-allocation promise, checked where it is hardest to keep: a chain that
    nothing has specialised yet, over contiguous inputs, is the case in which
    fused_cell would compile and load a kernel.  The static entry point must not:
    the compile counter and the free device memory stay as they were, and the
    result is the checker's."""
    import torch
    import paper_1801_00829_b200 as fo
    fo.load_library()
    rows, cols = 1029, 515
    w = datagen.cell_workload(rows, cols, seed=53)
    X, sides = to_dev(w["X"]), [("cell", to_dev(w["Y"])), ("cell", to_dev(w["Z"]))]
    # constants differ per variant so that each run meets a program nobody compiled
    k = {"full": 0.375, "none": 0.625}[agg]
    fresh = [("add", "t0", "a", "side1"), ("min", "t1", "t0", "side0"), ("mul", "t2", "t1", k),
             ("sub", "t3", "t2", "a")] + ([("neg", "t3", "t3")] if agg == "none" else [])
    shape = () if agg == "full" else (rows, cols)
    out = torch.empty(shape, dtype=torch.float64, device="cuda")
    fo.fused_cell_static([("sq", "t0", "a")], "t0", X, agg="full")   # the one-time address lookup
    torch.cuda.synchronize()
    compiled = fo.jit_stats()[1]
    free0 = torch.cuda.mem_get_info()[0]
    fo.fused_cell_static(fresh, "t3", X, sides, agg=agg, out=out)
    torch.cuda.synchronize()
    assert fo.jit_stats()[1] == compiled, "the static entry point compiled a kernel"
    assert torch.cuda.mem_get_info()[0] == free0, "device memory was allocated"
    sides_h = [("cell", w["Y"]), ("cell", w["Z"])]
    ref = oracle.cell(fresh, "t3", w["X"], sides_h, agg=agg)
    if agg == "full":
        scale = np.abs(w["X"]).sum() * 2 + np.abs(w["Y"]).sum() + np.abs(w["Z"]).sum()
        assert_close([out.item()], [ref], absscale=scale, what="static, fresh chain")
    else:
        assert_close(out.cpu().numpy(), ref, what="static, fresh chain")
    # after fused_cell has specialised the chain the static call reuses that kernel: same bits
    first = out.cpu().numpy().copy()
    again = fo.fused_cell(fresh, "t3", X, sides, agg=agg).cpu().numpy()
    fo.fused_cell_static(fresh, "t3", X, sides, agg=agg, out=out)
    assert out.cpu().numpy().tobytes() == again.tobytes() == first.tobytes()


@pytest.mark.gpu
def test_static_scratch_limit_is_reported():
    import torch
    import paper_1801_00829_b200 as fo
    from paper_1801_00829_b200 import binding as B
    lib = fo.load_library()
    limit = lib.fused_cell_static_limit_bytes()
    assert limit == 1 << 20
    # column aggregation of a wide matrix needs panels * cols doubles of scratch
    rows, cols = 64, 300_000
    X = torch.ones((rows, cols), dtype=torch.float64, device="cuda")
    m = B._mat(X)
    assert lib.fused_cell_workspace_bytes(C.byref(m), 2) > limit
    with pytest.raises(fo.FusedOpsError) as err:
        fo.fused_cell_static([("sq", "t0", "a")], "t0", X, agg="col")
    assert err.value.status == -8
    # the same matrix is fine for the variants whose scratch does not grow with it
    assert fo.fused_cell_static([("sq", "t0", "a")], "t0", X, agg="full").item() == float(rows * cols)
    assert fo.fused_cell([("sq", "t0", "a")], "t0", X, agg="col").cpu().numpy().tolist() == [float(rows)] * cols


def test_static_entry_point_rejects_bad_arguments_without_a_gpu():
    from paper_1801_00829_b200 import binding as B
    lib = B.load_library()
    ch, keep = B.make_chain([("sq", "t0", "a")], "t0")
    m = B.fo_mat()
    m.kind = 0
    m.dense.rows, m.dense.cols, m.dense.ld, m.dense.data = 64, 400_000, 400_000, 0x1000
    sarr = (B.fo_side * 1)()
    sc = (C.c_double * 8)()
    # too large for the built-in scratch: refused before anything touches a device
    assert lib.fused_cell_static(C.byref(ch), C.byref(m), sarr, 0, sc, 0, 2, C.c_void_p(0x2000), None) == -8
    assert lib.fused_cell_static(C.byref(ch), None, sarr, 0, sc, 0, 3, C.c_void_p(0x2000), None) == -1
    assert lib.fused_cell_static(C.byref(ch), C.byref(m), sarr, 0, sc, 0, 9, C.c_void_p(0x2000), None) == -4
