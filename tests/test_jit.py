"""Run-time specialised Cell / MAgg chains: the generated kernels compile (checked
without a GPU) and, on a GPU, give the interpreter's bits, are cached by chain, and
do not depend on the values of scalars and immediates."""
import numpy as np
import pytest

import datagen
import oracle
from util import assert_close, to_dev

import paper_1801_00829_b200 as fo

CHAINS = {
    "abs-fma": ([("sub", "t0", "a", "side0"), ("abs", "t1", "t0"), ("fma", "t2", "t1", "side1", 0.5)], ["t2"], 2, 0),
    "scalars": ([("mul", "t0", "a", "s0"), ("add", "t1", "t0", "s1"), ("max", "t2", "t1", "side0")], ["t2"], 1, 2),
    "cmp-sel": ([("gt", "t0", "a", "side0"), ("sel", "t1", "t0", "a", "side0"), ("min", "t2", "t1", 0.75)], ["t2"], 1, 0),
    "math": ([("abs", "t0", "a"), ("add", "t1", "t0", 1.0), ("log", "t2", "t1"), ("exp", "t3", "t2"),
              ("sqrt", "t4", "t3"), ("pow", "t5", "t4", 1.5), ("div", "t6", "t5", "t1"), ("neg", "t7", "t6")],
             ["t7"], 0, 0),
    "only-side1": ([("mul", "t0", "a", "side1")], ["t0"], 2, 0),
    "magg5": ([("mul", "t0", "a", "side0"), ("sub", "t1", "a", "side0"), ("sq", "t2", "t1"),
               ("eq", "t3", "a", "side0"), ("ne", "t4", "a", 0.0)], ["t0", "t1", "t2", "t3", "t4"], 1, 0),
    "passthrough": ([], ["a"], 0, 0),
}


@pytest.mark.parametrize("name", sorted(CHAINS))
@pytest.mark.parametrize("store", [False, True])
def test_generated_kernels_compile_without_a_gpu(name, store):
    steps, outs, n_sides, n_scalars = CHAINS[name]
    if store and len(outs) > 1:
        pytest.skip("no_agg has one result")
    rc, log = fo.jit_compile_check(steps, outs, n_sides, n_scalars, store)
    if rc == -4:
        pytest.skip("NVRTC not available here")
    assert rc == 0, log
    assert "error" not in log


def test_compile_check_rejects_bad_chain():
    rc, _ = fo.jit_compile_check([("mul", "t0", "a", "t3")], ["t0"])
    assert rc == -3


@pytest.mark.gpu
@pytest.mark.parametrize("name", sorted(CHAINS))
def test_jit_equals_interpreter_bitwise_and_checker(name):
    steps, outs, n_sides, n_scalars = CHAINS[name]
    rows, cols = 1031, 517                      # full tiles and a ragged tail
    X = datagen.uniform(61, 0, rows * cols, -1.0, 2.0).reshape(rows, cols)
    S = [datagen.uniform(61, 2 + k, rows * cols, -1.0, 2.0).reshape(rows, cols) for k in range(n_sides)]
    scalars = [1.25, -0.5][:n_scalars]
    sides_h = [("cell", s) for s in S]
    Xd, sides = to_dev(X), [("cell", to_dev(s)) for s in S]
    usable, c0, l0, f0 = fo.jit_stats()
    if not usable:
        pytest.skip("NVRTC or the driver library is not usable here")
    got = fo.fused_magg(steps, outs, Xd, sides, scalars).cpu().numpy()
    usable, c1, l1, f1 = fo.jit_stats()
    assert f1 == f0, "a specialised kernel failed to compile"
    assert l1 == l0 + 1 and c1 in (c0, c0 + 1)
    again = fo.fused_magg(steps, outs, Xd, sides, scalars).cpu().numpy()
    assert fo.jit_stats()[1] == c1                                   # cached: nothing compiled again
    assert again.tobytes() == got.tobytes()
    try:
        fo.force_interpreter(True)
        slow = fo.fused_magg(steps, outs, Xd, sides, scalars).cpu().numpy()
    finally:
        fo.force_interpreter(False)
    assert got.tobytes() == slow.tobytes()
    ref = oracle.magg(steps, outs, X, sides_h, scalars)
    absref = oracle.magg(steps + [("abs", "t%d" % k, o) for k, o in enumerate(outs)],
                         ["t%d" % k for k in range(len(outs))], X, sides_h, scalars)
    assert_close(got, ref, absscale=absref + 1.0, what=name)
    if len(outs) == 1:                                               # no_agg through the same mechanism
        e = fo.fused_cell(steps, outs[0], Xd, sides, scalars, agg="none").cpu().numpy()
        assert_close(e, oracle.cell(steps, outs[0], X, sides_h, scalars, agg="none"), what=name + " none")


@pytest.mark.gpu
def test_jit_kernel_is_reused_for_other_constants_and_can_be_switched_off():
    rows, cols = 300, 700
    X = datagen.normal(62, 0, rows * cols).reshape(rows, cols)
    Xd = to_dev(X)
    if not fo.jit_stats()[0]:
        pytest.skip("NVRTC or the driver library is not usable here")

    def chain(k):
        return [("mul", "t0", "a", "s0"), ("add", "t1", "t0", k)]

    a = fo.fused_cell(chain(2.0), "t1", Xd, scalars=[3.0]).item()
    compiled = fo.jit_stats()[1]
    b = fo.fused_cell(chain(-7.0), "t1", Xd, scalars=[0.25]).item()
    assert fo.jit_stats()[1] == compiled                             # same program, other constants
    assert_close([a], [oracle.cell(chain(2.0), "t1", X, scalars=[3.0])], absscale=np.abs(X).sum() * 3 + 2 * X.size)
    assert_close([b], [oracle.cell(chain(-7.0), "t1", X, scalars=[0.25])], absscale=np.abs(X).sum() + 7 * X.size)
    launches = fo.jit_stats()[2]
    try:
        fo.set_jit(False)
        c = fo.fused_cell(chain(-7.0), "t1", Xd, scalars=[0.25]).item()
    finally:
        fo.set_jit(True)
    assert fo.jit_stats()[2] == launches and c == b                  # interpreter, same bits


@pytest.mark.gpu
def test_prepared_mode_never_compiles_inside_a_call():
    rows, cols = 257, 130
    X = datagen.normal(63, 0, rows * cols).reshape(rows, cols)
    Xd = to_dev(X)
    if not fo.jit_stats()[0]:
        pytest.skip("NVRTC or the driver library is not usable here")
    fresh = [("mul", "t0", "a", 1.5), ("max", "t1", "t0", "a"), ("sub", "t2", "t1", 0.125)]
    ref = oracle.cell(fresh, "t2", X)
    scale = np.abs(X).sum() * 1.5 + 0.125 * X.size
    old = fo.set_jit(fo.binding.JIT_PREPARED)
    try:
        compiled, launches = fo.jit_stats()[1:3]
        a = fo.fused_cell(fresh, "t2", Xd).item()                    # not prepared: the interpreter runs
        assert fo.jit_stats()[1:3] == (compiled, launches)
        fo.jit_prepare(fresh, "t2")
        assert fo.jit_stats()[1] == compiled + 1
        fo.jit_prepare(fresh, "t2")                                  # cached: nothing compiled again
        assert fo.jit_stats()[1] == compiled + 1
        b = fo.fused_cell(fresh, "t2", Xd).item()                    # the prepared kernel is picked up
        assert fo.jit_stats()[1:3] == (compiled + 1, launches + 1)
    finally:
        fo.set_jit(old)
    assert a == b
    assert_close([a], [ref], absscale=scale)


@pytest.mark.parametrize("skeleton", [2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("name", ["abs-fma", "scalars", "math"])
def test_every_kernel_skeleton_compiles_without_a_gpu(name, skeleton):
    """The row-wise, column and CSR kernels of the Cell template with a generated chain
    (2 - 4 rows: row_agg, no_agg, full_agg; 5 columns; 6 - 8 CSR with 2, 8, 32 lanes per row)."""
    steps, outs, n_sides, n_scalars = CHAINS[name]
    rc, log = fo.jit_compile_check(steps, outs, n_sides, n_scalars, skeleton)
    if rc == -4:
        pytest.skip("NVRTC not available here")
    assert rc == 0, log
    assert "error" not in log


@pytest.mark.gpu
@pytest.mark.parametrize("name", ["abs-fma", "scalars", "cmp-sel"])
def test_jit_in_the_row_column_and_csr_kernels_equals_interpreter_bitwise_and_checker(name):
    """Layouts that do not take the flat stream: a padded leading dimension, a column-vector
    side, row and column aggregation, and a CSR main input.  Each runs a kernel compiled
    for the chain; the bits are the interpreter's, the values the checker's."""
    import torch
    steps, outs, n_sides, n_scalars = CHAINS[name]
    if not fo.jit_stats()[0]:
        pytest.skip("NVRTC or the driver library is not usable here")
    rows, cols = 517, 131
    X = datagen.uniform(71, 0, rows * cols, -1.0, 2.0).reshape(rows, cols)
    S = [datagen.uniform(71, 2 + k, rows * cols, -1.0, 2.0).reshape(rows, cols) for k in range(n_sides)]
    scalars = [1.25, -0.5][:n_scalars]
    pad = torch.zeros((rows, cols + 3), dtype=torch.float64, device="cuda")
    pad[:, :cols] = to_dev(X)
    Xd = pad[:, :cols]                                             # leading dimension cols + 3
    sides_d = [("cell", to_dev(s)) for s in S]
    sides_h = [("cell", s) for s in S]
    for agg in ("full", "row", "col", "none"):
        launches = fo.jit_stats()[2]
        got = fo.fused_cell(steps, outs[0], Xd, sides_d, scalars, agg=agg).cpu().numpy()
        assert fo.jit_stats()[2] == launches + 1, "the %s kernel was not specialised" % agg
        try:
            fo.force_interpreter(True)
            slow = fo.fused_cell(steps, outs[0], Xd, sides_d, scalars, agg=agg).cpu().numpy()
        finally:
            fo.force_interpreter(False)
        assert got.tobytes() == slow.tobytes()
        ref = oracle.cell(steps, outs[0], X, sides_h, scalars, agg=agg)
        absref = oracle.cell(steps + [("abs", "t7", outs[0])], "t7", X, sides_h, scalars, agg=agg)
        assert_close(got, ref, absscale=np.asarray(absref) + 1.0, what="%s %s" % (name, agg))
    # a CSR main input: stored cells only
    w = datagen.outer_workload(rows, cols, 2, 0.1, seed=72)
    Xh = {k: w[k] for k in ("rows", "cols", "rowptr", "colidx", "vals")}
    Xc = fo.CSR(rows, cols, to_dev(w["rowptr"]), to_dev(w["colidx"]), to_dev(w["vals"]))
    for agg in ("full", "row", "col", "none"):
        launches = fo.jit_stats()[2]
        got = fo.fused_cell(steps, outs[0], Xc, sides_d, scalars, agg=agg).cpu().numpy()
        assert fo.jit_stats()[2] == launches + 1
        try:
            fo.force_interpreter(True)
            slow = fo.fused_cell(steps, outs[0], Xc, sides_d, scalars, agg=agg).cpu().numpy()
        finally:
            fo.force_interpreter(False)
        if agg != "col":                                           # (col_agg over CSR adds through atomics)
            assert got.tobytes() == slow.tobytes()
        ref = oracle.cell(steps, outs[0], Xh, sides_h, scalars, agg=agg)
        absref = oracle.cell(steps + [("abs", "t7", outs[0])], "t7", Xh, sides_h, scalars, agg=agg)
        assert_close(got, ref, absscale=np.asarray(absref) + 1.0, what="%s csr %s" % (name, agg))


@pytest.mark.gpu
def test_prepare_call_makes_the_kernel_of_a_call_ready():
    import torch
    if not fo.jit_stats()[0]:
        pytest.skip("NVRTC or the driver library is not usable here")
    rows, cols = 300, 77
    X = datagen.normal(73, 0, rows * cols).reshape(rows, cols)
    r = datagen.uniform(73, 1, rows, 0.5, 1.5)
    Xd, rd = to_dev(X), to_dev(r)
    fresh = [("mul", "t0", "a", "side0"), ("min", "t1", "t0", 0.625), ("add", "t2", "t1", "a")]
    old = fo.set_jit(fo.binding.JIT_PREPARED)
    try:
        compiled, launches = fo.jit_stats()[1:3]
        fo.jit_prepare_call(fresh, "t2", Xd, [("row", rd)], agg="row")       # a column-vector side: the row-wise kernel
        assert fo.jit_stats()[1] == compiled + 1
        got = fo.fused_cell(fresh, "t2", Xd, [("row", rd)], agg="row").cpu().numpy()
        assert fo.jit_stats()[1:3] == (compiled + 1, launches + 1)
        other = fo.fused_cell(fresh, "t2", Xd, [("row", rd)], agg="col").cpu().numpy()   # not prepared: interpreted
        assert fo.jit_stats()[1:3] == (compiled + 1, launches + 1)
    finally:
        fo.set_jit(old)
    assert_close(got, oracle.cell(fresh, "t2", X, [("row", r)], agg="row"),
                 absscale=np.abs(X).sum(axis=1) * 3 + cols, what="prepared row_agg")
    assert_close(other, oracle.cell(fresh, "t2", X, [("row", r)], agg="col"),
                 absscale=np.abs(X).sum(axis=0) * 3 + rows, what="interpreted col_agg")
    # a chain with a built-in form needs nothing
    fo.jit_prepare_call([("mul", "t0", "a", "side0")], "t0", Xd, [("cell", Xd)], agg="full")
    assert fo.jit_stats()[1] == compiled + 1


OUTER_GENERIC = [("sub", "t1", "a", "d"), ("abs", "t2", "t1"), ("add", "t3", "t2", 0.25)]


@pytest.mark.parametrize("kernel", range(8))
def test_outer_kernels_compile_with_a_generated_chain_without_a_gpu(kernel):
    rc, log = fo.jit_compile_check_outer(OUTER_GENERIC, "t3", 0, 0, kernel)
    if rc == -4:
        pytest.skip("NVRTC not available here")
    assert rc == 0, log
    assert "error" not in log
    sides_chain = [("sub", "t0", "a", "d"), ("mul", "t1", "t0", "side0"), ("add", "t2", "t1", "side1")]
    rc, log = fo.jit_compile_check_outer(sides_chain, "t2", 2, 0, kernel)
    assert rc == 0, log


@pytest.mark.gpu
@pytest.mark.parametrize("schedule", ["bulk", "pipe", "direct", "dense"])
def test_outer_chain_compiled_at_run_time_equals_interpreter_bitwise_and_checker(schedule):
    if not fo.jit_stats()[0]:
        pytest.skip("NVRTC or the driver library is not usable here")
    w = datagen.outer_workload(300, 257, 20, 0.3 if schedule == "dense" else 0.05, seed=77)
    Xh = {k: w[k] for k in ("rows", "cols", "rowptr", "colidx", "vals")}
    X = fo.CSR(w["rows"], w["cols"], to_dev(w["rowptr"]), to_dev(w["colidx"]), to_dev(w["vals"]))
    Ud, Vd = to_dev(w["U"]), to_dev(w["V"])
    fo.tune("outer.kernel", schedule)
    try:
        for agg in ("full", "none") + (() if schedule in ("dense", "bulk") else ("right",)) + (("left",) if schedule == "direct" else ()):
            launches = fo.jit_stats()[2]
            fast = fo.fused_outer(OUTER_GENERIC, "t3", X, Ud, Vd, agg=agg).cpu().numpy()
            assert fo.jit_stats()[2] == launches + 1, "%s %s was not specialised" % (schedule, agg)
            try:
                fo.force_interpreter(True)
                slow = fo.fused_outer(OUTER_GENERIC, "t3", X, Ud, Vd, agg=agg).cpu().numpy()
            finally:
                fo.force_interpreter(False)
            if agg != "left":                                      # (left_mm adds through atomics)
                assert fast.tobytes() == slow.tobytes()
            ref = oracle.outer(OUTER_GENERIC, "t3", Xh, w["U"], w["V"], agg=agg, mode="masked")
            assert_close(fast, ref, absscale=np.abs(ref) + 1.0, what="outer jit %s %s" % (schedule, agg))
    finally:
        fo.tune("outer.kernel", None)
    # side inputs through a compiled chain (the per-cell kernel with plain gathers)
    r = datagen.uniform(77, 9, w["rows"], 0.5, 2.0)
    chain = [("sub", "t0", "a", "d"), ("mul", "t1", "t0", "side0")]
    got = fo.fused_outer(chain, "t1", X, Ud, Vd, agg="none", sides=[("row", to_dev(r))]).cpu().numpy()
    assert_close(got, oracle.outer(chain, "t1", Xh, w["U"], w["V"], agg="none", sides=[("row", r)]),
                 what="outer jit sides")


ROW_GENERIC = [("mul", "t0", "side0", "d"), ("abs", "t1", "t0"), ("sub", "t2", "t1", 0.5)]


@pytest.mark.parametrize("kernel", range(6))
def test_row_kernels_compile_with_a_generated_chain_without_a_gpu(kernel):
    rc, log = fo.jit_compile_check_row(ROW_GENERIC, "t2", 1, 0, kernel)
    if rc == -4:
        pytest.skip("NVRTC not available here")
    assert rc == 0, log
    assert "error" not in log


@pytest.mark.gpu
@pytest.mark.parametrize("layout", ["dense-1000", "dense-100", "narrow-10", "csr"])
def test_row_chain_compiled_at_run_time_equals_interpreter_bitwise_and_checker(layout):
    if not fo.jit_stats()[0]:
        pytest.skip("NVRTC or the driver library is not usable here")
    rows = 3001
    if layout == "csr":
        c = datagen.row_csr_workload(rows, 500, 0.02, seed=91)
        Xh = {k: c[k] for k in ("rows", "cols", "rowptr", "colidx", "vals")}
        X = fo.CSR(rows, 500, to_dev(c["rowptr"]), to_dev(c["colidx"]), to_dev(c["vals"]))
        v, w = c["v"], c["w"]
        Xabs = dict(Xh, vals=np.abs(c["vals"]))
    else:
        cols = int(layout.split("-")[1])
        r = datagen.row_dense_workload(rows, cols, seed=91)
        Xh, v, w = r["X"], r["v"], r["w"]
        X = to_dev(Xh)
        Xabs = np.abs(Xh)
    for agg in ("col_t", "row", "full", "none"):
        launches = fo.jit_stats()[2]
        fast = fo.fused_row(ROW_GENERIC, "t2", X, to_dev(v), [("row", to_dev(w))], agg=agg).cpu().numpy()
        assert fo.jit_stats()[2] == launches + 1, "%s %s was not specialised" % (layout, agg)
        try:
            fo.force_interpreter(True)
            slow = fo.fused_row(ROW_GENERIC, "t2", X, to_dev(v), [("row", to_dev(w))], agg=agg).cpu().numpy()
        finally:
            fo.force_interpreter(False)
        if not (layout == "csr" and agg == "col_t"):               # (the CSR column scatter adds through atomics)
            assert fast.tobytes() == slow.tobytes()
        ref = oracle.row(ROW_GENERIC, "t2", Xh, v, [("row", w)], agg=agg)
        scale = oracle.row([("mul", "t0", "side0", "d"), ("add", "t2", "t0", 0.5)], "t2", Xabs, np.abs(v),
                           [("row", w)], agg=agg)
        assert_close(fast, ref, absscale=np.abs(scale) + 1e-300, what="row jit %s %s" % (layout, agg))
