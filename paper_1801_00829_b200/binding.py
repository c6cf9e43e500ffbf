"""ctypes binding of libfusedops.so: argument marshalling only.

Every step of the fused operators runs inside the CUDA library.  PyTorch is used
for device memory (inputs, outputs, the scratch workspace) and for the current
stream; nothing here computes.  If the library is missing or no CUDA device is
present the calls raise - there is no CPU path.

Chains are written as lists of steps ``(op, dst, a[, b[, c]])`` with ``dst`` one
of "t0".."t7" and operands "a" (main value), "d" (dot product), "sideK", "sK"
(K-th scalar), "tK" or a Python float (an immediate); see include/fusedops.h.
"""
from __future__ import annotations

import ctypes as C
import os
import threading

import torch

from . import build as _build

FO_MAX_OPS, FO_MAX_TMPS, FO_MAX_SIDES, FO_MAX_SCALARS, FO_MAX_OUT = 32, 8, 4, 8, 8

OPCODES = {name: i for i, name in enumerate([
    "mov", "neg", "abs", "sqrt", "exp", "log", "sq",
    "add", "sub", "mul", "div", "min", "max", "pow",
    "eq", "ne", "lt", "le", "gt", "ge", "sel", "fma"])}
ARITY = {**{n: 1 for n in ("mov", "neg", "abs", "sqrt", "exp", "log", "sq")},
         **{n: 2 for n in ("add", "sub", "mul", "div", "min", "max", "pow",
                           "eq", "ne", "lt", "le", "gt", "ge")},
         "sel": 3, "fma": 3}

CELL_AGG = {"none": 0, "row": 1, "col": 2, "full": 3}
ROW_AGG = {"none": 0, "row": 1, "col": 2, "full": 3, "col_t": 4}
ROW_B1_AGG = {"none": 5, "col_t": 6}
OUTER_AGG = {"left": 0, "right": 1, "none": 2, "full": 3}
ACCESS = {"cell": 0, "row": 1, "col": 2}

STATUS = {0: "FO_OK", -1: "FO_ERR_NULL", -2: "FO_ERR_SHAPE", -3: "FO_ERR_CHAIN",
          -4: "FO_ERR_UNSUPPORTED", -5: "FO_ERR_WORKSPACE", -6: "FO_ERR_CUDA",
          -7: "FO_ERR_DEVICE_TIMEOUT", -8: "FO_ERR_STATIC_LIMIT"}


class FusedOpsError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__("%s: %s (%s)" % (what, STATUS.get(status, status), _status_text(status)))


# ------------------------------------------------------------------ C structs
class fo_dense(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64), ("data", C.c_void_p)]


class fo_csr(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("nnz", C.c_int64),
                ("rowptr", C.c_void_p), ("colidx", C.c_void_p), ("vals", C.c_void_p)]


class fo_mat(C.Structure):
    _fields_ = [("kind", C.c_int32), ("reserved", C.c_int32), ("dense", fo_dense), ("csr", fo_csr)]


class fo_side(C.Structure):
    _fields_ = [("m", fo_dense), ("access", C.c_int32), ("reserved", C.c_int32), ("sparse", C.c_void_p)]


class fo_op(C.Structure):
    _fields_ = [("opcode", C.c_uint8), ("dst", C.c_uint8), ("a", C.c_uint8), ("b", C.c_uint8),
                ("c", C.c_uint8), ("reserved", C.c_uint8 * 3), ("imm", C.c_double)]


class fo_chain(C.Structure):
    _fields_ = [("n_ops", C.c_int32), ("n_out", C.c_int32), ("ops", C.POINTER(fo_op)),
                ("out", C.c_uint8 * FO_MAX_OUT)]


EXPORTS = [
    "fused_cell", "fused_magg", "fused_row", "fused_outer", "fused_row_b1",
    "fused_row_b1_workspace_bytes",
    "fused_cell_workspace_bytes", "fused_magg_workspace_bytes", "fused_row_workspace_bytes",
    "fused_outer_workspace_bytes", "fo_workspace_init", "fo_query_device_status",
    "fo_status_string", "fo_last_cuda_error", "fo_set_force_interpreter",
    "fused_cell_static", "fused_cell_static_limit_bytes",
    "fo_set_jit", "fo_jit_stats", "fo_jit_prepare", "fo_jit_prepare_call", "fo_jit_compile_check", "fo_jit_compile_check_outer", "fo_jit_compile_check_row",
    "fo_probe_out_len", "fo_probe_l2_gather", "fo_probe_bulk_gather", "fo_probe_fp64_fma", "fo_chain_describe", "fo_tune", "fo_cell_stamps",
]

_lib = None
_lock = threading.Lock()


def load_library(path=None):
    """Loads (building first if stale) libfusedops.so and declares its prototypes."""
    global _lib
    with _lock:
        if _lib is not None and path is None:
            return _lib
        lib = C.CDLL(path or _build.build_library())
        vp, dp, i32, sz = C.c_void_p, C.c_void_p, C.c_int, C.c_size_t
        chain_p, mat_p, side_p = C.POINTER(fo_chain), C.POINTER(fo_mat), C.POINTER(fo_side)
        scal_p = C.POINTER(C.c_double)
        lib.fused_cell.argtypes = [chain_p, mat_p, side_p, i32, scal_p, i32, i32, dp, vp, vp, sz, vp]
        lib.fused_magg.argtypes = [chain_p, mat_p, side_p, i32, scal_p, i32, dp, vp, sz, vp]
        lib.fused_row.argtypes = [chain_p, mat_p, dp, side_p, i32, scal_p, i32, i32, dp, vp, sz, vp]
        lib.fused_outer.argtypes = [chain_p, C.POINTER(fo_csr), C.POINTER(fo_dense),
                                    C.POINTER(fo_dense), side_p, i32, scal_p, i32, i32, dp, vp, vp, sz, vp]
        lib.fused_row_b1.argtypes = [chain_p, chain_p, mat_p, C.POINTER(fo_dense), side_p, i32, scal_p, i32,
                                     i32, dp, vp, sz, vp]
        for f in (lib.fused_cell, lib.fused_magg, lib.fused_row, lib.fused_outer, lib.fused_row_b1):
            f.restype = C.c_int
        lib.fused_row_b1_workspace_bytes.argtypes = [mat_p, i32, i32]
        lib.fused_row_b1_workspace_bytes.restype = C.c_size_t
        lib.fused_cell_workspace_bytes.argtypes = [mat_p, i32]
        lib.fused_magg_workspace_bytes.argtypes = [mat_p, i32]
        lib.fused_row_workspace_bytes.argtypes = [mat_p, i32]
        lib.fused_outer_workspace_bytes.argtypes = [C.POINTER(fo_csr), i32, i32]
        for f in (lib.fused_cell_workspace_bytes, lib.fused_magg_workspace_bytes,
                  lib.fused_row_workspace_bytes, lib.fused_outer_workspace_bytes):
            f.restype = C.c_size_t
        lib.fo_workspace_init.argtypes = [vp, sz, vp]
        lib.fo_workspace_init.restype = C.c_int
        lib.fo_query_device_status.argtypes = [vp, vp, C.POINTER(C.c_int)]
        lib.fo_query_device_status.restype = C.c_int
        lib.fo_status_string.argtypes = [C.c_int]
        lib.fo_status_string.restype = C.c_char_p
        lib.fo_last_cuda_error.argtypes = []
        lib.fo_last_cuda_error.restype = C.c_int
        lib.fused_cell_static.argtypes = [chain_p, mat_p, side_p, i32, scal_p, i32, i32, dp, vp]
        lib.fused_cell_static.restype = C.c_int
        lib.fused_cell_static_limit_bytes.argtypes = []
        lib.fused_cell_static_limit_bytes.restype = C.c_size_t
        lib.fo_set_jit.argtypes = [C.c_int]
        lib.fo_set_jit.restype = C.c_int
        ip = C.POINTER(C.c_int)
        lib.fo_jit_stats.argtypes = [ip, ip, ip]
        lib.fo_jit_stats.restype = C.c_int
        lib.fo_cell_stamps.argtypes = [vp, vp, C.POINTER(C.c_ulonglong)]
        lib.fo_cell_stamps.restype = C.c_int
        lib.fo_tune.argtypes = [C.c_char_p, C.c_char_p]
        lib.fo_tune.restype = C.c_int
        lib.fo_jit_prepare_call.argtypes = [chain_p, mat_p, side_p, i32, i32, i32, i32]
        lib.fo_jit_prepare_call.restype = C.c_int
        lib.fo_jit_prepare.argtypes = [chain_p, i32, i32, i32]
        lib.fo_jit_prepare.restype = C.c_int
        lib.fo_jit_compile_check.argtypes = [chain_p, i32, i32, i32, C.c_char_p, sz]
        lib.fo_jit_compile_check.restype = C.c_int
        lib.fo_jit_compile_check_outer.argtypes = [chain_p, i32, i32, i32, C.c_char_p, sz]
        lib.fo_jit_compile_check_outer.restype = C.c_int
        lib.fo_jit_compile_check_row.argtypes = [chain_p, i32, i32, i32, C.c_char_p, sz]
        lib.fo_jit_compile_check_row.restype = C.c_int
        lib.fo_set_force_interpreter.argtypes = [C.c_int]
        lib.fo_set_force_interpreter.restype = C.c_int
        lib.fo_chain_describe.argtypes = [chain_p, i32, i32, scal_p, i32, i32, C.c_char_p, sz]
        lib.fo_chain_describe.restype = C.c_int
        lib.fo_probe_out_len.argtypes = []
        lib.fo_probe_out_len.restype = C.c_size_t
        lib.fo_probe_l2_gather.argtypes = [C.POINTER(fo_dense), vp, C.c_longlong, dp, vp]
        lib.fo_probe_l2_gather.restype = C.c_int
        lib.fo_probe_bulk_gather.argtypes = [C.POINTER(fo_dense), vp, C.c_longlong, dp, vp]
        lib.fo_probe_bulk_gather.restype = C.c_int
        lib.fo_probe_fp64_fma.argtypes = [C.c_longlong, dp, vp]
        lib.fo_probe_fp64_fma.restype = C.c_int
        if path is None:
            _lib = lib
        return lib


def _status_text(status):
    try:
        return load_library().fo_status_string(int(status)).decode()
    except Exception:
        return "?"


def _check(status, what):
    if status != 0:
        raise FusedOpsError(status, what)


# ------------------------------------------------------------------ marshalling
def _operand(x, allow_imm=True, rowsum_side=None):
    """Operand name -> (operand byte, immediate or None).  "rowsum" (second chain of
    fused_row_b1) is the side slot `rowsum_side`, right behind the call's own sides."""
    if x == "rowsum" and rowsum_side is not None:
        return 0x40 | int(rowsum_side), None
    if isinstance(x, (int, float)) and not isinstance(x, bool):
        if not allow_imm:
            raise ValueError("an output cannot be an immediate")
        return 0xC2, float(x)
    if not isinstance(x, str):
        raise ValueError("bad operand %r" % (x,))
    if x == "a":
        return 0xC0, None
    if x == "d":
        return 0xC1, None
    if x.startswith("side") and x[4:].isdigit():
        return 0x40 | int(x[4:]), None
    if x[0] == "t" and x[1:].isdigit():
        return 0x00 | int(x[1:]), None
    if x[0] == "s" and x[1:].isdigit():
        return 0x80 | int(x[1:]), None
    raise ValueError("bad operand %r" % (x,))


def make_chain(steps, outputs, rowsum_side=None):
    """Builds the fo_chain for `steps` and `outputs`; returns (chain, keepalive)."""
    steps = list(steps)
    outputs = [outputs] if isinstance(outputs, (str, float, int)) else list(outputs)
    if len(steps) > 255 or len(outputs) > FO_MAX_OUT:
        raise ValueError("chain too long")
    ops = (fo_op * max(1, len(steps)))()
    for i, st in enumerate(steps):
        name, dst, srcs = st[0], st[1], st[2:]
        if name not in OPCODES:
            raise ValueError("unknown op %r" % (name,))
        if len(srcs) != ARITY[name]:
            raise ValueError("%s takes %d operands" % (name, ARITY[name]))
        if not (isinstance(dst, str) and dst[0] == "t" and dst[1:].isdigit()):
            raise ValueError("dst must be a temporary, got %r" % (dst,))
        ops[i].opcode = OPCODES[name]
        ops[i].dst = int(dst[1:]) & 0xff
        imm = None
        enc = []
        for s in srcs:
            b, im = _operand(s, rowsum_side=rowsum_side)
            if im is not None:
                if imm is not None and imm != im:
                    raise ValueError("a step can carry one immediate value")
                imm = im
            enc.append(b)
        enc += [0] * (3 - len(enc))
        ops[i].a, ops[i].b, ops[i].c = enc
        ops[i].imm = imm if imm is not None else 0.0
    ch = fo_chain()
    ch.n_ops = len(steps)
    ch.n_out = len(outputs)
    ch.ops = C.cast(ops, C.POINTER(fo_op))
    for k, o in enumerate(outputs):
        ch.out[k] = _operand(o, allow_imm=False, rowsum_side=rowsum_side)[0]
    return ch, ops


class CSR:
    """A CSR matrix held in device tensors (int32 rowptr / colidx, float64 vals)."""

    def __init__(self, rows, cols, rowptr, colidx, vals):
        self.rows, self.cols = int(rows), int(cols)
        self.rowptr, self.colidx, self.vals = rowptr, colidx, vals
        assert rowptr.dtype == torch.int32 and colidx.dtype == torch.int32
        assert vals.dtype == torch.float64
        assert rowptr.numel() == self.rows + 1 and colidx.numel() == vals.numel()
        self.nnz = int(vals.numel())

    @property
    def device(self):
        return self.vals.device

    def as_struct(self):
        s = fo_csr()
        s.rows, s.cols, s.nnz = self.rows, self.cols, self.nnz
        s.rowptr, s.colidx, s.vals = self.rowptr.data_ptr(), self.colidx.data_ptr(), self.vals.data_ptr()
        return s


def _dense_struct(t, column=False):
    """fo_dense of a float64 tensor.  2-D: rows must be contiguous (stride(1) == 1).
    1-D: a row vector (1 x n, contiguous), or with column=True a column vector
    (n x 1) whose stride becomes the leading dimension."""
    assert t.dtype == torch.float64, "float64 only"
    d = fo_dense()
    d.data = t.data_ptr()
    if t.dim() == 1 and column:
        d.rows, d.cols = t.numel(), 1
        d.ld = max(int(t.stride(0)), 1) if t.numel() > 1 else 1
    elif t.dim() == 1:
        assert t.numel() <= 1 or t.stride(0) == 1, "row vectors must be contiguous"
        d.rows, d.cols = 1, t.numel()
        d.ld = max(t.numel(), 1)
    else:
        assert t.dim() == 2
        r, c = t.shape
        assert t.numel() == 0 or c == 1 or t.stride(1) == 1, "rows must be contiguous"
        d.rows, d.cols = r, c
        d.ld = max(int(t.stride(0)) if r > 1 else c, c, 1)
    return d


def _mat(X):
    m = fo_mat()
    if isinstance(X, CSR):
        m.kind = 1
        m.csr = X.as_struct()
    else:
        m.kind = 0
        m.dense = _dense_struct(X)
    return m


def _sides(sides, rows, cols):
    """fo_side array for [(access, tensor or CSR), ...].  A CSR side (access "cell") is
    passed through the struct's `sparse` pointer; the structs it points to hang off the
    returned array so that they live as long as it does."""
    arr = (fo_side * max(1, len(sides)))()
    arr._keep = []
    for k, (access, t) in enumerate(sides):
        acc = ACCESS[access]
        if isinstance(t, CSR):
            assert acc == 0, "a CSR side is read at (row, column)"
            st = t.as_struct()
            arr._keep.append(st)
            arr[k].sparse = C.addressof(st)
            arr[k].access = acc
            continue
        if acc == 0:
            arr[k].m = _dense_struct(t)
        elif acc == 1:
            assert t.dim() == 1 or (t.dim() == 2 and t.shape[1] == 1)
            t1 = t if t.dim() == 1 else t[:, 0]
            arr[k].m = _dense_struct(t1, column=True)
        else:
            assert t.dim() == 1 or (t.dim() == 2 and t.shape[0] == 1)
            t1 = t if t.dim() == 1 else t[0]
            arr[k].m = _dense_struct(t1)
        arr[k].access = acc
    return arr


def _scalars(scalars):
    arr = (C.c_double * max(1, len(scalars)))(*[float(s) for s in scalars])
    return arr


def _stream(device):
    return C.c_void_p(torch.cuda.current_stream(device).cuda_stream)


# ------------------------------------------------------------------ workspace
_ws = {}


def workspace(device, nbytes):
    """A cached, initialised scratch buffer of at least nbytes on `device`."""
    if device.type != "cuda":
        raise RuntimeError("fused operators need CUDA tensors (no CPU path)")
    # one buffer per (device, stream): calls that may overlap on the GPU must not share scratch
    stream = torch.cuda.current_stream(device)
    key = (device.index if device.index is not None else torch.cuda.current_device(), stream.cuda_stream)
    buf = _ws.get(key)
    if buf is None or buf.numel() < nbytes:
        if buf is not None:
            buf.record_stream(stream)         # kernels already queued may still use the old one
        size = max(int(nbytes), 1 << 20)
        buf = torch.empty(size, dtype=torch.uint8, device=device)
        assert buf.data_ptr() % 256 == 0
        _check(load_library().fo_workspace_init(C.c_void_p(buf.data_ptr()), buf.numel(),
                                                _stream(device)), "fo_workspace_init")
        _ws[key] = buf
    return buf


def force_interpreter(on):
    """Route every Cell / MAgg chain through the interpreter (True) or let known
    chains use their compile-time specialisation (False).  Returns the old setting."""
    return bool(load_library().fo_set_force_interpreter(1 if on else 0))


def tune(name, value=None):
    """Sets (or with value None clears) a measurement knob of the library; see fo_tune."""
    _check(load_library().fo_tune(name.encode(), None if value is None else str(value).encode()), "fo_tune")


def jit_prepare_call(steps, outputs, X, sides=(), n_scalars=0, agg="full", magg=False):
    """Compiles and caches exactly the kernel that fused_cell / fused_magg would run for
    these arguments (dense X)."""
    ch, keep = make_chain(steps, outputs)
    sides = list(sides)
    m = _mat(X)
    sarr = _sides(sides, X.shape[0], X.shape[1])
    _check(load_library().fo_jit_prepare_call(C.byref(ch), C.byref(m), sarr, len(sides), n_scalars,
                                              CELL_AGG[agg], 1 if magg else 0), "fo_jit_prepare_call")


def cell_stamps(device=None):
    """(start, scan done, partials published, result written) of the last streaming Cell /
    MAgg call made with the knob cell.stamps = 1, in ns of the GPU's global timer."""
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    buf = workspace(device, 16384)
    ns = (C.c_ulonglong * 4)()
    _check(load_library().fo_cell_stamps(C.c_void_p(buf.data_ptr()), _stream(device), ns), "fo_cell_stamps")
    return tuple(int(x) for x in ns)


JIT_OFF, JIT_FIRST_USE, JIT_PREPARED = 0, 1, 2


def set_jit(mode):
    """Mode of the run-time specialisation of Cell / MAgg chains: JIT_OFF (False),
    JIT_FIRST_USE (True; compile a chain when it is first seen), JIT_PREPARED (only
    kernels made by jit_prepare or earlier calls; nothing is compiled inside a
    call).  Returns the old mode."""
    return int(load_library().fo_set_jit(int(mode)))


def jit_prepare(steps, outputs, n_sides=0, n_scalars=0, store=False):
    """Compiles and caches the run-time specialised kernel of a chain for the current device."""
    ch, keep = make_chain(steps, outputs)
    _check(load_library().fo_jit_prepare(C.byref(ch), n_sides, n_scalars, 1 if store else 0), "fo_jit_prepare")


def jit_stats():
    """(usable, kernels compiled, specialised launches, failed compilations)."""
    a, b, c = C.c_int(0), C.c_int(0), C.c_int(0)
    ok = load_library().fo_jit_stats(C.byref(a), C.byref(b), C.byref(c))
    return bool(ok), a.value, b.value, c.value


def jit_compile_check(steps, outputs, n_sides=0, n_scalars=0, store=False):
    """Generates and compiles a specialised kernel of a Cell chain without running it (no GPU
    needed).  store: False / True the flat stream (aggregating / no_agg), 2 .. 8 the other
    skeletons (see fo_jit_compile_check).  Returns (status, compiler log)."""
    ch, keep = make_chain(steps, outputs)
    log = C.create_string_buffer(1 << 16)
    rc = load_library().fo_jit_compile_check(C.byref(ch), n_sides, n_scalars, int(store), log, len(log))
    return rc, log.value.decode(errors="replace")


def jit_compile_check_outer(steps, output, n_sides=0, n_scalars=0, kernel=0):
    """Generates and compiles a specialised Outer kernel for a chain (no GPU needed).
    Returns (status, compiler log)."""
    ch, keep = make_chain(steps, output)
    log = C.create_string_buffer(1 << 16)
    rc = load_library().fo_jit_compile_check_outer(C.byref(ch), n_sides, n_scalars, int(kernel), log, len(log))
    return rc, log.value.decode(errors="replace")


def jit_compile_check_row(steps, output, n_sides=0, n_scalars=0, kernel=0):
    """Generates and compiles a specialised Row kernel for a chain (no GPU needed).
    Returns (status, compiler log)."""
    ch, keep = make_chain(steps, output)
    log = C.create_string_buffer(1 << 16)
    rc = load_library().fo_jit_compile_check_row(C.byref(ch), n_sides, n_scalars, int(kernel), log, len(log))
    return rc, log.value.decode(errors="replace")


def chain_describe(steps, outputs, use="cell", n_sides=0, scalars=(), k=0):
    """The k-th result of a chain as an expression over its inputs (host only)."""
    ch, keep = make_chain(steps, outputs)
    text = C.create_string_buffer(8192)
    _check(load_library().fo_chain_describe(C.byref(ch), {"cell": 0, "row": 1, "outer": 2}[use], n_sides,
                                            _scalars(scalars), len(scalars), k, text, len(text)),
           "fo_chain_describe")
    return text.value.decode()


def probe_l2_gather(V, idx, out=None):
    """Gathers the rows idx (int32) of the dense matrix V once; returns the bytes moved.
    Time it with events on the current stream."""
    lib = load_library()
    assert V.dtype == torch.float64 and V.dim() == 2 and idx.dtype == torch.int32 and idx.is_contiguous()
    if out is None:
        out = torch.empty(lib.fo_probe_out_len(), dtype=torch.float64, device=V.device)
    vs = _dense_struct(V)
    _check(lib.fo_probe_l2_gather(C.byref(vs), C.c_void_p(idx.data_ptr()), idx.numel(),
                                  C.c_void_p(out.data_ptr()), _stream(V.device)), "fo_probe_l2_gather")
    return idx.numel() * V.shape[1] * 8


def probe_bulk_gather(V, idx, out=None):
    """The same gather through the bulk-copy engine; returns the bytes moved.  After a
    synchronise, out[probe_bulk_flag_index(V.device)] is 0.0 unless a bounded wait ran out."""
    lib = load_library()
    assert V.dtype == torch.float64 and V.dim() == 2 and idx.dtype == torch.int32 and idx.is_contiguous()
    if out is None:
        out = torch.empty(lib.fo_probe_out_len(), dtype=torch.float64, device=V.device)
    vs = _dense_struct(V)
    _check(lib.fo_probe_bulk_gather(C.byref(vs), C.c_void_p(idx.data_ptr()), idx.numel(),
                                    C.c_void_p(out.data_ptr()), _stream(V.device)), "fo_probe_bulk_gather")
    return idx.numel() * V.shape[1] * 8


def probe_bulk_flag_index():
    return int(load_library().fo_probe_out_len()) // 8


def probe_fp64_fma(iters, out):
    """Runs 8 * iters multiply-adds per launched thread; returns the flop count."""
    lib = load_library()
    _check(lib.fo_probe_fp64_fma(int(iters), C.c_void_p(out.data_ptr()), _stream(out.device)),
           "fo_probe_fp64_fma")
    return 16 * int(iters) * lib.fo_probe_out_len()


def probe_out_len():
    return int(load_library().fo_probe_out_len())


def device_status(device=None):
    """Synchronises and returns the workspace's device-side status (0 = ok)."""
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    buf = workspace(device, 16384)
    st = C.c_int(0)
    _check(load_library().fo_query_device_status(C.c_void_p(buf.data_ptr()), _stream(device),
                                                 C.byref(st)), "fo_query_device_status")
    return st.value


# ------------------------------------------------------------------ the four calls
def fused_cell(steps, output, X, sides=(), scalars=(), agg="full", out=None, out_nnz=None):
    """Cell template.  Returns a tensor: scalar (1,), (rows,), (cols,) or (rows, cols).
    out_nnz: an int64 tensor of one element that receives the number of non-zero values
    of a no_agg result."""
    lib = load_library()
    sides = list(sides)
    ch, keep = make_chain(steps, output)
    m = _mat(X)
    rows, cols = (X.rows, X.cols) if isinstance(X, CSR) else X.shape
    dev = X.device
    a = CELL_AGG[agg]
    if out is None:
        shape = {"full": (1,), "row": (rows,), "col": (cols,),
                 "none": (X.nnz,) if isinstance(X, CSR) else (rows, cols)}[agg]
        out = torch.empty(shape, dtype=torch.float64, device=dev)
    need = lib.fused_cell_workspace_bytes(C.byref(m), a)
    ws = workspace(dev, max(need, 16384))
    sarr, sc = _sides(sides, rows, cols), _scalars(scalars)
    if out_nnz is not None:
        assert out_nnz.dtype == torch.int64 and out_nnz.numel() == 1 and out_nnz.device == dev
    _check(lib.fused_cell(C.byref(ch), C.byref(m), sarr, len(sides), sc, len(scalars), a,
                          C.c_void_p(out.data_ptr()), C.c_void_p(out_nnz.data_ptr()) if out_nnz is not None else None,
                          C.c_void_p(ws.data_ptr()), ws.numel(), _stream(dev)), "fused_cell")
    return out


def fused_cell_static(steps, output, X, sides=(), scalars=(), agg="full", out=None):
    """fused_cell for callers that may not allocate device memory for scratch: the
    library's built-in 1 MiB scratch array is used instead of a workspace tensor.
    Raises FusedOpsError(FO_ERR_STATIC_LIMIT) if the call would need more.  Calls
    that can overlap on the GPU must not use it concurrently.  Such callers pass
    `out` themselves; it is only created here as a convenience for tests."""
    lib = load_library()
    sides = list(sides)
    ch, keep = make_chain(steps, output)
    m = _mat(X)
    rows, cols = X.shape
    dev = X.device
    a = CELL_AGG[agg]
    if out is None:
        shape = {"full": (1,), "row": (rows,), "col": (cols,), "none": (rows, cols)}[agg]
        out = torch.empty(shape, dtype=torch.float64, device=dev)
    sarr, sc = _sides(sides, rows, cols), _scalars(scalars)
    _check(lib.fused_cell_static(C.byref(ch), C.byref(m), sarr, len(sides), sc, len(scalars), a,
                                 C.c_void_p(out.data_ptr()), _stream(dev)), "fused_cell_static")
    return out


def fused_magg(steps, outputs, X, sides=(), scalars=(), out=None):
    """MAgg template.  Returns a (k,) tensor, one full sum per output."""
    lib = load_library()
    sides = list(sides)
    outputs = list(outputs)
    ch, keep = make_chain(steps, outputs)
    m = _mat(X)
    rows, cols = (X.rows, X.cols) if isinstance(X, CSR) else X.shape
    dev = X.device
    if out is None:
        out = torch.empty(len(outputs), dtype=torch.float64, device=dev)
    need = lib.fused_magg_workspace_bytes(C.byref(m), len(outputs))
    ws = workspace(dev, max(need, 16384))
    sarr, sc = _sides(sides, rows, cols), _scalars(scalars)
    _check(lib.fused_magg(C.byref(ch), C.byref(m), sarr, len(sides), sc, len(scalars),
                          C.c_void_p(out.data_ptr()), C.c_void_p(ws.data_ptr()), ws.numel(),
                          _stream(dev)), "fused_magg")
    return out


def fused_row(steps, output, X, v, sides=(), scalars=(), agg="col_t", out=None):
    """Row template.  Returns (cols,), (rows,), (1,) or, for agg "none", (rows, cols) /
    (nnz,) for a dense / CSR main input."""
    lib = load_library()
    sides = list(sides)
    ch, keep = make_chain(steps, output)
    m = _mat(X)
    rows, cols = (X.rows, X.cols) if isinstance(X, CSR) else X.shape
    dev = X.device
    a = ROW_AGG[agg]
    assert v.dtype == torch.float64 and v.numel() == cols and (v.numel() <= 1 or v.stride(-1) == 1)
    if out is None:
        shape = {"col_t": (cols,), "col": (cols,), "row": (rows,), "full": (1,),
                 "none": (X.nnz,) if isinstance(X, CSR) else (rows, cols)}[agg]
        out = torch.empty(shape, dtype=torch.float64, device=dev)
    need = lib.fused_row_workspace_bytes(C.byref(m), a)
    ws = workspace(dev, max(need, 16384))
    sarr, sc = _sides(sides, rows, cols), _scalars(scalars)
    _check(lib.fused_row(C.byref(ch), C.byref(m), C.c_void_p(v.data_ptr()), sarr, len(sides), sc,
                         len(scalars), a, C.c_void_p(out.data_ptr()), C.c_void_p(ws.data_ptr()),
                         ws.numel(), _stream(dev)), "fused_row")
    return out


def fused_row_b1(pre, pre_out, post, post_out, X, B, sides=(), scalars=(), agg="col_t", out=None):
    """Row template with a matrix-valued row intermediate (side matrix B, n x k).
    `pre` may be None; in `post` the operand "rowsum" names the row sum of `pre`.
    Returns (cols, k) for agg "col_t", (rows, k) for "none"."""
    lib = load_library()
    sides = list(sides)
    post_ch, keep2 = make_chain(post, post_out, rowsum_side=len(sides) if pre is not None else None)
    pre_ref = None
    if pre is not None:
        pre_ch, keep1 = make_chain(pre, pre_out)
        pre_ref = C.byref(pre_ch)
    m = _mat(X)
    rows, cols = (X.rows, X.cols) if isinstance(X, CSR) else X.shape
    dev = X.device
    a = ROW_B1_AGG[agg]
    assert B.dtype == torch.float64 and B.dim() == 2
    k = B.shape[1]
    bs = _dense_struct(B)
    if out is None:
        out = torch.empty((cols, k) if agg == "col_t" else (rows, k), dtype=torch.float64, device=dev)
    need = lib.fused_row_b1_workspace_bytes(C.byref(m), k, a)
    ws = workspace(dev, max(need, 16384))
    sarr, sc = _sides(sides, rows, k), _scalars(scalars)
    _check(lib.fused_row_b1(pre_ref, C.byref(post_ch), C.byref(m), C.byref(bs), sarr, len(sides), sc,
                            len(scalars), a, C.c_void_p(out.data_ptr()), C.c_void_p(ws.data_ptr()),
                            ws.numel(), _stream(dev)), "fused_row_b1")
    return out


def fused_outer(steps, output, X, U, V, scalars=(), agg="full", out=None, sides=(), out_nnz=None):
    """Outer template over the stored cells of the CSR matrix X.  sides: dense side inputs
    [("cell" | "row" | "col", tensor), ...] read at the stored cell; out_nnz as in fused_cell."""
    lib = load_library()
    ch, keep = make_chain(steps, output)
    xs = X.as_struct()
    us, vs = _dense_struct(U), _dense_struct(V)
    dev = X.device
    a = OUTER_AGG[agg]
    rank = U.shape[1]
    if out is None:
        shape = {"full": (1,), "none": (X.nnz,), "right": (X.rows, rank), "left": (X.cols, rank)}[agg]
        out = torch.empty(shape, dtype=torch.float64, device=dev)
    need = lib.fused_outer_workspace_bytes(C.byref(xs), rank, a)
    ws = workspace(dev, max(need, 16384))
    sc = _scalars(scalars)
    sides = list(sides)
    sarr = _sides(sides, X.rows, X.cols)
    if out_nnz is not None:
        assert out_nnz.dtype == torch.int64 and out_nnz.numel() == 1 and out_nnz.device == dev
    _check(lib.fused_outer(C.byref(ch), C.byref(xs), C.byref(us), C.byref(vs), sarr, len(sides), sc,
                           len(scalars), a, C.c_void_p(out.data_ptr()),
                           C.c_void_p(out_nnz.data_ptr()) if out_nnz is not None else None,
                           C.c_void_p(ws.data_ptr()), ws.numel(), _stream(dev)), "fused_outer")
    return out
