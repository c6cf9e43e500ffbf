// Cell and MAgg templates over a dense main input (Table 1; Section 2.2,
// cell-wise listing; Section 5.2 "Cell Operations", "Multi-Aggregate
// Operations").  One scan of the inputs: every thread evaluates the operator
// chain on four cells at a time in registers and keeps running sums; CTAs
// publish partial sums and the last CTA to finish adds them in index order.
//
// Three kernels:
//   cell_flat_kernel  contiguous inputs, cell-shaped sides only: the matrix is
//                     one flat array streamed with 128-bit loads (full_agg,
//                     MAgg, no_agg);
//   cell_rows_kernel  general case (leading dimensions, row / column vector
//                     sides): a warp per row (no_agg, row_agg, full_agg, MAgg);
//   cell_cols_kernel  col_agg: a thread per column pair, a CTA per panel of rows.
#include <stdlib.h>

#include <atomic>

#include "cell_tiles.cuh"
#include "jit.h"
#include "cell_csr.h"
#include "spec.cuh"

namespace fo {

namespace {

// Non-zero entries of an elementwise result: integer counts, so the total does not
// depend on the order in which the CTAs add theirs.
__global__ void __launch_bounds__(kThreads)
count_nonzero_kernel(const double *__restrict__ values, long long n, unsigned long long *out_nnz)
{
    __shared__ unsigned int s_count;
    if (threadIdx.x == 0) s_count = 0u;
    __syncthreads();
    unsigned int mine = 0;
    for (long long i = blockIdx.x * (long long)kThreads + threadIdx.x; i < n; i += (long long)gridDim.x * kThreads)
        mine += __ldcg(values + i) != 0.0 ? 1u : 0u;
    mine = __reduce_add_sync(0xffffffffu, mine);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&s_count, mine);
    __syncthreads();
    if (threadIdx.x == 0 && s_count) atomicAdd(out_nnz, (unsigned long long)s_count);
}

__global__ void fill_zero_kernel(double *out, long long n)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
         i += (long long)gridDim.x * blockDim.x)
        out[i] = 0.0;
}

// ------------------------------------------------------------------ host
bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

// CTAs per SM of the streaming kernels (the knob cell.ctas_per_sm, 1..8, overrides the
// default; results do not depend on it beyond the order of the per-CTA partial sums).
int cell_ctas_per_sm()
{
    const int v = tune_int("cell.ctas_per_sm", 3);    // measured: 2-3 is best for 10-100 MB inputs, larger inputs do not care
    return (v >= 1 && v <= 8) ? v : 3;
}

// Grid of a streaming kernel: every CTA gets work, at most `cap` CTAs.
int stream_grid(long long units, int sms)
{
    const long long cap = (long long)(sms > 0 ? sms : 148) * cell_ctas_per_sm();
    long long g = units < cap ? units : cap;
    if (g > kMaxPartials) g = kMaxPartials;
    if (g < 1) g = 1;
    return (int)g;
}

// Row panels of the column-aggregation kernel: enough CTAs to fill the GPU, at
// least 32 rows per panel, one ticket per column tile.
// Column pairs a CTA covers: 256, or fewer for narrow matrices (a power of two).
int col_cx(long long cols)
{
    // column pairs per tile: all of them in one tile up to 512 columns, else as many
    // equal tiles of at most 256 pairs as it takes - no ragged last tile, so that for,
    // say, 100 columns 250 of the 256 threads have a column pair (50 pairs x 5 row lanes)
    const long long half = (cols + 1) / 2;
    const long long tiles = (half + 255) / 256;
    long long cx = tiles > 0 ? (half + tiles - 1) / tiles : 1;
    if (cx < 1) cx = 1;
    return (int)cx;
}

int col_panels(long long rows, long long cols)
{
    const long long tiles = (cols + 2 * col_cx(cols) - 1) / (2 * col_cx(cols));
    if (tiles > kMaxGroups) return 1;
    long long p = (148 * 8 + tiles - 1) / tiles;
    const long long maxp = (rows + 31) / 32;
    if (p > maxp) p = maxp;
    if (p > kMaxPartials) p = kMaxPartials;
    if (p < 1) p = 1;
    return (int)p;
}

size_t cell_ws_bytes(long long rows, long long cols, int agg, int n_out)
{
    switch (agg) {
        case FO_CELL_FULL_AGG: return sizeof(WsHead) + (size_t)kMaxPartials * n_out * sizeof(double);
        case FO_CELL_COL_AGG:
            return sizeof(WsHead) + (size_t)col_panels(rows, cols) * (size_t)cols * sizeof(double);
        default: return sizeof(WsHead);
    }
}

int check_dense(const fo_dense &d)
{
    if (d.rows < 0 || d.cols < 0 || d.ld < d.cols) return FO_ERR_SHAPE;
    if (d.rows > 0 && d.cols > 0 && !d.data) return FO_ERR_NULL;
    return FO_OK;
}

template <class EVAL, int NOUT>
cudaError_t launch_cell(const DevChain &ch, const CellParams &p, int agg, bool flat, bool aligned,
                        int grid, cudaStream_t st)
{
    if (agg == FO_CELL_COL_AGG) {
        if constexpr (NOUT == 1) {
            // row panels: as many as fill every SM exactly once with the CTAs this kernel
            // can keep resident (a second, partly filled wave would cost up to a wave's time);
            // p.panels, which sized the workspace, is the upper bound
            const long long tiles = (p.cols + 2 * p.cx - 1) / (2 * p.cx);
            CellParams q = p;
            int nb = 0;
            const cudaError_t oe = aligned
                ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, cell_cols_kernel<EVAL, true>, kThreads, 0)
                : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, cell_cols_kernel<EVAL, false>, kThreads, 0);
            const int sms = sm_count();
            if (oe == cudaSuccess && nb > 0 && sms > 0) {
                long long want = ((long long)sms * nb) / tiles;
                if (want < 1) want = 1;
                if (want < q.panels) q.panels = (int)want;
            }
            const dim3 g((unsigned)tiles, (unsigned)q.panels);
            if (aligned) cell_cols_kernel<EVAL, true><<<g, kThreads, 0, st>>>(ch, q);
            else cell_cols_kernel<EVAL, false><<<g, kThreads, 0, st>>>(ch, q);
        }
    } else if (flat) {
        if (agg == FO_CELL_NO_AGG) {
            if constexpr (NOUT == 1) cell_flat_kernel<EVAL, 1, true><<<grid, kThreads, 0, st>>>(ch, p);
        } else {
            cell_flat_kernel<EVAL, NOUT, false><<<grid, kThreads, 0, st>>>(ch, p);
        }
    } else if (agg == FO_CELL_FULL_AGG) {
        if (aligned) cell_rows_kernel<EVAL, NOUT, kAggFull, true><<<grid, kThreads, 0, st>>>(ch, p);
        else cell_rows_kernel<EVAL, NOUT, kAggFull, false><<<grid, kThreads, 0, st>>>(ch, p);
    } else if constexpr (NOUT == 1) {
        if (agg == FO_CELL_ROW_AGG) {
            if (aligned) cell_rows_kernel<EVAL, 1, kAggRow, true><<<grid, kThreads, 0, st>>>(ch, p);
            else cell_rows_kernel<EVAL, 1, kAggRow, false><<<grid, kThreads, 0, st>>>(ch, p);
        } else {
            if (aligned) cell_rows_kernel<EVAL, 1, kAggNone, true><<<grid, kThreads, 0, st>>>(ch, p);
            else cell_rows_kernel<EVAL, 1, kAggNone, false><<<grid, kThreads, 0, st>>>(ch, p);
        }
    }
    return cudaGetLastError();
}

template <int NR>
cudaError_t launch_cell_interp(const DevChain &ch, const CellParams &p, int agg, bool flat,
                               bool aligned, int grid, cudaStream_t st)
{
    if (ch.n_out == 1) return launch_cell<EvalInterp<NR>, 1>(ch, p, agg, flat, aligned, grid, st);
    if (ch.n_out <= 4) return launch_cell<EvalInterp<NR>, 4>(ch, p, agg, flat, aligned, grid, st);
    return launch_cell<EvalInterp<NR>, 8>(ch, p, agg, flat, aligned, grid, st);
}

template <int ID>
cudaError_t launch_cell_spec(const DevChain &ch, const CellParams &p, int agg, bool flat,
                             bool aligned, int grid, cudaStream_t st)
{
    return launch_cell<EvalSpec<ID>, SpecFn<ID>::kOut>(ch, p, agg, flat, aligned, grid, st);
}

// The run-time specialised kernel of a chain without a built-in form: the same three
// skeletons (flat stream, rows, columns) with the chain written out as straight-line
// code.  FO_OK if launched (launch = false: made ready), kJitUnavailable if the caller
// should interpret instead.
int launch_cell_jit(const DevChain &ch, const CellParams &p, int agg, bool flat, bool aligned, int grid,
                    cudaStream_t st, bool may_compile, bool launch)
{
    if (agg == FO_CELL_COL_AGG) {
        if (ch.n_out != 1) return kJitUnavailable;
        const JitSpec sp = {kJitCols, aligned ? 1 : 0, 0, 0};
        const int rc = jit_launch(sp, ch, &p, 1, 1, st, may_compile, false);
        if (rc != FO_OK || !launch) return rc;
        // row panels as for the ahead-of-time kernels: one full wave of resident CTAs
        const long long tiles = (p.cols + 2 * p.cx - 1) / (2 * p.cx);
        CellParams q = p;
        const int nb = jit_occupancy(sp, ch), sms = sm_count();
        if (nb > 0 && sms > 0) {
            long long want = ((long long)sms * nb) / tiles;
            if (want < 1) want = 1;
            if (want < q.panels) q.panels = (int)want;
        }
        return jit_launch(sp, ch, &q, (unsigned)tiles, (unsigned)q.panels, st, false, true);
    }
    JitSpec sp;
    if (flat) sp = JitSpec{kJitFlat, agg == FO_CELL_NO_AGG ? 1 : 0, 0, 0};
    else sp = JitSpec{kJitRows, agg == FO_CELL_FULL_AGG ? kAggFull : agg == FO_CELL_ROW_AGG ? kAggRow : kAggNone,
                      aligned ? 1 : 0, 0};
    if (sp.kind == kJitRows && agg != FO_CELL_FULL_AGG && ch.n_out != 1) return kJitUnavailable;
    return jit_launch(sp, ch, &p, (unsigned)grid, 1, st, may_compile, launch);
}

// Test / benchmark switch: run every chain through the interpreter.
bool g_force_interpreter = false;

// Common body of fused_cell and fused_magg.
int run_cell(const fo_chain *chain, const fo_mat *X, const fo_side *sides, int n_sides,
             const double *scalars, int n_scalars, int agg, bool magg, double *out, long long *out_nnz,
             void *ws, size_t ws_bytes, void *stream, bool may_compile, bool prepare_only = false)
{
    if (!chain || !X || (!out && !prepare_only)) return FO_ERR_NULL;
    if (n_sides > 0 && !sides) return FO_ERR_NULL;
    if (agg < FO_CELL_NO_AGG || agg > FO_CELL_FULL_AGG) return FO_ERR_UNSUPPORTED;
    if (out_nnz && agg != FO_CELL_NO_AGG) return FO_ERR_UNSUPPORTED;      // a count needs an elementwise result
    if (out_nnz) {
        // the elementwise result first, then one more pass over it for the count
        const int rc = run_cell(chain, X, sides, n_sides, scalars, n_scalars, agg, magg, out, nullptr, ws,
                                ws_bytes, stream, may_compile);
        if (rc != FO_OK) return rc;
        const long long n = X->kind == FO_CSR ? X->csr.nnz : X->dense.rows * X->dense.cols;
        const cudaError_t e = launch_count_nonzero(out, n, out_nnz, (cudaStream_t)stream);
        return e == cudaSuccess ? FO_OK : cuda_fail(e);
    }
    if (X->kind == FO_CSR)
        return run_cell_csr(chain, X->csr, sides, n_sides, scalars, n_scalars, agg, magg, out, ws, ws_bytes,
                            stream, may_compile);
    if (X->kind != FO_DENSE) return FO_ERR_SHAPE;
    const fo_dense &xd = X->dense;
    int rc = check_dense(xd);
    if (rc != FO_OK) return rc;

    DevChain ch;
    rc = translate_chain(chain, kUseCell, n_sides, scalars, n_scalars, 1, magg ? FO_MAX_OUT : 1, &ch);
    if (rc != FO_OK) return rc;

    CellParams p;
    memset(&p, 0, sizeof(p));
    p.X = xd.data; p.rows = xd.rows; p.cols = xd.cols; p.ldx = xd.ld;
    p.sides.n = n_sides;
    bool flat = (xd.ld == xd.cols) && aligned16(xd.data);
    bool aligned = aligned16(xd.data) && (xd.ld % 2 == 0);
    for (int k = 0; k < n_sides; ++k) {
        const fo_side &s = sides[k];
        if (s.sparse) return FO_ERR_UNSUPPORTED;       // sparse sides: CSR main input of Cell / MAgg only
        rc = check_dense(s.m);
        if (rc != FO_OK) return rc;
        switch (s.access) {
            case FO_AT_CELL:
                if (s.m.rows != xd.rows || s.m.cols != xd.cols) return FO_ERR_SHAPE;
                if ((ch.side_used >> k) & 1u) {
                    flat = flat && s.m.ld == s.m.cols && aligned16(s.m.data);
                    aligned = aligned && aligned16(s.m.data) && (s.m.ld % 2 == 0);
                }
                break;
            case FO_AT_ROW:
                if (s.m.rows != xd.rows || s.m.cols != 1) return FO_ERR_SHAPE;
                if ((ch.side_used >> k) & 1u) flat = false;
                break;
            case FO_AT_COL:
                if (s.m.rows != 1 || s.m.cols != xd.cols) return FO_ERR_SHAPE;
                if ((ch.side_used >> k) & 1u) flat = false;
                break;
            default: return FO_ERR_SHAPE;
        }
        p.sides.s[k].data = s.m.data;
        p.sides.s[k].ld = s.m.ld;
        p.sides.s[k].access = s.access;
    }
    if (agg == FO_CELL_NO_AGG) flat = flat && aligned16(out);
    if (agg == FO_CELL_ROW_AGG || agg == FO_CELL_COL_AGG) flat = false;

    const size_t need = cell_ws_bytes(xd.rows, xd.cols, agg, ch.n_out);
    rc = prepare_only ? FO_OK : check_workspace(ws, ws_bytes, need);
    if (rc != FO_OK) return rc;
    p.head = (WsHead *)ws;
    p.partials = (double *)((char *)ws + sizeof(WsHead));
    p.out = out;
    p.stamps = tune_int("cell.stamps", 0) ? reinterpret_cast<unsigned long long *>(&p.head->pad[0]) : nullptr;

    cudaStream_t st = (cudaStream_t)stream;
    const long long ncells = xd.rows * xd.cols;
    if (ncells == 0 && prepare_only) return FO_OK;
    if (ncells == 0) {      // nothing to scan: the aggregates are empty sums
        const long long nout = agg == FO_CELL_FULL_AGG ? ch.n_out
                             : agg == FO_CELL_ROW_AGG ? xd.rows
                             : agg == FO_CELL_COL_AGG ? xd.cols : 0;
        if (nout > 0) fill_zero_kernel<<<(unsigned)((nout + 255) / 256 > 1024 ? 1024 : (nout + 255) / 256),
                                         256, 0, st>>>(out, nout);
        const cudaError_t e = cudaGetLastError();
        return e == cudaSuccess ? FO_OK : cuda_fail(e);
    }

    const int sms = sm_count();
    if (sms <= 0) return cuda_fail(cudaErrorNoDevice);
    int grid;
    if (agg == FO_CELL_COL_AGG) {
        p.panels = col_panels(xd.rows, xd.cols);
        p.cx = col_cx(xd.cols);
        grid = 0;
    } else if (flat) {
        grid = stream_grid((ncells + 1023) >> 10, sms);
    } else {
        grid = stream_grid((xd.rows + 7) / 8, sms);
    }

    cudaError_t e;
    const int spec = g_force_interpreter ? kSpecNone : match_cell_spec(ch);
    if (prepare_only && spec != kSpecNone) return FO_OK;       // built-in straight-line code: nothing to make ready
    switch (spec) {
        case kSpecMul2: e = launch_cell_spec<kSpecMul2>(ch, p, agg, flat, aligned, grid, st); break;
        case kSpecMul3: e = launch_cell_spec<kSpecMul3>(ch, p, agg, flat, aligned, grid, st); break;
        case kSpecSq: e = launch_cell_spec<kSpecSq>(ch, p, agg, flat, aligned, grid, st); break;
        case kSpecMagg2: e = launch_cell_spec<kSpecMagg2>(ch, p, agg, flat, aligned, grid, st); break;
        case kSpecMagg3: e = launch_cell_spec<kSpecMagg3>(ch, p, agg, flat, aligned, grid, st); break;
        case kSpecScaledAdd: {
            DevChain c2 = ch;                     // the straight-line code reads its constant from slot 0
            c2.consts[0] = ch.consts[scaled_add_const(ch)];
            e = launch_cell_spec<kSpecScaledAdd>(c2, p, agg, flat, aligned, grid, st);
            break;
        }
        default:
            // no built-in specialisation: a kernel compiled for this chain at run time, else the interpreter
            if (!g_force_interpreter) {
                const bool compile_ok = prepare_only || (may_compile && jit_first_use());
                const int jrc = launch_cell_jit(ch, p, agg, flat, aligned, grid, st, compile_ok, !prepare_only);
                if (jrc == FO_OK) return FO_OK;
                if (jrc != kJitUnavailable) return jrc;
            }
            if (prepare_only) return jit_enabled() ? FO_ERR_CHAIN : FO_ERR_UNSUPPORTED;
            if (ch.n_regs <= 4) e = launch_cell_interp<4>(ch, p, agg, flat, aligned, grid, st);
            else if (ch.n_regs <= 8) e = launch_cell_interp<8>(ch, p, agg, flat, aligned, grid, st);
            else e = launch_cell_interp<kRegs>(ch, p, agg, flat, aligned, grid, st);
    }
    return e == cudaSuccess ? FO_OK : cuda_fail(e);
}

}  // namespace

bool force_interpreter() { return g_force_interpreter; }

cudaError_t launch_count_nonzero(const double *values, long long n, long long *out_nnz, cudaStream_t st)
{
    cudaError_t e = cudaMemsetAsync(out_nnz, 0, sizeof(long long), st);
    if (e != cudaSuccess || n <= 0) return e;
    long long grid = (n + 4 * kThreads - 1) / (4 * kThreads);
    const long long cap = (long long)(sm_count() > 0 ? sm_count() : 148) * 8;
    if (grid > cap) grid = cap;
    count_nonzero_kernel<<<(unsigned)grid, kThreads, 0, st>>>(values, n, (unsigned long long *)out_nnz);
    return cudaGetLastError();
}

}  // namespace fo

namespace fo {
namespace {

// Scratch of fused_cell_static: one array per GPU that loads the library, held
// until the process exits.  Zero-initialised at load, which is the state the
// ticket counters need; every call leaves them at zero again.
constexpr size_t kStaticWsBytes = 1u << 20;
static __device__ __align__(256) unsigned char g_static_ws[kStaticWsBytes];

// Device address of g_static_ws on the current device (NULL on failure).  In host
// code the symbol's name is only a handle: the address a kernel can use has to
// be asked for, once per device, with that device current.
void *static_ws_address()
{
    static std::atomic<void *> cached[64];       // zero-initialised; a slot is only ever set to one value
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= 64) {
        cuda_fail(e != cudaSuccess ? e : cudaErrorInvalidDevice);
        return nullptr;
    }
    void *ptr = cached[dev].load(std::memory_order_acquire);
    if (!ptr) {
        e = cudaGetSymbolAddress((void **)&ptr, g_static_ws);
        if (e != cudaSuccess) {
            cuda_fail(e);
            return nullptr;
        }
        cached[dev].store(ptr, std::memory_order_release);
    }
    return ptr;
}

}  // namespace
}  // namespace fo

extern "C" {

int fused_cell_static(const fo_chain *chain, const fo_mat *X, const fo_side *sides, int n_sides,
                      const double *scalars, int n_scalars, int agg, double *out, void *stream)
{
    if (!X) return FO_ERR_NULL;
    if (agg < FO_CELL_NO_AGG || agg > FO_CELL_FULL_AGG) return FO_ERR_UNSUPPORTED;
    if (X->kind != FO_DENSE) return (X->kind == FO_CSR) ? FO_ERR_UNSUPPORTED : FO_ERR_SHAPE;
    if (X->dense.rows < 0 || X->dense.cols < 0) return FO_ERR_SHAPE;
    const size_t need = fo::cell_ws_bytes(X->dense.rows, X->dense.cols, agg, 1);
    if (need > fo::kStaticWsBytes) return FO_ERR_STATIC_LIMIT;
    void *ws = fo::static_ws_address();
    if (!ws) return FO_ERR_CUDA;
    // never compiles or loads a kernel: a chain specialised earlier is reused, any other
    // one runs through the built-in code
    return fo::run_cell(chain, X, sides, n_sides, scalars, n_scalars, agg, false, out, nullptr, ws,
                        fo::kStaticWsBytes, stream, false);
}

size_t fused_cell_static_limit_bytes(void) { return fo::kStaticWsBytes; }

int fo_jit_prepare_call(const fo_chain *chain, const fo_mat *X, const fo_side *sides, int n_sides, int n_scalars,
                        int agg, int magg)
{
    if (n_scalars < 0 || n_scalars > FO_MAX_SCALARS) return FO_ERR_UNSUPPORTED;
    const double scalars[FO_MAX_SCALARS] = {0};
    if (X && X->kind == FO_CSR) return FO_ERR_UNSUPPORTED;     // chains over a CSR main input are interpreted
    return fo::run_cell(chain, X, sides, n_sides, scalars, n_scalars, magg ? FO_CELL_FULL_AGG : agg, magg != 0,
                        nullptr, nullptr, nullptr, 0, nullptr, true, true);
}

int fo_cell_stamps(void *ws, void *stream, unsigned long long *ns)
{
    if (!ws || !ns) return FO_ERR_NULL;
    fo::WsHead *head = (fo::WsHead *)ws;
    unsigned long long raw[4];
    cudaError_t e = cudaMemcpyAsync(raw, &head->pad[0], sizeof(raw), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(&head->pad[0], 0, sizeof(raw), (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return fo::cuda_fail(e);
    ns[0] = ~raw[0];
    ns[1] = raw[1];
    ns[2] = raw[2];
    ns[3] = raw[3];
    return FO_OK;
}

int fo_set_force_interpreter(int on)
{
    const int prev = fo::g_force_interpreter ? 1 : 0;
    fo::g_force_interpreter = on != 0;
    return prev;
}

size_t fused_cell_workspace_bytes(const fo_mat *X, int agg)
{
    if (!X || agg < FO_CELL_NO_AGG || agg > FO_CELL_FULL_AGG) return 0;
    if (X->kind == FO_CSR) return fo::cell_csr_ws_bytes(agg, 1);
    if (X->kind != FO_DENSE || X->dense.rows < 0 || X->dense.cols < 0) return 0;
    return fo::cell_ws_bytes(X->dense.rows, X->dense.cols, agg, 1);
}

size_t fused_magg_workspace_bytes(const fo_mat *X, int n_out)
{
    if (!X || n_out < 1 || n_out > FO_MAX_OUT) return 0;
    if (X->kind == FO_CSR) return fo::cell_csr_ws_bytes(FO_CELL_FULL_AGG, n_out);
    if (X->kind != FO_DENSE) return 0;
    return fo::cell_ws_bytes(X->dense.rows, X->dense.cols, FO_CELL_FULL_AGG, n_out);
}

int fused_cell(const fo_chain *chain, const fo_mat *X, const fo_side *sides, int n_sides,
               const double *scalars, int n_scalars, int agg, double *out, long long *out_nnz, void *ws,
               size_t ws_bytes, void *stream)
{
    return fo::run_cell(chain, X, sides, n_sides, scalars, n_scalars, agg, false, out, out_nnz, ws,
                        ws_bytes, stream, true);
}

int fused_magg(const fo_chain *chain, const fo_mat *X, const fo_side *sides, int n_sides,
               const double *scalars, int n_scalars, double *out, void *ws, size_t ws_bytes,
               void *stream)
{
    return fo::run_cell(chain, X, sides, n_sides, scalars, n_scalars, FO_CELL_FULL_AGG, true, out,
                        nullptr, ws, ws_bytes, stream, true);
}

}  // extern "C"
