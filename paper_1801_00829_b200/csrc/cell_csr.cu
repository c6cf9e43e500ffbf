// Cell and MAgg templates over a CSR main input: the sparse-safe binding of
// Table 1 / Section 2.2 - the chain runs on the stored cells only, side inputs
// are read at each stored cell's (row, column).
//
// A warp takes blocks of 32 consecutive rows; G lanes share a row (G from the
// matrix's mean row length), 32 / G rows at a time, with a warp-uniform trip
// count.  The cells of a block are one contiguous piece of colidx / vals, so the
// loads of neighbouring groups fall into the same cache lines.  Aggregation:
//   full  per-lane sums -> CTA -> workspace partial -> last CTA (fixed order);
//   row   the G lanes of a row are added by a shuffle tree (fixed order);
//   none  one value per stored cell, in X's pattern;
//   col   out[col] += value with global fp64 atomics after zeroing `out`
//         (the order of these additions is not fixed).
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <type_traits>

#include "cell_csr.h"
#include "cell_csr.cuh"
#include "jit.h"
#include "spec.cuh"

namespace fo {

namespace {

__global__ void csr_fill_zero_kernel(double *out, long long n)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
         i += (long long)gridDim.x * blockDim.x)
        out[i] = 0.0;
}

cudaError_t fill_zero(double *out, long long n, cudaStream_t st)
{
    if (n <= 0) return cudaSuccess;
    const long long b = (n + 255) / 256;
    csr_fill_zero_kernel<<<(unsigned)(b > 1024 ? 1024 : b), 256, 0, st>>>(out, n);
    return cudaGetLastError();
}

template <class EVAL, int NOUT>
cudaError_t launch_by_group(const DevChain &ch, const CsrCellParams &p, double mean_len, int grid,
                            cudaStream_t st)
{
    if (mean_len <= 12.0) cell_csr_kernel<EVAL, NOUT, 2><<<grid, kThreads, 0, st>>>(ch, p);
    else if (mean_len <= 48.0) cell_csr_kernel<EVAL, NOUT, 8><<<grid, kThreads, 0, st>>>(ch, p);
    else cell_csr_kernel<EVAL, NOUT, 32><<<grid, kThreads, 0, st>>>(ch, p);
    return cudaGetLastError();
}

}  // namespace

size_t cell_csr_ws_bytes(int agg, int n_out)
{
    if (agg == FO_CELL_FULL_AGG) return sizeof(WsHead) + (size_t)kMaxPartials * (size_t)n_out * sizeof(double);
    return sizeof(WsHead);
}

int run_cell_csr(const fo_chain *chain, const fo_csr &X, const fo_side *sides, int n_sides,
                 const double *scalars, int n_scalars, int agg, bool magg, double *out, void *ws,
                 size_t ws_bytes, void *stream, bool may_compile)
{
    if (X.rows < 0 || X.cols < 0 || X.nnz < 0) return FO_ERR_SHAPE;
    if (X.nnz > 0x7fffffffLL) return FO_ERR_UNSUPPORTED;
    if (!X.rowptr) return FO_ERR_NULL;
    if (X.nnz > 0 && (!X.colidx || !X.vals)) return FO_ERR_NULL;

    DevChain ch;
    int rc = translate_chain(chain, kUseCell, n_sides, scalars, n_scalars, 1, magg ? FO_MAX_OUT : 1, &ch);
    if (rc != FO_OK) return rc;

    CsrCellParams p;
    memset(&p, 0, sizeof(p));
    p.rowptr = X.rowptr; p.colidx = X.colidx; p.vals = X.vals;
    p.rows = X.rows; p.cols = X.cols;
    p.agg = agg;
    p.sides.n = n_sides;
    for (int k = 0; k < n_sides; ++k) {
        const fo_side &s = sides[k];
        if (s.sparse) {
            const fo_csr &y = *s.sparse;
            if (s.access != FO_AT_CELL || y.rows != X.rows || y.cols != X.cols || y.nnz < 0) return FO_ERR_SHAPE;
            if (y.nnz > 0x7fffffffLL) return FO_ERR_UNSUPPORTED;
            if (!y.rowptr) return FO_ERR_NULL;
            if (y.nnz > 0 && (!y.colidx || !y.vals)) return FO_ERR_NULL;
            p.sides.s[k].data = y.vals;
            p.sides.s[k].ld = 0;
            p.sides.s[k].access = kAtCellSparse;
            p.side_rowptr[k] = y.rowptr;
            p.side_colidx[k] = y.colidx;
            continue;
        }
        if (s.m.rows < 0 || s.m.cols < 0 || s.m.ld < s.m.cols) return FO_ERR_SHAPE;
        if (s.m.rows > 0 && s.m.cols > 0 && !s.m.data) return FO_ERR_NULL;
        switch (s.access) {
            case FO_AT_CELL: if (s.m.rows != X.rows || s.m.cols != X.cols) return FO_ERR_SHAPE; break;
            case FO_AT_ROW: if (s.m.rows != X.rows || s.m.cols != 1) return FO_ERR_SHAPE; break;
            case FO_AT_COL: if (s.m.rows != 1 || s.m.cols != X.cols) return FO_ERR_SHAPE; break;
            default: return FO_ERR_SHAPE;
        }
        p.sides.s[k].data = s.m.data;
        p.sides.s[k].ld = s.m.ld;
        p.sides.s[k].access = s.access;
    }
    rc = check_workspace(ws, ws_bytes, cell_csr_ws_bytes(agg, ch.n_out));
    if (rc != FO_OK) return rc;
    p.head = (WsHead *)ws;
    p.partials = (double *)((char *)ws + sizeof(WsHead));
    p.out = out;
    cudaStream_t st = (cudaStream_t)stream;

    // empty sums, and the accumulator of the atomic column sums
    cudaError_t e = cudaSuccess;
    if (agg == FO_CELL_COL_AGG) e = fill_zero(out, X.cols, st);
    if (X.nnz == 0 || X.rows == 0) {
        if (agg == FO_CELL_FULL_AGG) e = fill_zero(out, ch.n_out, st);
        else if (agg == FO_CELL_ROW_AGG) e = fill_zero(out, X.rows, st);
        return e == cudaSuccess ? FO_OK : cuda_fail(e);
    }
    if (e != cudaSuccess) return cuda_fail(e);

    const int sms = sm_count();
    if (sms <= 0) return cuda_fail(cudaErrorNoDevice);
    const double mean_len = (double)X.nnz / (double)X.rows;
    // rows a warp takes at a time: 32, or fewer when the matrix has too few rows to give every
    // warp of the machine a block (never fewer than 32 / G, G = the lanes that share a row)
    const int lanes_per_row = mean_len <= 12.0 ? 2 : mean_len <= 48.0 ? 8 : 32;
    int rb = 32;
    while (rb > 32 / lanes_per_row && (X.rows + rb - 1) / rb < (long long)sms * 16) rb >>= 1;
    p.rb = rb;
    const long long nblocks = (X.rows + rb - 1) / rb;
    long long grid = (nblocks + kThreads / 32 - 1) / (kThreads / 32);
    if (grid > (long long)sms * 8) grid = (long long)sms * 8;
    if (grid > kMaxPartials) grid = kMaxPartials;

    switch (force_interpreter() ? kSpecNone : match_cell_spec(ch)) {
        case kSpecMul2: e = launch_by_group<EvalSpec<kSpecMul2>, 1>(ch, p, mean_len, (int)grid, st); break;
        case kSpecMul3: e = launch_by_group<EvalSpec<kSpecMul3>, 1>(ch, p, mean_len, (int)grid, st); break;
        case kSpecSq: e = launch_by_group<EvalSpec<kSpecSq>, 1>(ch, p, mean_len, (int)grid, st); break;
        case kSpecMagg2: e = launch_by_group<EvalSpec<kSpecMagg2>, 2>(ch, p, mean_len, (int)grid, st); break;
        case kSpecMagg3: e = launch_by_group<EvalSpec<kSpecMagg3>, 3>(ch, p, mean_len, (int)grid, st); break;
        default:
            // no built-in specialisation: the same kernel compiled for this chain at run time,
            // else the interpreter
            if (!force_interpreter()) {
                const JitSpec sp = {kJitCsr, lanes_per_row, 0, 0};
                const int jrc = jit_launch(sp, ch, &p, (unsigned)grid, 1, st, may_compile && jit_first_use(), true);
                if (jrc == FO_OK) return FO_OK;
                if (jrc != kJitUnavailable) return jrc;
            }
            if (ch.n_out == 1) e = launch_by_group<EvalInterp<kRegs>, 1>(ch, p, mean_len, (int)grid, st);
            else e = launch_by_group<EvalInterp<kRegs>, FO_MAX_OUT>(ch, p, mean_len, (int)grid, st);
    }
    return e == cudaSuccess ? FO_OK : cuda_fail(e);
}

}  // namespace fo
