// Row template (Table 1; Fig. 1(b); Section 5.2 "Row Operations"): one pass over
// the rows of X computing, per row i,  d = X_i . v,  t_i = chain(d, sides_i),
// and then  out += t_i * X_i^T  (col_t_agg),  out[i] = t_i  (row_agg)  or
// out = sum_i t_i  (full_agg).  The row is read from HBM once and used twice
// from on-chip memory - the GPU form of the paper's "each row fits L1" argument.
//
// Dense X: a CTA streams tiles of rows into a shared-memory ring with bulk
// asynchronous copies (mbarrier-tracked, waits bounded); warps own column slices
// of the rows, of v and of the output accumulator, all in registers.  CSR X: a
// warp per block of 32 rows, an 8-lane group per row; v and the output
// accumulator live in shared memory.
#include <stdio.h>
#include <stdlib.h>

#include <type_traits>

#include "jit.h"
#include "row_kernels.cuh"

namespace fo {

namespace {

__global__ void row_fill_zero_kernel(double *out, long long n)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
         i += (long long)gridDim.x * blockDim.x)
        out[i] = 0.0;
}

// ------------------------------------------------------------------- host
constexpr long long kDenseMaxCols = 8192;
constexpr long long kCsrMaxCols = 8192;
constexpr size_t kSmemBudget = 208 * 1024;   // dynamic shared memory of the dense kernel

bool aligned16(const void *q) { return ((uintptr_t)q & 15u) == 0; }

int row_grid_cap() { return 148 * 4; }     // bound used for workspace sizing

size_t row_ws_bytes(long long cols, int agg)
{
    if (agg == FO_ROW_COL_T_AGG)      // per-CTA vectors plus one vector per group of CTAs
        return sizeof(WsHead) + (size_t)(row_grid_cap() + row_grid_cap() / kGroup + 1) * (size_t)cols * sizeof(double);
    if (agg == FO_ROW_FULL_AGG) return sizeof(WsHead) + (size_t)row_grid_cap() * sizeof(double);
    return sizeof(WsHead);
}

template <int NCH, int W, int R, bool STAGED>
cudaError_t launch_dense_agg(const DevChain &ch, const RowParams &p, int agg, int grid, size_t smem,
                             cudaStream_t st)
{
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<grid, kDenseBlock, smem, st>>>(ch, p);
        return cudaGetLastError();
    };
    if (agg == FO_ROW_COL_T_AGG) return go(row_dense_kernel<NCH, W, R, kRowColT, STAGED>);
    if (agg == FO_ROW_NO_AGG) return go(row_dense_kernel<NCH, W, R, kRowNone, STAGED>);
    if (agg == FO_ROW_ROW_AGG) return go(row_dense_kernel<NCH, W, R, kRowRow, STAGED>);
    return go(row_dense_kernel<NCH, W, R, kRowFull, STAGED>);
}

// Shape of the dense kernel for rows of n columns: chunks per lane, warps per
// group, rows per group and stage.  cols <= 64 * nch * w; nch * r <= 8 keeps a
// stage's rows in 32 registers per lane.
struct DenseShape {
    int nch, w, r;
};

// The shapes below are the ones compiled.
DenseShape dense_shape(long long n)
{
    // measured on B200: several small independent groups beat one large group
    // (1000 columns: {4,4,2} 6.6 TB/s, {2,8,4} 6.4, {1,16,8} 5.1)
    // (512: {1,8,8} 6.2 vs {2,4,4} 5.9; 2048: {2,16,4} 6.0 vs {4,8,2} 5.1)
    if (n <= 64) return {1, 1, 8};
    if (n <= 128) return {1, 2, 8};
    if (n <= 256) return {1, 4, 8};
    if (n <= 512) return {1, 8, 8};
    if (n <= 1024) return {4, 4, 2};
    if (n <= 2048) return {2, 16, 4};
    if (n <= 4096) return {4, 16, 2};
    return {8, 16, 1};
}

template <bool STAGED>
cudaError_t launch_dense(const DevChain &ch, const RowParams &p, int agg, int grid, size_t smem,
                         cudaStream_t st)
{
    const DenseShape k = dense_shape(p.cols);
#define FO_SHAPE(A, B, C) \
    if (k.nch == A && k.w == B && k.r == C) return launch_dense_agg<A, B, C, STAGED>(ch, p, agg, grid, smem, st);
    FO_SHAPE(1, 1, 8) FO_SHAPE(1, 2, 8) FO_SHAPE(1, 4, 8) FO_SHAPE(1, 8, 8) FO_SHAPE(4, 4, 2)
    FO_SHAPE(2, 16, 4) FO_SHAPE(4, 16, 2) FO_SHAPE(8, 16, 1)
#undef FO_SHAPE
    return cudaErrorInvalidValue;
}

}  // namespace

}  // namespace fo

extern "C" {

size_t fused_row_workspace_bytes(const fo_mat *X, int agg)
{
    if (!X) return 0;
    if (agg == FO_ROW_COL_AGG) agg = FO_ROW_COL_T_AGG;
    if (agg != FO_ROW_COL_T_AGG && agg != FO_ROW_ROW_AGG && agg != FO_ROW_FULL_AGG && agg != FO_ROW_NO_AGG) return 0;
    const long long cols = X->kind == FO_DENSE ? X->dense.cols : X->kind == FO_CSR ? X->csr.cols : -1;
    if (cols < 0) return 0;
    return fo::row_ws_bytes(cols, agg);
}

int fused_row(const fo_chain *chain, const fo_mat *X, const double *v, const fo_side *sides,
              int n_sides, const double *scalars, int n_scalars, int agg, double *out, void *ws,
              size_t ws_bytes, void *stream)
{
    using namespace fo;
    if (!chain || !X) return FO_ERR_NULL;
    if (n_sides > 0 && !sides) return FO_ERR_NULL;
    // col_agg (1 x n) and col_t_agg (n x 1) hold the same n values
    if (agg == FO_ROW_COL_AGG) agg = FO_ROW_COL_T_AGG;
    if (agg != FO_ROW_COL_T_AGG && agg != FO_ROW_ROW_AGG && agg != FO_ROW_FULL_AGG && agg != FO_ROW_NO_AGG)
        return FO_ERR_UNSUPPORTED;
    if (X->kind != FO_DENSE && X->kind != FO_CSR) return FO_ERR_SHAPE;
    const bool csr = X->kind == FO_CSR;
    const long long rows = csr ? X->csr.rows : X->dense.rows;
    const long long cols = csr ? X->csr.cols : X->dense.cols;
    if (rows < 0 || cols < 0) return FO_ERR_SHAPE;
    if (csr) {
        if (X->csr.nnz < 0 || X->csr.nnz >= (1ll << 31)) return FO_ERR_UNSUPPORTED;
        if (!X->csr.rowptr) return FO_ERR_NULL;
        if (X->csr.nnz > 0 && (!X->csr.colidx || !X->csr.vals)) return FO_ERR_NULL;
    } else {
        if (X->dense.ld < cols) return FO_ERR_SHAPE;
        if (rows > 0 && cols > 0 && !X->dense.data) return FO_ERR_NULL;
    }
    if (cols > 0 && !v) return FO_ERR_NULL;

    DevChain ch;
    int rc = translate_chain(chain, kUseRow, n_sides, scalars, n_scalars, 1, 1, &ch);
    if (rc != FO_OK) return rc;

    RowParams p;
    memset(&p, 0, sizeof(p));
    p.rows = rows; p.cols = cols; p.v = v;
    p.sides.n = n_sides;
    for (int k = 0; k < n_sides; ++k) {
        const fo_side &s = sides[k];
        if (s.sparse) return FO_ERR_UNSUPPORTED;       // sparse sides: CSR main input of Cell / MAgg only
        if (s.access != FO_AT_ROW) return FO_ERR_SHAPE;
        if (s.m.rows != rows || s.m.cols != 1 || s.m.ld < 1) return FO_ERR_SHAPE;
        if (rows > 0 && !s.m.data) return FO_ERR_NULL;
        p.sides.s[k].data = s.m.data;
        p.sides.s[k].ld = s.m.ld;
        p.sides.s[k].access = s.access;
    }
    if (agg == FO_ROW_COL_T_AGG && cols > (csr ? kCsrMaxCols : kDenseMaxCols)) return FO_ERR_UNSUPPORTED;
    if (cols > kCsrMaxCols) return FO_ERR_UNSUPPORTED;
    if (!csr && cols > kDenseMaxCols) return FO_ERR_UNSUPPORTED;

    // row chains evaluated inline: t = side0 * d (either operand order) and t = d
    p.chain_kind = kChainGeneric;
    if (ch.n_ops == 0 && ch.out[0] == 0) p.chain_kind = kChainDot;
    if (ch.n_ops == 1 && ch.ops[0].opcode == FO_OP_MUL && ch.out[0] == ch.ops[0].dst &&
        ((ch.ops[0].a == 0 && ch.ops[0].b == 1) || (ch.ops[0].a == 1 && ch.ops[0].b == 0)))
        p.chain_kind = kChainSideTimesDot;

    rc = check_workspace(ws, ws_bytes, row_ws_bytes(cols, agg));
    if (rc != FO_OK) return rc;
    p.head = (WsHead *)ws;
    p.partials = (double *)((char *)ws + sizeof(WsHead));
    p.out = out;
    cudaStream_t st = (cudaStream_t)stream;

    const long long nout = agg == FO_ROW_COL_T_AGG ? cols : agg == FO_ROW_ROW_AGG ? rows
                           : agg == FO_ROW_NO_AGG ? (csr ? X->csr.nnz : rows * cols) : 1;
    if (!out && nout > 0) return FO_ERR_NULL;
    if (rows == 0 || cols == 0) {
        // no rows: empty sums; no columns: d = 0 for every row, which the chain may
        // still map to a non-zero t - handled by the kernels below unless rows == 0
        if (rows == 0 || agg == FO_ROW_COL_T_AGG || agg == FO_ROW_NO_AGG) {
            // (no_agg without rows or columns has nothing to write)
            if (agg == FO_ROW_NO_AGG) return FO_OK;
            if (nout > 0) {
                const long long b = (nout + 255) / 256;
                row_fill_zero_kernel<<<(unsigned)(b > 1024 ? 1024 : b), 256, 0, st>>>(out, nout);
            }
            const cudaError_t e = cudaGetLastError();
            return e == cudaSuccess ? FO_OK : cuda_fail(e);
        }
    }

    const int sms = sm_count();
    if (sms <= 0) return cuda_fail(cudaErrorNoDevice);
    cudaError_t e;
    // a chain without an inline form: the same kernels compiled for it at run time, else interpreted
    const bool try_jit = p.chain_kind == kChainGeneric && !force_interpreter();
    const int kagg = agg == FO_ROW_COL_T_AGG ? kRowColT : agg == FO_ROW_ROW_AGG ? kRowRow
                     : agg == FO_ROW_FULL_AGG ? kRowFull : kRowNone;
    if (csr) {
        p.rowptr = X->csr.rowptr; p.colidx = X->csr.colidx; p.vals = X->csr.vals;
        const size_t smem = (size_t)cols * 8 * 2 + (size_t)kWarps * kCsrStage * 12;    // staged kernel
        // lanes per row from the mean row length: about four trips for a typical row
        const double mean_len = rows > 0 ? (double)X->csr.nnz / (double)rows : 0.0;
        const int lanes_per_row = mean_len <= 12.0 ? 2 : mean_len <= 24.0 ? 4 : mean_len <= 48.0 ? 8
                                  : mean_len <= 96.0 ? 16 : 32;
        // rows a warp takes at a time: 32, or fewer when there are too few rows to give every warp
        // of the machine a block (never fewer than 32 / lanes per row)
        int rb = 32;
        while (rb > 32 / lanes_per_row && (rows + rb - 1) / rb < (long long)sms * 16) rb >>= 1;
        p.rb = rb;
        long long grid = ((rows + rb - 1) / rb + kWarps - 1) / kWarps;
        const long long cap = (long long)sms * 3 < row_grid_cap() ? (long long)sms * 3 : row_grid_cap();
        if (grid > cap) grid = cap;
        if (grid < 1) grid = 1;
        // the column scatter works from a staged slice, everything else from registers
        const size_t smem_reg = (size_t)cols * 8;
        auto go = [&](auto kern, size_t bytes) -> cudaError_t {
            cudaError_t e2 = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
            if (e2 != cudaSuccess) return e2;
            kern<<<(unsigned)grid, kThreads, bytes, st>>>(ch, p);
            return cudaGetLastError();
        };
        auto by_agg = [&](auto g) -> cudaError_t {
            constexpr int G = decltype(g)::value;
            if (try_jit) {
                const JitSpec js = agg == FO_ROW_COL_T_AGG ? JitSpec{kJitRowCsr, G, 0, 0, 0, 0}
                                                           : JitSpec{kJitRowCsrReg, kagg, G, 0, 0, 0};
                const int jrc = jit_launch(js, ch, &p, (unsigned)grid, 1, st, jit_first_use(), true,
                                           agg == FO_ROW_COL_T_AGG ? smem : smem_reg);
                if (jrc == FO_OK) return cudaSuccess;
                if (jrc != kJitUnavailable) return cudaErrorLaunchFailure;
            }
            if (agg == FO_ROW_COL_T_AGG)
                return p.chain_kind == kChainGeneric ? go(row_csr_kernel<G, true>, smem)
                                                     : go(row_csr_kernel<G, false>, smem);
            const bool gen = p.chain_kind == kChainGeneric;
            if (agg == FO_ROW_NO_AGG)
                return gen ? go(row_csr_reg_kernel<kRowNone, G, true>, smem_reg)
                           : go(row_csr_reg_kernel<kRowNone, G, false>, smem_reg);
            if (agg == FO_ROW_ROW_AGG)
                return gen ? go(row_csr_reg_kernel<kRowRow, G, true>, smem_reg)
                           : go(row_csr_reg_kernel<kRowRow, G, false>, smem_reg);
            return gen ? go(row_csr_reg_kernel<kRowFull, G, true>, smem_reg)
                       : go(row_csr_reg_kernel<kRowFull, G, false>, smem_reg);
        };
        if (mean_len <= 12.0) e = by_agg(std::integral_constant<int, 2>());
        else if (mean_len <= 24.0) e = by_agg(std::integral_constant<int, 4>());
        else if (mean_len <= 48.0) e = by_agg(std::integral_constant<int, 8>());
        else if (mean_len <= 96.0) e = by_agg(std::integral_constant<int, 16>());
        else e = by_agg(std::integral_constant<int, 32>());
    } else {
        p.X = X->dense.data; p.ldx = X->dense.ld;
        p.out_vec = (aligned16(out) && cols % 2 == 0) ? 1 : 0;
        if (cols <= kNarrowMax) {
            // a thread per row; the knob row.narrow = 0 keeps the warp-per-row-slice kernel
            if (tune_int("row.narrow", 1) != 0) {
                const bool vec = aligned16(p.X) && (p.ldx % 2 == 0) && (cols % 2 == 0);
                long long grid = (rows + kThreads - 1) / kThreads;
                const long long cap = (long long)sms * 4 < row_grid_cap() ? (long long)sms * 4 : row_grid_cap();
                if (grid > cap) grid = cap;
                if (grid < 1) grid = 1;
                auto gon = [&](auto nc) -> cudaError_t {
                    constexpr int NC = decltype(nc)::value;
                    if (try_jit) {
                        const JitSpec js = {kJitRowNarrow, NC, kagg, vec ? 1 : 0, 0, 0};
                        const int jrc = jit_launch(js, ch, &p, (unsigned)grid, 1, st, jit_first_use(), true);
                        if (jrc == FO_OK) return cudaSuccess;
                        if (jrc != kJitUnavailable) return cudaErrorLaunchFailure;
                    }
#define FO_NARROW(A)                                                                        \
    do {                                                                                    \
        if (vec) row_narrow_kernel<NC, A, true><<<(unsigned)grid, kThreads, 0, st>>>(ch, p);  \
        else row_narrow_kernel<NC, A, false><<<(unsigned)grid, kThreads, 0, st>>>(ch, p);     \
    } while (0)
                    if (agg == FO_ROW_COL_T_AGG) FO_NARROW(kRowColT);
                    else if (agg == FO_ROW_ROW_AGG) FO_NARROW(kRowRow);
                    else if (agg == FO_ROW_FULL_AGG) FO_NARROW(kRowFull);
                    else FO_NARROW(kRowNone);
#undef FO_NARROW
                    return cudaGetLastError();
                };
                e = cols <= 4 ? gon(std::integral_constant<int, 4>())
                    : cols <= 8 ? gon(std::integral_constant<int, 8>())
                    : cols <= 16 ? gon(std::integral_constant<int, 16>())
                                 : gon(std::integral_constant<int, 32>());
                return e == cudaSuccess ? FO_OK : cuda_fail(e);
            }
        }
        const bool staged = aligned16(p.X) && (p.ldx % 2 == 0) && (cols % 2 == 0) && cols >= 2;
        // ring geometry: every group of warps has its own ring of `stages` slots of r rows
        const DenseShape sh = dense_shape(cols);
        const int groups = kDenseWarps / sh.w;
        p.rows_per_stage = sh.r;
        const size_t slot_bytes = (size_t)sh.r * cols * 8 + (size_t)FO_MAX_SIDES * sh.r * 8;
        int stages = (int)(kSmemBudget / (slot_bytes * groups));
        if (stages > 8) stages = 8;
        if (stages * groups > kDenseMaxSlots) stages = kDenseMaxSlots / groups;
        if (stages < 2) stages = 2;
        p.stages = staged ? stages : 1;
        // used sides ride in the ring when they are contiguous, 16-byte aligned vectors
        p.sides_in_ring = staged ? 1 : 0;
        for (int k = 0; k < n_sides; ++k)
            if (((ch.side_used >> k) & 1u) && (p.sides.s[k].ld != 1 || !aligned16(p.sides.s[k].data)))
                p.sides_in_ring = 0;
        if (ch.side_used == 0) p.sides_in_ring = 0;
        size_t smem = staged ? slot_bytes * groups * stages : 0;     // the rings
        const size_t qs_bytes = (size_t)groups * cols * 8;           // group accumulators
        if (agg == FO_ROW_COL_T_AGG && smem < qs_bytes) smem = qs_bytes;
        const long long ntiles = (rows + sh.r - 1) / sh.r;
        long long grid = (ntiles + groups - 1) / groups;
        if (grid > sms) grid = sms;
        if (grid > row_grid_cap()) grid = row_grid_cap();
        if (grid < 1) grid = 1;
        if (try_jit) {
            const DenseShape k = dense_shape(cols);
            const JitSpec js = {kJitRowDense, k.nch, k.w, k.r, kagg, staged ? 1 : 0};
            const int jrc = jit_launch(js, ch, &p, (unsigned)grid, 1, st, jit_first_use(), true, smem, nullptr,
                                       kDenseBlock);
            if (jrc == FO_OK) return FO_OK;
            if (jrc != kJitUnavailable) return jrc;
        }
        e = staged ? launch_dense<true>(ch, p, agg, (int)grid, smem, st)
                   : launch_dense<false>(ch, p, agg, (int)grid, smem, st);
    }
    return e == cudaSuccess ? FO_OK : cuda_fail(e);
}

}  // extern "C"
