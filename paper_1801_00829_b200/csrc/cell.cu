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

#include "cell_flat.cuh"
#include "jit.h"
#include "cell_csr.h"
#include "spec.cuh"

namespace fo {

namespace {

// ------------------------------------------------------------------ rows
// Loads the pair (col, col+1) of a row; elements at or beyond `cols` read as 0.
template <bool ALIGNED>
__device__ __forceinline__ double2 load_pair(const double *row, long long col, long long cols)
{
    if (col + 1 < cols) {
        if (ALIGNED) return ld_stream2(row + col);
        return make_double2(ld_stream1(row + col), ld_stream1(row + col + 1));
    }
    if (col < cols) return make_double2(ld_stream1(row + col), 0.0);
    return make_double2(0.0, 0.0);
}

__device__ __forceinline__ double2 load_pair_cached(const double *row, long long col, long long cols)
{
    return make_double2(col < cols ? __ldg(row + col) : 0.0, col + 1 < cols ? __ldg(row + col + 1) : 0.0);
}

// Inputs of the cells (rowa, ca), (rowa, ca+1), (rowb, cb), (rowb, cb+1).
template <class EVAL, bool ALIGNED>
__device__ __forceinline__ void load_inputs_2d(const DevChain &ch, const CellParams &p,
                                               long long rowa, long long ca, long long rowb,
                                               long long cb, bool have_b, double (&in)[kIn][kV])
{
    put4(in[0], load_pair<ALIGNED>(p.X + rowa * p.ldx, ca, p.cols),
         have_b ? load_pair<ALIGNED>(p.X + rowb * p.ldx, cb, p.cols) : make_double2(0.0, 0.0));
#pragma unroll
    for (int k = 0; k < FO_MAX_SIDES; ++k) {
        if (EVAL::uses_side(ch, k)) {
            const DevSide sd = p.sides.s[k];
            if (sd.access == FO_AT_ROW) {
                const double va = __ldg(sd.data + rowa * sd.ld);
                const double vb = have_b ? __ldg(sd.data + rowb * sd.ld) : 0.0;
                put4(in[1 + k], make_double2(va, va), make_double2(vb, vb));
            } else if (sd.access == FO_AT_CELL) {
                put4(in[1 + k], load_pair<ALIGNED>(sd.data + rowa * sd.ld, ca, p.cols),
                     have_b ? load_pair<ALIGNED>(sd.data + rowb * sd.ld, cb, p.cols)
                            : make_double2(0.0, 0.0));
            } else {              // row vector, reused by every row: keep it cached
                put4(in[1 + k], load_pair_cached(sd.data, ca, p.cols),
                     have_b ? load_pair_cached(sd.data, cb, p.cols) : make_double2(0.0, 0.0));
            }
        }
    }
}

template <class EVAL, int NOUT, int AGG, bool ALIGNED>
__global__ void __launch_bounds__(kThreads)
cell_rows_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ CellParams p)
{
    __shared__ double s_red[NOUT * 32];
    __shared__ unsigned int s_flag;
    double acc[NOUT];
#pragma unroll
    for (int k = 0; k < NOUT; ++k) acc[k] = 0.0;

    const int lane = threadIdx.x & 31;
    const long long warp0 = (long long)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    const long long nwarps = (long long)gridDim.x * (kThreads / 32);

    // Rows of at most 64 columns: a warp takes several rows at a time instead of leaving most
    // lanes without a column.  LPR lanes (a power of two >= cols / 2) share a row, 32 / LPR rows
    // go into the first pair of values of a lane and as many into the second.
    if (p.cols <= 64) {
        int lpr = 1;
        while (2 * lpr < p.cols) lpr <<= 1;
        const int rw = 32 / lpr, sub = lane % lpr, rsel = lane / lpr;
        const long long ca = 2 * sub;
        for (long long r0 = warp0 * (2 * rw); r0 < p.rows; r0 += nwarps * (2 * rw)) {
            const long long rowa = r0 + rsel, rowb = r0 + rw + rsel;
            const bool have_a = rowa < p.rows, have_b = rowb < p.rows;
            const long long ra = have_a ? rowa : p.rows - 1;        // loads stay inside the matrix
            double in[kIn][kV];
            load_inputs_2d<EVAL, ALIGNED>(ch, p, ra, ca, rowb, ca, have_b, in);
            double o[NOUT][kV];
            EVAL::template run<kV, NOUT>(ch, in, o);
            const bool valid[kV] = {have_a && ca < p.cols, have_a && ca + 1 < p.cols,
                                    have_b && ca < p.cols, have_b && ca + 1 < p.cols};
            if (AGG == kAggNone) {
                double *oa = p.out + rowa * p.cols, *ob = p.out + rowb * p.cols;
                if (valid[0]) oa[ca] = o[0][0];
                if (valid[1]) oa[ca + 1] = o[0][1];
                if (valid[2]) ob[ca] = o[0][2];
                if (valid[3]) ob[ca + 1] = o[0][3];
            } else if (AGG == kAggRow) {
                double sa = (valid[0] ? o[0][0] : 0.0) + (valid[1] ? o[0][1] : 0.0);
                double sb = (valid[2] ? o[0][2] : 0.0) + (valid[3] ? o[0][3] : 0.0);
                for (int off = lpr >> 1; off >= 1; off >>= 1) {
                    sa += __shfl_xor_sync(0xffffffffu, sa, off);
                    sb += __shfl_xor_sync(0xffffffffu, sb, off);
                }
                if (sub == 0 && have_a) p.out[rowa] = sa;
                if (sub == 0 && have_b) p.out[rowb] = sb;
            } else {
                add_outputs<NOUT>(o, valid, acc);
            }
        }
    } else
    for (long long row = warp0; row < p.rows; row += nwarps) {
        double rowacc[NOUT];
#pragma unroll
        for (int k = 0; k < NOUT; ++k) rowacc[k] = 0.0;
        for (long long c0 = 0; c0 < p.cols; c0 += 128) {
            const long long ca = c0 + 2 * lane, cb = ca + 64;
            double in[kIn][kV];
            load_inputs_2d<EVAL, ALIGNED>(ch, p, row, ca, row, cb, true, in);
            double o[NOUT][kV];
            EVAL::template run<kV, NOUT>(ch, in, o);
            const bool valid[kV] = {ca < p.cols, ca + 1 < p.cols, cb < p.cols, cb + 1 < p.cols};
            if (AGG == kAggNone) {
                double *orow = p.out + row * p.cols;
                if (valid[0]) orow[ca] = o[0][0];
                if (valid[1]) orow[ca + 1] = o[0][1];
                if (valid[2]) orow[cb] = o[0][2];
                if (valid[3]) orow[cb + 1] = o[0][3];
            } else if (AGG == kAggRow) {
                add_outputs<NOUT>(o, valid, rowacc);
            } else {
                add_outputs<NOUT>(o, valid, acc);
            }
        }
        if (AGG == kAggRow) {
            const double s = warp_sum(rowacc[0]);
            if (lane == 0) p.out[row] = s;
        }
    }

    if (AGG == kAggFull) {
        block_sum<NOUT>(acc, s_red);
        if (threadIdx.x == 0) {
#pragma unroll
            for (int k = 0; k < NOUT; ++k)
                if (k < ch.n_out) p.partials[(size_t)blockIdx.x * ch.n_out + k] = acc[k];
        }
        if (publish_and_is_last(p.head, &s_flag))
            final_sum_small(p.partials, gridDim.x, ch.n_out, p.out, s_red);
    }
}

// ------------------------------------------------------------------ cols
// grid.x: tiles of 2 * cx columns; grid.y: row panels.  The 256 threads of a CTA
// form cx column pairs by 256 / cx row lanes (cx = p.cx <= 256, chosen so that the
// column tiles are equal and narrow matrices still fill the CTA); a thread owns a column pair
// and walks every (256 / cx)-th row of its panel, two rows per chain evaluation;
// the row lanes are then added in order through shared memory.
template <class EVAL, bool ALIGNED>
__global__ void __launch_bounds__(kThreads)
cell_cols_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ CellParams p)
{
    __shared__ unsigned int s_flag;
    __shared__ double2 s_lane[kThreads];
    const int cx = p.cx, ry = kThreads / cx;          // threads beyond cx * ry idle
    const int tx = threadIdx.x % cx, ty = threadIdx.x / cx;
    const long long col = ((long long)blockIdx.x * cx + tx) * 2;
    const long long per = (p.rows + p.panels - 1) / p.panels;
    const long long r0 = (long long)blockIdx.y * per;
    const long long r1 = (r0 + per < p.rows) ? r0 + per : p.rows;
    double a0 = 0.0, a1 = 0.0;

    if (col < p.cols && ty < ry) {
        long long row = r0 + ty;
        // four rows per turn while they last: twice the loads in flight per thread
        for (; row + 3 * ry < r1; row += 4 * ry) {
            double in[kIn][kV], in2[kIn][kV];
            load_inputs_2d<EVAL, ALIGNED>(ch, p, row, col, row + ry, col, true, in);
            load_inputs_2d<EVAL, ALIGNED>(ch, p, row + 2 * ry, col, row + 3 * ry, col, true, in2);
            double o[1][kV], o2[1][kV];
            EVAL::template run<kV, 1>(ch, in, o);
            EVAL::template run<kV, 1>(ch, in2, o2);
            a0 += o[0][0];
            a1 += o[0][1];
            a0 += o[0][2];
            a1 += o[0][3];
            a0 += o2[0][0];
            a1 += o2[0][1];
            a0 += o2[0][2];
            a1 += o2[0][3];
        }
        for (; row < r1; row += 2 * ry) {
            const bool two = row + ry < r1;
            double in[kIn][kV];
            load_inputs_2d<EVAL, ALIGNED>(ch, p, row, col, row + ry, col, two, in);
            double o[1][kV];
            EVAL::template run<kV, 1>(ch, in, o);
            a0 += o[0][0];
            a1 += o[0][1];
            if (two) {
                a0 += o[0][2];
                a1 += o[0][3];
            }
        }
    }
    if (ry > 1) {
        s_lane[threadIdx.x] = make_double2(a0, a1);
        __syncthreads();
        if (ty == 0) {
            for (int k = 1; k < ry; ++k) {
                a0 += s_lane[k * cx + tx].x;
                a1 += s_lane[k * cx + tx].y;
            }
        }
    }
    if (col < p.cols && ty == 0) {
        if (p.panels == 1) {
            p.out[col] = a0;
            if (col + 1 < p.cols) p.out[col + 1] = a1;
        } else {
            double *pp = p.partials + (size_t)blockIdx.y * p.cols;
            pp[col] = a0;
            if (col + 1 < p.cols) pp[col + 1] = a1;
        }
    }
    if (p.panels == 1) return;
    // the last panel of this column tile to finish adds the tile's partials, panel 0 first
    if (take_ticket(&p.head->group[blockIdx.x], (unsigned)p.panels, &s_flag) && col < p.cols && ty == 0) {
        double s0 = 0.0, s1 = 0.0;
        const bool two = col + 1 < p.cols;
        for (int g = 0; g < p.panels; ++g) {
            s0 += __ldcg(p.partials + (size_t)g * p.cols + col);
            if (two) s1 += __ldcg(p.partials + (size_t)g * p.cols + col + 1);
        }
        p.out[col] = s0;
        if (two) p.out[col + 1] = s1;
    }
}

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

// Test / benchmark switch: run every chain through the interpreter.
bool g_force_interpreter = false;

// Common body of fused_cell and fused_magg.
int run_cell(const fo_chain *chain, const fo_mat *X, const fo_side *sides, int n_sides,
             const double *scalars, int n_scalars, int agg, bool magg, double *out, long long *out_nnz,
             void *ws, size_t ws_bytes, void *stream, bool may_compile)
{
    if (!chain || !X || !out) return FO_ERR_NULL;
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
                            stream);
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
    rc = check_workspace(ws, ws_bytes, need);
    if (rc != FO_OK) return rc;
    p.head = (WsHead *)ws;
    p.partials = (double *)((char *)ws + sizeof(WsHead));
    p.out = out;
    p.stamps = tune_int("cell.stamps", 0) ? reinterpret_cast<unsigned long long *>(&p.head->pad[0]) : nullptr;

    cudaStream_t st = (cudaStream_t)stream;
    const long long ncells = xd.rows * xd.cols;
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
    switch (g_force_interpreter ? kSpecNone : match_cell_spec(ch)) {
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
            // no built-in specialisation: a kernel compiled for this chain at run time
            // (flat streaming case), else the interpreter
            if (!g_force_interpreter && flat && (agg == FO_CELL_FULL_AGG || agg == FO_CELL_NO_AGG)) {
                const int jrc = jit_launch_flat(ch, p, agg == FO_CELL_NO_AGG, grid, st, may_compile);
                if (jrc == FO_OK) return FO_OK;
                if (jrc != kJitUnavailable) return jrc;
            }
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
