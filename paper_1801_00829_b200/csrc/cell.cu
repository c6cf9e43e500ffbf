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
#include "chain.cuh"

namespace fo {

namespace {

struct CellParams {
    const double *X;
    long long rows, cols, ldx;
    DevSides sides;
    WsHead *head;
    double *partials;
    double *out;
    int panels;           // cell_cols_kernel: number of row panels
    int pad;
};

constexpr int kV = 4;     // cells per thread per chain evaluation

enum { kAggNone = 0, kAggRow = 1, kAggFull = 3 };

template <int NR>
__device__ __forceinline__ void add_outputs(const DevChain &ch, const RegFile<NR, kV> &f,
                                            const bool (&valid)[kV], double *acc, int nout_max)
{
    for (int k = 0; k < nout_max; ++k) {
        if (k < ch.n_out) {
            double o[kV];
            operand<NR, kV>(ch, f, ch.out[k], o);
            double s = 0.0;
#pragma unroll
            for (int i = 0; i < kV; ++i) s += valid[i] ? o[i] : 0.0;
            acc[k] += s;
        }
    }
}

// ------------------------------------------------------------------ flat
template <int NR, int NOUT, bool STORE>
__global__ void __launch_bounds__(kThreads)
cell_flat_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ CellParams p)
{
    __shared__ double s_red[NOUT * 32];
    __shared__ unsigned int s_flag;
    double acc[NOUT];
#pragma unroll
    for (int k = 0; k < NOUT; ++k) acc[k] = 0.0;

    const long long ncells = p.rows * p.cols;
    const long long ntiles = ncells >> 10;          // full tiles of 1024 cells
    const int t = threadIdx.x;

    for (long long tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const long long o0 = (tile << 10) + 2 * t, o1 = o0 + 512;
        RegFile<NR, kV> f;
        {
            const double2 m0 = ld_stream2(p.X + o0), m1 = ld_stream2(p.X + o1);
            f.r[0][0] = m0.x; f.r[0][1] = m0.y; f.r[0][2] = m1.x; f.r[0][3] = m1.y;
        }
#pragma unroll
        for (int k = 0; k < FO_MAX_SIDES; ++k) {
            if (1 + k < NR && (ch.side_used >> k) & 1u) {
                const double *sp = p.sides.s[k].data;
                const double2 m0 = ld_stream2(sp + o0), m1 = ld_stream2(sp + o1);
                const int R = (1 + k < NR) ? 1 + k : 0;
                f.r[R][0] = m0.x; f.r[R][1] = m0.y; f.r[R][2] = m1.x; f.r[R][3] = m1.y;
            }
        }
        run_chain<NR, kV>(ch, f);
        if (STORE) {
            double o[kV];
            operand<NR, kV>(ch, f, ch.out[0], o);
            *reinterpret_cast<double2 *>(p.out + o0) = make_double2(o[0], o[1]);
            *reinterpret_cast<double2 *>(p.out + o1) = make_double2(o[2], o[3]);
        } else {
            const bool valid[kV] = {true, true, true, true};
            add_outputs<NR>(ch, f, valid, acc, NOUT);
        }
    }

    // ragged tail (< 1024 cells): one CTA, scalar loads
    const long long tail0 = ntiles << 10;
    if (tail0 < ncells && blockIdx.x == (unsigned)(ntiles % gridDim.x)) {
        RegFile<NR, kV> f;
        bool valid[kV];
        long long idx[kV];
#pragma unroll
        for (int i = 0; i < kV; ++i) {
            idx[i] = tail0 + t + i * kThreads;
            valid[i] = idx[i] < ncells;
            f.r[0][i] = valid[i] ? ld_stream1(p.X + idx[i]) : 0.0;
        }
#pragma unroll
        for (int k = 0; k < FO_MAX_SIDES; ++k) {
            if (1 + k < NR && (ch.side_used >> k) & 1u) {
                const int R = (1 + k < NR) ? 1 + k : 0;
#pragma unroll
                for (int i = 0; i < kV; ++i)
                    f.r[R][i] = valid[i] ? ld_stream1(p.sides.s[k].data + idx[i]) : 0.0;
            }
        }
        run_chain<NR, kV>(ch, f);
        if (STORE) {
            double o[kV];
            operand<NR, kV>(ch, f, ch.out[0], o);
#pragma unroll
            for (int i = 0; i < kV; ++i)
                if (valid[i]) p.out[idx[i]] = o[i];
        } else {
            add_outputs<NR>(ch, f, valid, acc, NOUT);
        }
    }

    if (!STORE) {
        block_sum<NOUT>(acc, s_red);
        if (t == 0) {
            for (int k = 0; k < NOUT; ++k)
                if (k < ch.n_out) p.partials[(size_t)blockIdx.x * ch.n_out + k] = acc[k];
        }
        if (publish_and_is_last(p.head, &s_flag))
            final_sum_small(p.partials, gridDim.x, ch.n_out, p.out, s_red);
    }
}

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

template <int NR, bool ALIGNED>
__device__ __forceinline__ void load_row_inputs(const DevChain &ch, const CellParams &p,
                                                long long row, long long ca, long long cb,
                                                RegFile<NR, kV> &f)
{
    {
        const double *xr = p.X + row * p.ldx;
        const double2 m0 = load_pair<ALIGNED>(xr, ca, p.cols), m1 = load_pair<ALIGNED>(xr, cb, p.cols);
        f.r[0][0] = m0.x; f.r[0][1] = m0.y; f.r[0][2] = m1.x; f.r[0][3] = m1.y;
    }
#pragma unroll
    for (int k = 0; k < FO_MAX_SIDES; ++k) {
        if (1 + k < NR && (ch.side_used >> k) & 1u) {
            const int R = (1 + k < NR) ? 1 + k : 0;
            const DevSide sd = p.sides.s[k];
            if (sd.access == FO_AT_ROW) {
                const double v = __ldg(sd.data + row * sd.ld);
                f.r[R][0] = v; f.r[R][1] = v; f.r[R][2] = v; f.r[R][3] = v;
            } else {
                const double *sr = sd.data + (sd.access == FO_AT_CELL ? row * sd.ld : 0);
                double2 m0, m1;
                if (sd.access == FO_AT_CELL) {
                    m0 = load_pair<ALIGNED>(sr, ca, p.cols);
                    m1 = load_pair<ALIGNED>(sr, cb, p.cols);
                } else {          // row vector, reused by every row: keep it cached
                    m0 = make_double2(ca < p.cols ? __ldg(sr + ca) : 0.0,
                                      ca + 1 < p.cols ? __ldg(sr + ca + 1) : 0.0);
                    m1 = make_double2(cb < p.cols ? __ldg(sr + cb) : 0.0,
                                      cb + 1 < p.cols ? __ldg(sr + cb + 1) : 0.0);
                }
                f.r[R][0] = m0.x; f.r[R][1] = m0.y; f.r[R][2] = m1.x; f.r[R][3] = m1.y;
            }
        }
    }
}

template <int NR, int NOUT, int AGG, bool ALIGNED>
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

    for (long long row = warp0; row < p.rows; row += nwarps) {
        double rowacc[1] = {0.0};
        for (long long c0 = 0; c0 < p.cols; c0 += 128) {
            const long long ca = c0 + 2 * lane, cb = ca + 64;
            RegFile<NR, kV> f;
            load_row_inputs<NR, ALIGNED>(ch, p, row, ca, cb, f);
            run_chain<NR, kV>(ch, f);
            const bool valid[kV] = {ca < p.cols, ca + 1 < p.cols, cb < p.cols, cb + 1 < p.cols};
            if (AGG == kAggNone) {
                double o[kV];
                operand<NR, kV>(ch, f, ch.out[0], o);
                double *orow = p.out + row * p.cols;
                if (valid[0]) orow[ca] = o[0];
                if (valid[1]) orow[ca + 1] = o[1];
                if (valid[2]) orow[cb] = o[2];
                if (valid[3]) orow[cb + 1] = o[3];
            } else if (AGG == kAggRow) {
                add_outputs<NR>(ch, f, valid, rowacc, 1);
            } else {
                add_outputs<NR>(ch, f, valid, acc, NOUT);
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
            for (int k = 0; k < NOUT; ++k)
                if (k < ch.n_out) p.partials[(size_t)blockIdx.x * ch.n_out + k] = acc[k];
        }
        if (publish_and_is_last(p.head, &s_flag))
            final_sum_small(p.partials, gridDim.x, ch.n_out, p.out, s_red);
    }
}

// ------------------------------------------------------------------ cols
// grid.x: tiles of 512 columns; grid.y: row panels.  A thread owns a column pair
// and walks its panel two rows at a time.
template <int NR, bool ALIGNED>
__global__ void __launch_bounds__(kThreads)
cell_cols_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ CellParams p)
{
    __shared__ unsigned int s_flag;
    const long long col = (long long)blockIdx.x * 512 + 2 * threadIdx.x;
    const long long per = (p.rows + p.panels - 1) / p.panels;
    const long long r0 = (long long)blockIdx.y * per;
    const long long r1 = (r0 + per < p.rows) ? r0 + per : p.rows;
    double a0 = 0.0, a1 = 0.0;

    if (col < p.cols) {
        for (long long row = r0; row < r1; row += 2) {
            const bool two = row + 1 < r1;
            RegFile<NR, kV> f;
            {
                const double2 m0 = load_pair<ALIGNED>(p.X + row * p.ldx, col, p.cols);
                const double2 m1 = two ? load_pair<ALIGNED>(p.X + (row + 1) * p.ldx, col, p.cols)
                                       : make_double2(0.0, 0.0);
                f.r[0][0] = m0.x; f.r[0][1] = m0.y; f.r[0][2] = m1.x; f.r[0][3] = m1.y;
            }
#pragma unroll
            for (int k = 0; k < FO_MAX_SIDES; ++k) {
                if (1 + k < NR && (ch.side_used >> k) & 1u) {
                    const int R = (1 + k < NR) ? 1 + k : 0;
                    const DevSide sd = p.sides.s[k];
                    double2 m0, m1;
                    if (sd.access == FO_AT_ROW) {
                        const double v0 = __ldg(sd.data + row * sd.ld);
                        const double v1 = two ? __ldg(sd.data + (row + 1) * sd.ld) : 0.0;
                        m0 = make_double2(v0, v0);
                        m1 = make_double2(v1, v1);
                    } else if (sd.access == FO_AT_CELL) {
                        m0 = load_pair<ALIGNED>(sd.data + row * sd.ld, col, p.cols);
                        m1 = two ? load_pair<ALIGNED>(sd.data + (row + 1) * sd.ld, col, p.cols)
                                 : make_double2(0.0, 0.0);
                    } else {
                        m0 = make_double2(__ldg(sd.data + col),
                                          col + 1 < p.cols ? __ldg(sd.data + col + 1) : 0.0);
                        m1 = m0;
                    }
                    f.r[R][0] = m0.x; f.r[R][1] = m0.y; f.r[R][2] = m1.x; f.r[R][3] = m1.y;
                }
            }
            run_chain<NR, kV>(ch, f);
            double o[kV];
            operand<NR, kV>(ch, f, ch.out[0], o);
            a0 += o[0];
            a1 += o[1];
            if (two) {
                a0 += o[2];
                a1 += o[3];
            }
        }
        double *pp = p.partials + (size_t)blockIdx.y * p.cols;
        pp[col] = a0;
        if (col + 1 < p.cols) pp[col + 1] = a1;
    }
    if (publish_and_is_last(p.head, &s_flag))
        final_sum_columns(p.partials, p.panels, p.cols, p.out);
}

__global__ void fill_zero_kernel(double *out, long long n)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
         i += (long long)gridDim.x * blockDim.x)
        out[i] = 0.0;
}

// ------------------------------------------------------------------ host
bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

struct CellPlan {
    bool flat;          // flat streaming kernel applies
    bool aligned;       // 128-bit loads are legal in the row / column kernels
    int grid;           // CTAs (flat / rows) or column tiles (cols)
    int panels;         // cols kernel
    size_t ws_need;
};

// Grid of a streaming kernel: every CTA gets work, at most `cap` CTAs.
int stream_grid(long long units, int sms)
{
    const long long cap = (long long)(sms > 0 ? sms : 148) * 8;
    long long g = units < cap ? units : cap;
    if (g > kMaxPartials) g = kMaxPartials;
    if (g < 1) g = 1;
    return (int)g;
}

int col_panels(long long rows, long long cols)
{
    const long long tiles = (cols + 511) / 512;
    long long p = (148 * 8 + tiles - 1) / tiles;
    const long long maxp = (rows + 7) / 8;          // at least 8 rows per panel
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

template <int NR, int NOUT>
cudaError_t launch_cell(const DevChain &ch, const CellParams &p, int agg, bool flat, bool aligned,
                        int grid, cudaStream_t st)
{
    if (agg == FO_CELL_COL_AGG) {
        if constexpr (NOUT == 1) {
            const dim3 g((unsigned)((p.cols + 511) / 512), (unsigned)p.panels);
            if (aligned) cell_cols_kernel<NR, true><<<g, kThreads, 0, st>>>(ch, p);
            else cell_cols_kernel<NR, false><<<g, kThreads, 0, st>>>(ch, p);
        }
    } else if (flat) {
        if (agg == FO_CELL_NO_AGG) {
            if constexpr (NOUT == 1) cell_flat_kernel<NR, 1, true><<<grid, kThreads, 0, st>>>(ch, p);
        } else {
            cell_flat_kernel<NR, NOUT, false><<<grid, kThreads, 0, st>>>(ch, p);
        }
    } else if (agg == FO_CELL_FULL_AGG) {
        if (aligned) cell_rows_kernel<NR, NOUT, kAggFull, true><<<grid, kThreads, 0, st>>>(ch, p);
        else cell_rows_kernel<NR, NOUT, kAggFull, false><<<grid, kThreads, 0, st>>>(ch, p);
    } else if constexpr (NOUT == 1) {
        if (agg == FO_CELL_ROW_AGG) {
            if (aligned) cell_rows_kernel<NR, 1, kAggRow, true><<<grid, kThreads, 0, st>>>(ch, p);
            else cell_rows_kernel<NR, 1, kAggRow, false><<<grid, kThreads, 0, st>>>(ch, p);
        } else {
            if (aligned) cell_rows_kernel<NR, 1, kAggNone, true><<<grid, kThreads, 0, st>>>(ch, p);
            else cell_rows_kernel<NR, 1, kAggNone, false><<<grid, kThreads, 0, st>>>(ch, p);
        }
    }
    return cudaGetLastError();
}

template <int NR>
cudaError_t launch_cell_nr(const DevChain &ch, const CellParams &p, int agg, bool flat,
                           bool aligned, int grid, cudaStream_t st)
{
    if (ch.n_out == 1) return launch_cell<NR, 1>(ch, p, agg, flat, aligned, grid, st);
    if (ch.n_out <= 4) return launch_cell<NR, 4>(ch, p, agg, flat, aligned, grid, st);
    return launch_cell<NR, 8>(ch, p, agg, flat, aligned, grid, st);
}

// Common body of fused_cell and fused_magg.
int run_cell(const fo_chain *chain, const fo_mat *X, const fo_side *sides, int n_sides,
             const double *scalars, int n_scalars, int agg, bool magg, double *out, void *ws,
             size_t ws_bytes, void *stream)
{
    if (!chain || !X || !out) return FO_ERR_NULL;
    if (n_sides > 0 && !sides) return FO_ERR_NULL;
    if (agg < FO_CELL_NO_AGG || agg > FO_CELL_FULL_AGG) return FO_ERR_UNSUPPORTED;
    if (X->kind != FO_DENSE) return (X->kind == FO_CSR) ? FO_ERR_UNSUPPORTED : FO_ERR_SHAPE;
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
        grid = 0;
    } else if (flat) {
        grid = stream_grid((ncells + 1023) >> 10, sms);
    } else {
        grid = stream_grid((xd.rows + 7) / 8, sms);
    }

    cudaError_t e;
    if (ch.n_regs <= 4) e = launch_cell_nr<4>(ch, p, agg, flat, aligned, grid, st);
    else if (ch.n_regs <= 8) e = launch_cell_nr<8>(ch, p, agg, flat, aligned, grid, st);
    else e = launch_cell_nr<kRegs>(ch, p, agg, flat, aligned, grid, st);
    return e == cudaSuccess ? FO_OK : cuda_fail(e);
}

}  // namespace

}  // namespace fo

extern "C" {

size_t fused_cell_workspace_bytes(const fo_mat *X, int agg)
{
    if (!X || X->kind != FO_DENSE || X->dense.rows < 0 || X->dense.cols < 0) return 0;
    if (agg < FO_CELL_NO_AGG || agg > FO_CELL_FULL_AGG) return 0;
    return fo::cell_ws_bytes(X->dense.rows, X->dense.cols, agg, 1);
}

size_t fused_magg_workspace_bytes(const fo_mat *X, int n_out)
{
    if (!X || X->kind != FO_DENSE || n_out < 1 || n_out > FO_MAX_OUT) return 0;
    return fo::cell_ws_bytes(X->dense.rows, X->dense.cols, FO_CELL_FULL_AGG, n_out);
}

int fused_cell(const fo_chain *chain, const fo_mat *X, const fo_side *sides, int n_sides,
               const double *scalars, int n_scalars, int agg, double *out, void *ws,
               size_t ws_bytes, void *stream)
{
    return fo::run_cell(chain, X, sides, n_sides, scalars, n_scalars, agg, false, out, ws,
                        ws_bytes, stream);
}

int fused_magg(const fo_chain *chain, const fo_mat *X, const fo_side *sides, int n_sides,
               const double *scalars, int n_scalars, double *out, void *ws, size_t ws_bytes,
               void *stream)
{
    return fo::run_cell(chain, X, sides, n_sides, scalars, n_scalars, FO_CELL_FULL_AGG, true, out,
                        ws, ws_bytes, stream);
}

}  // extern "C"
