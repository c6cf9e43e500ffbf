// The row-wise and column-wise kernels of the Cell / MAgg templates over a dense
// main input (general layouts: leading dimensions, row / column vector sides;
// row_agg, col_agg), written - like the flat kernel - so that they can be compiled
// ahead of time and at run time: device code only, depending on cell_flat.cuh.
#pragma once

#include "cell_flat.cuh"

namespace fo {

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
__device__ __forceinline__ void cell_rows_body(const DevChain &ch, const CellParams &p)
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
__device__ __forceinline__ void cell_cols_body(const DevChain &ch, const CellParams &p)
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

template <class EVAL, int NOUT, int AGG, bool ALIGNED>
__global__ void __launch_bounds__(kThreads)
cell_rows_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ CellParams p)
{
    cell_rows_body<EVAL, NOUT, AGG, ALIGNED>(ch, p);
}

template <class EVAL, bool ALIGNED>
__global__ void __launch_bounds__(kThreads)
cell_cols_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ CellParams p)
{
    cell_cols_body<EVAL, ALIGNED>(ch, p);
}

}  // namespace fo
