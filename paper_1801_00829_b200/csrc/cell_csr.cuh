// The kernel of the Cell / MAgg templates over a CSR main input (the sparse-safe
// binding), written so that it can be compiled ahead of time and at run time:
// device code only, depending on cell_flat.cuh.
#pragma once

#include "cell_flat.cuh"

namespace fo {

struct CsrCellParams {
    const int *rowptr;
    const int *colidx;
    const double *vals;
    long long rows, cols;
    DevSides sides;
    WsHead *head;
    double *partials;
    double *out;
    int agg;                 // FO_CELL_*
    int rb;                  // rows a warp takes at a time: 32, fewer (a power of two >= 32 / G) for small inputs
    // sparse sides (access == kAtCellSparse): sides.s[k].data holds the values
    const int *side_rowptr[FO_MAX_SIDES];
    const int *side_colidx[FO_MAX_SIDES];
};

constexpr int kAtCellSparse = 3;      // a CSR side input read at (row, column); 0.0 where it stores nothing

// Value of a CSR side at column j of a row whose stored cells are [sb, se):
// binary search in the row's ascending column indices.
__device__ __forceinline__ double sparse_side_value(const int *colidx, const double *vals, int sb, int se, int j)
{
    int lo = sb, hi = se;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(colidx + mid) < j) lo = mid + 1;
        else hi = mid;
    }
    return (lo < se && __ldg(colidx + lo) == j) ? __ldg(vals + lo) : 0.0;
}

template <class EVAL, int NOUT, int G>
__device__ __forceinline__ void cell_csr_body(const DevChain &ch, const CsrCellParams &p)
{
    __shared__ double s_red[NOUT * 32];
    __shared__ unsigned int s_flag;
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int lg = lane & (G - 1), grp = lane / G;
    const int agg = p.agg;
    double acc[NOUT];
#pragma unroll
    for (int k = 0; k < NOUT; ++k) acc[k] = 0.0;

    const int RB = p.rb;
    const long long nblocks = (p.rows + RB - 1) / RB;
    const long long warp0 = (long long)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    const long long nwarps = (long long)gridDim.x * (kThreads / 32);
    const int nit = G * RB / 32;                     // >= 1: RB >= 32 / G

    for (long long blk = warp0; blk < nblocks; blk += nwarps) {
        const long long myrow = blk * RB + (lane < RB ? lane : RB);     // lanes past the block: an empty row
        const int beg_l = __ldg(p.rowptr + (myrow < p.rows ? myrow : p.rows));
        const int end_l = (lane < RB) ? __ldg(p.rowptr + (myrow + 1 < p.rows ? myrow + 1 : p.rows)) : beg_l;
#pragma unroll 1
        for (int it = 0; it < nit; ++it) {
            const int rr = it * (32 / G) + grp;
            const long long row = blk * RB + rr;
            const int beg = __shfl_sync(full, beg_l, rr);
            const int end = __shfl_sync(full, end_l, rr);
            const int trips = __reduce_max_sync(full, (end - beg + G - 1) / G);
            // sides indexed by the row: one value for the whole row
            double srow[FO_MAX_SIDES];
#pragma unroll
            for (int k = 0; k < FO_MAX_SIDES; ++k)
                srow[k] = (EVAL::uses_side(ch, k) && p.sides.s[k].access == FO_AT_ROW && beg < end)
                              ? __ldg(p.sides.s[k].data + row * p.sides.s[k].ld) : 0.0;
            // sparse sides: the row's piece of the side's cells
            int ssb[FO_MAX_SIDES], sse[FO_MAX_SIDES];
#pragma unroll
            for (int k = 0; k < FO_MAX_SIDES; ++k) {
                const bool sp = EVAL::uses_side(ch, k) && p.sides.s[k].access == kAtCellSparse && beg < end;
                ssb[k] = sp ? __ldg(p.side_rowptr[k] + row) : 0;
                sse[k] = sp ? __ldg(p.side_rowptr[k] + row + 1) : 0;
            }
            double rowacc = 0.0;
            int q = beg + lg;
            for (int s = 0; s < trips; ++s, q += G) {
                const bool ok = q < end;
                const int j = ok ? __ldg(p.colidx + q) : 0;
                double in[kIn][1];
                in[0][0] = ok ? __ldg(p.vals + q) : 0.0;
#pragma unroll
                for (int k = 0; k < FO_MAX_SIDES; ++k) {
                    double v = 0.0;
                    if (EVAL::uses_side(ch, k)) {
                        const DevSide sd = p.sides.s[k];
                        if (sd.access == FO_AT_ROW) v = srow[k];
                        else if (sd.access == kAtCellSparse) {
                            if (ok) v = sparse_side_value(p.side_colidx[k], sd.data, ssb[k], sse[k], j);
                        } else if (ok) v = __ldg(sd.data + (sd.access == FO_AT_CELL ? row * sd.ld + j : (long long)j));
                    }
                    in[1 + k][0] = v;
                }
                double o[NOUT][1];
                EVAL::template run<1, NOUT>(ch, in, o);
                if (agg == FO_CELL_FULL_AGG) {
#pragma unroll
                    for (int k = 0; k < NOUT; ++k) acc[k] += ok ? o[k][0] : 0.0;
                } else if (agg == FO_CELL_ROW_AGG) {
                    rowacc += ok ? o[0][0] : 0.0;
                } else if (agg == FO_CELL_NO_AGG) {
                    if (ok) p.out[q] = o[0][0];
                } else {
                    if (ok) atomicAdd(p.out + j, o[0][0]);
                }
            }
            if (agg == FO_CELL_ROW_AGG) {
#pragma unroll
                for (int o2 = G / 2; o2 >= 1; o2 >>= 1) rowacc += __shfl_xor_sync(full, rowacc, o2);
                if (lg == 0 && row < p.rows) p.out[row] = rowacc;
            }
        }
    }

    if (agg == FO_CELL_FULL_AGG) {
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

template <class EVAL, int NOUT, int G>
__global__ void __launch_bounds__(kThreads)
cell_csr_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ CsrCellParams p)
{
    cell_csr_body<EVAL, NOUT, G>(ch, p);
}

}  // namespace fo
