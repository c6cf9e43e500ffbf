// Outer template (Table 1; Fig. 1(d); Eq. 1 and the outer-product listing of
// Section 2.2): for every stored cell (i, j) of the CSR matrix X evaluate
// w = chain(a = X_ij, d = U_i . V_j) and aggregate.  U V^T is never formed.
//
// Schedule: CTAs own contiguous row ranges holding equal shares of the stored
// cells (binary search on rowptr); inside a CTA a warp owns a row at a time.
// The row U_i sits in registers, spread over the 8 lanes of a group; the four
// groups of a warp take different stored cells of the row and gather their V_j
// rows with 128-bit loads (V is read many times and stays in L2).
#include <stdio.h>
#include <stdlib.h>

#include "chain.cuh"

namespace fo {

namespace {

struct OuterParams {
    const int *rowptr;
    const int *colidx;
    const double *vals;
    long long rows, cols, nnz;
    int rank;
    int chain_kind;              // kOuterGeneric or a chain evaluated inline
    const double *U;
    long long ldu;
    const double *V;
    long long ldv;
    WsHead *head;
    double *partials;
    double *out;
    int kconst;                  // constant-table index an inline chain reads
    int pad;
};

enum { kOutFull = 0, kOutNone = 1, kOutRight = 2, kOutLeft = 3 };

// Chains evaluated inline, in the chain's own operation order (same bits as the
// interpreter): the weighted squared loss of Eq. 1, (a != 0) * (a - d)^2, and the
// sparse micro-benchmark expression of Section 5.2, a * log(d + eps).
enum { kOuterGeneric = 0, kOuterWsloss = 1, kOuterXlogd = 2, kOuterMaskDot = 3 };

template <bool ALIGNED>
__device__ __forceinline__ double2 ld_pair_cached(const double *row, int col, int n)
{
    if (col + 1 < n) {
        if (ALIGNED) return __ldg(reinterpret_cast<const double2 *>(row + col));
        return make_double2(__ldg(row + col), __ldg(row + col + 1));
    }
    if (col < n) return make_double2(__ldg(row + col), 0.0);
    return make_double2(0.0, 0.0);
}

__device__ __forceinline__ double outer_chain(const DevChain &ch, int kind, int kc, double a, double d)
{
    if (kind == kOuterWsloss) {
        const double t0 = a != 0.0 ? 1.0 : 0.0;
        const double t1 = a - d;
        const double t2 = t1 * t1;
        return t0 * t2;
    }
    if (kind == kOuterXlogd) return a * slow_log(d + ch.consts[kc]);
    if (kind == kOuterMaskDot) return (a != 0.0 ? 1.0 : 0.0) * d;      // (X != 0) * (U V^T), Eq. 1
    RegFile<kRegs, 1> f;
    f.r[0][0] = a;
    f.r[1][0] = d;
    run_chain<kRegs, 1>(ch, f);
    double o[1];
    operand<kRegs, 1>(ch, f, ch.out[0], o);
    return o[0];
}

// First row r in [0, rows] with rowptr[r] >= target.
__device__ __forceinline__ long long lower_row(const int *rowptr, long long rows, long long target)
{
    long long lo = 0, hi = rows;
    while (lo < hi) {
        const long long mid = (lo + hi) >> 1;
        if (__ldg(rowptr + mid) < target) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// NK2: double2 chunks per lane (rank <= 16 * NK2).
//
// A warp walks its row in chunks of 32 stored cells.  Column indices and values
// of a chunk are loaded one per lane (coalesced); the four 8-lane groups then
// take cells 0-3, 4-7, ... of the chunk, two cells per group and trip, gather
// the V rows and reduce their dot products; each dot product is routed back to
// the lane that holds its cell, so the operator chain runs once per chunk with
// one cell per lane.
template <int NK2, int AGG, bool ALIGNED>
__global__ void __launch_bounds__(kThreads, (NK2 > 8 ? 1 : 2))
outer_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ OuterParams p)
{
    __shared__ double s_red[32];
    __shared__ unsigned int s_flag;
    __shared__ long long s_rows[2];

    if (threadIdx.x == 0) {
        const long long G = gridDim.x, b = blockIdx.x;
        s_rows[0] = (b == 0) ? 0 : lower_row(p.rowptr, p.rows, (p.nnz * b) / G);
        s_rows[1] = (b == G - 1) ? p.rows : lower_row(p.rowptr, p.rows, (p.nnz * (b + 1)) / G);
    }
    __syncthreads();
    const long long row_lo = s_rows[0], row_hi = s_rows[1];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int l8 = lane & 7, grp = lane >> 3;
    const unsigned full = 0xffffffffu;
    const int rank = p.rank;
    double acc = 0.0;

    for (long long row = row_lo + warp; row < row_hi; row += kThreads / 32) {
        const int beg = __ldg(p.rowptr + row), end = __ldg(p.rowptr + row + 1);
        double2 u[NK2], racc[NK2];
        const double *urow = p.U + row * p.ldu;
#pragma unroll
        for (int c = 0; c < NK2; ++c) {
            u[c] = (beg < end) ? ld_pair_cached<ALIGNED>(urow, 16 * c + 2 * l8, rank)
                               : make_double2(0.0, 0.0);
            racc[c] = make_double2(0.0, 0.0);
        }
        for (int c0 = beg; c0 < end; c0 += 32) {
            const int cnt = (end - c0 < 32) ? end - c0 : 32;
            const bool valid = lane < cnt;
            const int jmine = valid ? __ldg(p.colidx + c0 + lane) : 0;
            const double amine = valid ? __ldg(p.vals + c0 + lane) : 0.0;
            double dmine = 0.0;
            const int nit = (cnt + 3) >> 2;
            for (int it = 0; it < nit; it += 2) {
                const int srcA = it * 4 + grp, srcB = srcA + 4;
                const bool actA = srcA < cnt, actB = srcB < cnt;
                const int jA = __shfl_sync(full, jmine, srcA & 31);
                const int jB = __shfl_sync(full, jmine, srcB & 31);
                const double *vA = p.V + (long long)jA * p.ldv;
                const double *vB = p.V + (long long)jB * p.ldv;
                double2 xA[NK2], xB[NK2];
#pragma unroll
                for (int c = 0; c < NK2; ++c) {
                    xA[c] = actA ? ld_pair_cached<ALIGNED>(vA, 16 * c + 2 * l8, rank) : make_double2(0.0, 0.0);
                    xB[c] = actB ? ld_pair_cached<ALIGNED>(vB, 16 * c + 2 * l8, rank) : make_double2(0.0, 0.0);
                }
                double dA = 0.0, dB = 0.0;
#pragma unroll
                for (int c = 0; c < NK2; ++c) {
                    dA = fma(u[c].x, xA[c].x, dA);
                    dA = fma(u[c].y, xA[c].y, dA);
                    dB = fma(u[c].x, xB[c].x, dB);
                    dB = fma(u[c].y, xB[c].y, dB);
                }
                dA += __shfl_xor_sync(full, dA, 4);
                dB += __shfl_xor_sync(full, dB, 4);
                dA += __shfl_xor_sync(full, dA, 2);
                dB += __shfl_xor_sync(full, dB, 2);
                dA += __shfl_xor_sync(full, dA, 1);
                dB += __shfl_xor_sync(full, dB, 1);
                // cell s of the chunk was handled by group (s & 3) in trip (s >> 2)
                const double allA = __shfl_sync(full, dA, (lane & 3) * 8);
                const double allB = __shfl_sync(full, dB, (lane & 3) * 8);
                if ((lane >> 2) == it) dmine = allA;
                if ((lane >> 2) == it + 1) dmine = allB;
            }
            const double w = outer_chain(ch, p.chain_kind, p.kconst, amine, dmine);
            if (AGG == kOutFull) {
                if (valid) acc += w;
            } else if (AGG == kOutNone) {
                if (valid) p.out[c0 + lane] = w;
            } else if (AGG == kOutLeft) {
                // second walk over the chunk: O_j += w_ij * U_i.  Rows of O are shared by
                // all warps, so the additions are global atomics (their order is not fixed).
                for (int it = 0; it < nit; ++it) {
                    const int src = it * 4 + grp;
                    const int j = __shfl_sync(full, jmine, src & 31);
                    const double ww = __shfl_sync(full, w, src & 31);
                    double *oj = p.out + (long long)j * rank;
                    if (src < cnt) {
#pragma unroll
                        for (int c = 0; c < NK2; ++c) {
                            const int col = 16 * c + 2 * l8;
                            if (col < rank) atomicAdd(oj + col, ww * u[c].x);
                            if (col + 1 < rank) atomicAdd(oj + col + 1, ww * u[c].y);
                        }
                    }
                }
            } else {
                // second walk over the chunk: O_i += w_ij * V_j (rows of V come from cache)
                for (int it = 0; it < nit; ++it) {
                    const int src = it * 4 + grp;
                    const bool act = src < cnt;
                    const int j = __shfl_sync(full, jmine, src & 31);
                    const double ww = __shfl_sync(full, w, src & 31);
                    const double *vj = p.V + (long long)j * p.ldv;
                    if (act) {
#pragma unroll
                        for (int c = 0; c < NK2; ++c) {
                            const double2 x = ld_pair_cached<ALIGNED>(vj, 16 * c + 2 * l8, rank);
                            racc[c].x = fma(ww, x.x, racc[c].x);
                            racc[c].y = fma(ww, x.y, racc[c].y);
                        }
                    }
                }
            }
        }
        if (AGG == kOutRight) {
            // the four groups hold partial rows: add them in a fixed order
#pragma unroll
            for (int c = 0; c < NK2; ++c) {
                racc[c].x += __shfl_xor_sync(full, racc[c].x, 8);
                racc[c].y += __shfl_xor_sync(full, racc[c].y, 8);
                racc[c].x += __shfl_xor_sync(full, racc[c].x, 16);
                racc[c].y += __shfl_xor_sync(full, racc[c].y, 16);
                const int col = 16 * c + 2 * l8;
                if (grp == 0) {
                    if (col < rank) p.out[row * rank + col] = racc[c].x;
                    if (col + 1 < rank) p.out[row * rank + col + 1] = racc[c].y;
                }
            }
        }
    }

    if (AGG == kOutFull) {
        double v1[1] = {acc};
        block_sum<1>(v1, s_red);
        if (threadIdx.x == 0) p.partials[blockIdx.x] = v1[0];
        if (publish_and_is_last(p.head, &s_flag))
            final_sum_small(p.partials, gridDim.x, 1, p.out, s_red);
    }
}

// ------------------------------------------------------------------ staged
// The same work with the V rows landing in shared memory first.  A warp owns a
// buffer of 16 rows; for half a chunk (16 stored cells) it issues all the 16-byte
// asynchronous copies of the 16 V rows at once, waits for them, and only then
// forms the dot products from shared memory.  The copies need no registers, so a
// warp keeps 16 rows (12.8 KB at rank 100) in flight instead of 8, and the right_mm
// variant reuses the staged rows instead of gathering them twice.
// Needs 16-byte aligned factor rows and an even rank (a row piece is one 16-byte copy).
constexpr int kStageRows = 16;

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc)
{
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}

template <int NK2, int AGG>
__global__ void __launch_bounds__(kThreads, 2)
outer_staged_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ OuterParams p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ double s_red[32];
    __shared__ unsigned int s_flag;
    __shared__ long long s_rows[2];

    if (threadIdx.x == 0) {
        const long long G = gridDim.x, b = blockIdx.x;
        s_rows[0] = (b == 0) ? 0 : lower_row(p.rowptr, p.rows, (p.nnz * b) / G);
        s_rows[1] = (b == G - 1) ? p.rows : lower_row(p.rowptr, p.rows, (p.nnz * (b + 1)) / G);
    }
    __syncthreads();
    const long long row_lo = s_rows[0], row_hi = s_rows[1];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int l8 = lane & 7, grp = lane >> 3;
    const unsigned full = 0xffffffffu;
    const int rank = p.rank;                       // even
    double *buf = reinterpret_cast<double *>(smem_raw) + (size_t)warp * kStageRows * rank;
    double acc = 0.0;

    for (long long row = row_lo + warp; row < row_hi; row += kThreads / 32) {
        const int beg = __ldg(p.rowptr + row), end = __ldg(p.rowptr + row + 1);
        double2 u[NK2], racc[NK2];
        const double *urow = p.U + row * p.ldu;
#pragma unroll
        for (int c = 0; c < NK2; ++c) {
            const int col = 16 * c + 2 * l8;
            u[c] = (beg < end && col < rank) ? __ldg(reinterpret_cast<const double2 *>(urow + col))
                                             : make_double2(0.0, 0.0);
            racc[c] = make_double2(0.0, 0.0);
        }
        for (int c0 = beg; c0 < end; c0 += 32) {
            const int cnt = (end - c0 < 32) ? end - c0 : 32;
            const bool valid = lane < cnt;
            const int jmine = valid ? __ldg(p.colidx + c0 + lane) : 0;
            const double amine = valid ? __ldg(p.vals + c0 + lane) : 0.0;
            double dmine = 0.0, wmine = 0.0;
            for (int h = 0; h < 2 && 16 * h < cnt; ++h) {
                // land the V rows of cells 16h .. 16h+15: group grp takes cells 16h + 4i + grp
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int sidx = 16 * h + 4 * i + grp;
                    const int j = __shfl_sync(full, jmine, sidx);
                    if (sidx < cnt) {
                        const double *vj = p.V + (long long)j * p.ldv;
                        double *dst = buf + (4 * i + grp) * rank;
#pragma unroll
                        for (int c = 0; c < NK2; ++c) {
                            const int col = 16 * c + 2 * l8;
                            if (col < rank) cp_async16(dst + col, vj + col);
                        }
                    }
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
                asm volatile("cp.async.wait_group 0;" ::: "memory");
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int sidx = 16 * h + 4 * i + grp;
                    const double *src = buf + (4 * i + grp) * rank;
                    double d = 0.0;
                    if (sidx < cnt) {
#pragma unroll
                        for (int c = 0; c < NK2; ++c) {
                            const int col = 16 * c + 2 * l8;
                            if (col < rank) {
                                const double2 x = *reinterpret_cast<const double2 *>(src + col);
                                d = fma(u[c].x, x.x, d);
                                d = fma(u[c].y, x.y, d);
                            }
                        }
                    }
                    d += __shfl_xor_sync(full, d, 4);
                    d += __shfl_xor_sync(full, d, 2);
                    d += __shfl_xor_sync(full, d, 1);
                    // cell s of the chunk was handled by group (s & 3) in trip (s >> 2)
                    const double all = __shfl_sync(full, d, (lane & 3) * 8);
                    if ((lane >> 2) == 4 * h + i) dmine = all;
                }
                if (AGG == kOutRight) {
                    // the chain's values for this half, then O_i += w * V_j from the staged rows
                    const double w = outer_chain(ch, p.chain_kind, p.kconst, amine, dmine);
                    if ((lane >> 4) == h) wmine = w;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int sidx = 16 * h + 4 * i + grp;
                        const double ww = __shfl_sync(full, w, sidx);
                        const double *src = buf + (4 * i + grp) * rank;
                        if (sidx < cnt) {
#pragma unroll
                            for (int c = 0; c < NK2; ++c) {
                                const int col = 16 * c + 2 * l8;
                                if (col < rank) {
                                    const double2 x = *reinterpret_cast<const double2 *>(src + col);
                                    racc[c].x = fma(ww, x.x, racc[c].x);
                                    racc[c].y = fma(ww, x.y, racc[c].y);
                                }
                            }
                        }
                    }
                }
                __syncwarp();          // the buffer is overwritten by the next half
            }
            if (AGG != kOutRight) {
                const double w = outer_chain(ch, p.chain_kind, p.kconst, amine, dmine);
                if (AGG == kOutFull) {
                    if (valid) acc += w;
                } else {
                    if (valid) p.out[c0 + lane] = w;
                }
            }
            (void)wmine;
        }
        if (AGG == kOutRight) {
            // the four groups hold partial rows: add them in a fixed order
#pragma unroll
            for (int c = 0; c < NK2; ++c) {
                racc[c].x += __shfl_xor_sync(full, racc[c].x, 8);
                racc[c].y += __shfl_xor_sync(full, racc[c].y, 8);
                racc[c].x += __shfl_xor_sync(full, racc[c].x, 16);
                racc[c].y += __shfl_xor_sync(full, racc[c].y, 16);
                const int col = 16 * c + 2 * l8;
                if (grp == 0) {
                    if (col < rank) p.out[row * rank + col] = racc[c].x;
                    if (col + 1 < rank) p.out[row * rank + col + 1] = racc[c].y;
                }
            }
        }
    }

    if (AGG == kOutFull) {
        double v1[1] = {acc};
        block_sum<1>(v1, s_red);
        if (threadIdx.x == 0) p.partials[blockIdx.x] = v1[0];
        if (publish_and_is_last(p.head, &s_flag))
            final_sum_small(p.partials, gridDim.x, 1, p.out, s_red);
    }
}

// ---------------------------------------------------------------- pipelined
// full_agg / no_agg: the same staging, software-pipelined inside the warp.  The
// warp's buffer is two halves of eight rows; a step lands the V rows of eight
// stored cells (two per 8-lane group) in one half while the other half is being
// reduced, and the reduction keeps four independent multiply-add chains per lane
// (two cells, two accumulators each) instead of one.  Copy groups are committed
// every step (an empty group at the tail) so that "all but the newest" always
// names the step about to be used.
// NK2 = ceil(rank / 16) exactly: only the last 16-column piece of a row needs a bounds check.
template <int NK2, int AGG>
__global__ void __launch_bounds__(kThreads, 2)
outer_pipe_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ OuterParams p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ double s_red[32];
    __shared__ unsigned int s_flag;
    __shared__ long long s_rows[2];

    if (threadIdx.x == 0) {
        const long long G = gridDim.x, b = blockIdx.x;
        s_rows[0] = (b == 0) ? 0 : lower_row(p.rowptr, p.rows, (p.nnz * b) / G);
        s_rows[1] = (b == G - 1) ? p.rows : lower_row(p.rowptr, p.rows, (p.nnz * (b + 1)) / G);
    }
    __syncthreads();
    const long long row_lo = s_rows[0], row_hi = s_rows[1];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int l8 = lane & 7, grp = lane >> 3;
    const unsigned full = 0xffffffffu;
    const int rank = p.rank;                       // even
    double *buf = reinterpret_cast<double *>(smem_raw) + (size_t)warp * kStageRows * rank;
    double *mybuf = buf + grp * rank + 2 * l8;     // this lane's piece of its group's first row
    double acc = 0.0;

    for (long long row = row_lo + warp; row < row_hi; row += kThreads / 32) {
        const int beg = __ldg(p.rowptr + row), end = __ldg(p.rowptr + row + 1);
        double2 u[NK2];
        const double *urow = p.U + row * p.ldu;
#pragma unroll
        for (int c = 0; c < NK2; ++c) {
            const int col = 16 * c + 2 * l8;
            u[c] = (beg < end && col < rank) ? __ldg(reinterpret_cast<const double2 *>(urow + col))
                                             : make_double2(0.0, 0.0);
        }
        double2 racc[AGG == kOutRight ? NK2 : 1];      // right_mm: this group's share of O_i
#pragma unroll
        for (int c = 0; c < (AGG == kOutRight ? NK2 : 1); ++c) racc[c] = make_double2(0.0, 0.0);
        for (int c0 = beg; c0 < end; c0 += 32) {
            const int cnt = (end - c0 < 32) ? end - c0 : 32;
            const bool valid = lane < cnt;
            const int jmine = valid ? __ldg(p.colidx + c0 + lane) : 0;
            const double amine = valid ? __ldg(p.vals + c0 + lane) : 0.0;
            const int nsteps = (cnt + 7) >> 3;
            double dmine = 0.0;

            // step s: group grp lands the V rows of cells 8 s + grp and 8 s + 4 + grp in
            // half (s & 1) of the buffer.  Past the end of a ragged chunk the chunk's last
            // cell is fetched again: no branch, and its result is never used.
            auto issue = [&](int s) {
                if (s < nsteps) {                     // uniform
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const int sidx = 8 * s + 4 * i + grp;
                        const int j = __shfl_sync(full, jmine, sidx < cnt ? sidx : cnt - 1);
                        const double *vj = p.V + (long long)j * p.ldv + 2 * l8;
                        double *dst = mybuf + ((s & 1) * 8 + 4 * i) * rank;
#pragma unroll
                        for (int c = 0; c < NK2; ++c)
                            if (c < NK2 - 1 || 16 * c + 2 * l8 < rank) cp_async16(dst + 16 * c, vj + 16 * c);
                    }
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
            };
            issue(0);
            for (int s = 0; s < nsteps; ++s) {
                issue(s + 1);
                asm volatile("cp.async.wait_group 1;" ::: "memory");
                __syncwarp();
                // two cells per group, two accumulators per cell: four independent chains
                double dx[2] = {0.0, 0.0}, dy[2] = {0.0, 0.0};
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const double *src = mybuf + ((s & 1) * 8 + 4 * i) * rank;
#pragma unroll
                    for (int c = 0; c < NK2; ++c) {
                        if (c < NK2 - 1 || 16 * c + 2 * l8 < rank) {
                            const double2 x = *reinterpret_cast<const double2 *>(src + 16 * c);
                            dx[i] = fma(u[c].x, x.x, dx[i]);
                            dy[i] = fma(u[c].y, x.y, dy[i]);
                        }
                    }
                }
                const double d0 = dx[0] + dy[0], d1 = dx[1] + dy[1];
                // two values over the 8 lanes of a group in three exchanges: the upper
                // four lanes end up with the second cell's total, the lower four with the first's
                const bool up = (lane & 4) != 0;
                double v = (up ? d1 : d0) + __shfl_xor_sync(full, up ? d0 : d1, 4);
                v += __shfl_xor_sync(full, v, 2);
                v += __shfl_xor_sync(full, v, 1);
                if (AGG == kOutRight) {
                    // the chain for the group's two cells (lower four lanes: the first, upper four:
                    // the second), then O_i += w * V_j from the rows still in the buffer
                    const int sidx = 8 * s + 4 * ((lane >> 2) & 1) + grp;
                    const double a = __shfl_sync(full, amine, sidx & 31);
                    double w = outer_chain(ch, p.chain_kind, p.kconst, a, v);
                    if (sidx >= cnt) w = 0.0;         // a row fetched again at a ragged end adds nothing
                    const double w0 = __shfl_sync(full, w, grp * 8), w1 = __shfl_sync(full, w, grp * 8 + 4);
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const double ww = i ? w1 : w0;
                        const double *src = mybuf + ((s & 1) * 8 + 4 * i) * rank;
#pragma unroll
                        for (int c = 0; c < NK2; ++c) {
                            if (c < NK2 - 1 || 16 * c + 2 * l8 < rank) {
                                const double2 x = *reinterpret_cast<const double2 *>(src + 16 * c);
                                racc[AGG == kOutRight ? c : 0].x = fma(ww, x.x, racc[AGG == kOutRight ? c : 0].x);
                                racc[AGG == kOutRight ? c : 0].y = fma(ww, x.y, racc[AGG == kOutRight ? c : 0].y);
                            }
                        }
                    }
                } else {
                    // cell c of the chunk was handled by group (c & 3) in trip (c >> 2)
                    const double all = __shfl_sync(full, v, (lane & 3) * 8 + ((lane >> 2) & 1) * 4);
                    if ((lane >> 3) == s) dmine = all;
                }
                __syncwarp();          // half (s & 1) is refilled by the issue after next
            }
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            if (AGG != kOutRight) {
                const double w = outer_chain(ch, p.chain_kind, p.kconst, amine, dmine);
                if (AGG == kOutFull) {
                    if (valid) acc += w;
                } else {
                    if (valid) p.out[c0 + lane] = w;
                }
            }
        }
        if (AGG == kOutRight) {
            // the four groups hold partial rows: add them in a fixed order
#pragma unroll
            for (int c = 0; c < (AGG == kOutRight ? NK2 : 1); ++c) {
                racc[c].x += __shfl_xor_sync(full, racc[c].x, 8);
                racc[c].y += __shfl_xor_sync(full, racc[c].y, 8);
                racc[c].x += __shfl_xor_sync(full, racc[c].x, 16);
                racc[c].y += __shfl_xor_sync(full, racc[c].y, 16);
                const int col = 16 * c + 2 * l8;
                if (grp == 0) {
                    if (col < rank) p.out[row * rank + col] = racc[c].x;
                    if (col + 1 < rank) p.out[row * rank + col + 1] = racc[c].y;
                }
            }
        }
    }

    if (AGG == kOutFull) {
        double v1[1] = {acc};
        block_sum<1>(v1, s_red);
        if (threadIdx.x == 0) p.partials[blockIdx.x] = v1[0];
        if (publish_and_is_last(p.head, &s_flag))
            final_sum_small(p.partials, gridDim.x, 1, p.out, s_red);
    }
}

__global__ void outer_fill_zero_kernel(double *out, long long n)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
         i += (long long)gridDim.x * blockDim.x)
        out[i] = 0.0;
}

bool aligned16(const void *q) { return ((uintptr_t)q & 15u) == 0; }

template <int NK2>
cudaError_t launch_outer(const DevChain &ch, const OuterParams &p, int agg, bool aligned, int grid,
                         cudaStream_t st)
{
#define FO_GO(A)                                                                   \
    do {                                                                           \
        if (aligned) outer_kernel<NK2, A, true><<<grid, kThreads, 0, st>>>(ch, p); \
        else outer_kernel<NK2, A, false><<<grid, kThreads, 0, st>>>(ch, p);        \
    } while (0)
    if (agg == FO_OUTER_FULL_AGG) FO_GO(kOutFull);
    else if (agg == FO_OUTER_NO_AGG) FO_GO(kOutNone);
    else if (agg == FO_OUTER_LEFT_MM) FO_GO(kOutLeft);
    else FO_GO(kOutRight);
#undef FO_GO
    return cudaGetLastError();
}

template <int NK2>
cudaError_t launch_outer_staged(const DevChain &ch, const OuterParams &p, int agg, int grid,
                                cudaStream_t st)
{
    const size_t smem = (size_t)(kThreads / 32) * kStageRows * p.rank * sizeof(double);
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<grid, kThreads, smem, st>>>(ch, p);
        return cudaGetLastError();
    };
    if (agg == FO_OUTER_FULL_AGG) return go(outer_staged_kernel<NK2, kOutFull>);
    if (agg == FO_OUTER_NO_AGG) return go(outer_staged_kernel<NK2, kOutNone>);
    return go(outer_staged_kernel<NK2, kOutRight>);
}

// full_agg / no_agg / right_mm through the pipelined kernel; NK2 is exactly ceil(rank / 16).
template <int NK2>
cudaError_t launch_outer_pipe(const DevChain &ch, const OuterParams &p, int agg, int grid, cudaStream_t st)
{
    const size_t smem = (size_t)(kThreads / 32) * kStageRows * p.rank * sizeof(double);
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<grid, kThreads, smem, st>>>(ch, p);
        return cudaGetLastError();
    };
    if (agg == FO_OUTER_FULL_AGG) return go(outer_pipe_kernel<NK2, kOutFull>);
    if (agg == FO_OUTER_NO_AGG) return go(outer_pipe_kernel<NK2, kOutNone>);
    return go(outer_pipe_kernel<NK2, kOutRight>);
}

// Recognises the chains that outer_chain() evaluates inline by the text of the
// translated program's result (chain_expression); multiplication and addition
// commute bit for bit, so both operand orders count.
int outer_chain_kind(const DevChain &ch, int *kconst)
{
    char e[160];
    *kconst = 0;
    if (chain_expression(ch, 0, e, sizeof(e)) != 0) return kOuterGeneric;
    auto match = [&](const char *pattern, int *k) -> bool {
        int n = 0;
        *k = -1;
        return sscanf(e, pattern, k, &n) == 1 && n > 0 && e[n] == 0 && *k >= 0 && *k < kConsts;
    };
    int k;
    if ((match("mul(ne(r0,k%d),mul(sub(r0,r1),sub(r0,r1)))%n", &k) ||
         match("mul(mul(sub(r0,r1),sub(r0,r1)),ne(r0,k%d))%n", &k)) && ch.consts[k] == 0.0)
        return kOuterWsloss;
    if (match("mul(r0,log(add(r1,k%d)))%n", &k) || match("mul(r0,log(add(k%d,r1)))%n", &k) ||
        match("mul(log(add(r1,k%d)),r0)%n", &k) || match("mul(log(add(k%d,r1)),r0)%n", &k)) {
        *kconst = k;
        return kOuterXlogd;
    }
    if ((match("mul(ne(r0,k%d),r1)%n", &k) || match("mul(r1,ne(r0,k%d))%n", &k)) && ch.consts[k] == 0.0)
        return kOuterMaskDot;
    return kOuterGeneric;
}

}  // namespace

}  // namespace fo

extern "C" {

size_t fused_outer_workspace_bytes(const fo_csr *X, int rank, int agg)
{
    if (!X || rank < 0 || rank > 256) return 0;
    if (agg < FO_OUTER_LEFT_MM || agg > FO_OUTER_FULL_AGG) return 0;
    return sizeof(fo::WsHead) + (size_t)fo::kMaxPartials * sizeof(double);
}

int fused_outer(const fo_chain *chain, const fo_csr *X, const fo_dense *U, const fo_dense *V,
                const double *scalars, int n_scalars, int agg, double *out, void *ws,
                size_t ws_bytes, void *stream)
{
    using namespace fo;
    if (!chain || !X || !U || !V || !out) return FO_ERR_NULL;
    if (agg != FO_OUTER_FULL_AGG && agg != FO_OUTER_NO_AGG && agg != FO_OUTER_RIGHT_MM &&
        agg != FO_OUTER_LEFT_MM)
        return FO_ERR_UNSUPPORTED;
    if (X->rows < 0 || X->cols < 0 || X->nnz < 0) return FO_ERR_SHAPE;
    if (X->nnz >= (1ll << 31)) return FO_ERR_UNSUPPORTED;
    if (U->rows != X->rows || V->rows != X->cols || U->cols != V->cols) return FO_ERR_SHAPE;
    if (U->ld < U->cols || V->ld < V->cols) return FO_ERR_SHAPE;
    const int rank = (int)U->cols;
    if (U->cols > 256) return FO_ERR_UNSUPPORTED;
    if (!X->rowptr) return FO_ERR_NULL;
    if (X->nnz > 0 && (!X->colidx || !X->vals)) return FO_ERR_NULL;
    if (rank > 0 && ((X->rows > 0 && !U->data) || (X->cols > 0 && !V->data))) return FO_ERR_NULL;

    DevChain ch;
    int rc = translate_chain(chain, kUseOuter, 0, scalars, n_scalars, 1, 1, &ch);
    if (rc != FO_OK) return rc;
    rc = check_workspace(ws, ws_bytes, fused_outer_workspace_bytes(X, rank, agg));
    if (rc != FO_OK) return rc;

    OuterParams p;
    memset(&p, 0, sizeof(p));
    p.rowptr = X->rowptr; p.colidx = X->colidx; p.vals = X->vals;
    p.rows = X->rows; p.cols = X->cols; p.nnz = X->nnz; p.rank = rank;
    p.U = U->data; p.ldu = U->ld; p.V = V->data; p.ldv = V->ld;
    p.head = (WsHead *)ws;
    p.partials = (double *)((char *)ws + sizeof(WsHead));
    p.out = out;
    p.chain_kind = fo::force_interpreter() ? fo::kOuterGeneric : fo::outer_chain_kind(ch, &p.kconst);
    cudaStream_t st = (cudaStream_t)stream;

    const bool empty = X->nnz == 0 || X->rows == 0;
    if (empty || agg == FO_OUTER_LEFT_MM) {
        // empty sums; left_mm accumulates into a zeroed result
        const long long nout = agg == FO_OUTER_FULL_AGG ? 1
                             : agg == FO_OUTER_RIGHT_MM ? X->rows * rank
                             : agg == FO_OUTER_LEFT_MM ? X->cols * rank : 0;
        if (nout > 0) {
            const long long b = (nout + 255) / 256;
            outer_fill_zero_kernel<<<(unsigned)(b > 1024 ? 1024 : b), 256, 0, st>>>(out, nout);
        }
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(e);
        if (empty) return FO_OK;
    }

    const int sms = sm_count();
    if (sms <= 0) return cuda_fail(cudaErrorNoDevice);
    const bool aligned = aligned16(U->data) && aligned16(V->data) && U->ld % 2 == 0 && V->ld % 2 == 0;
    long long grid = (long long)sms * 8;
    const long long by_rows = (X->rows + 7) / 8;
    if (grid > by_rows) grid = by_rows;
    if (grid > kMaxPartials) grid = kMaxPartials;
    if (grid < 1) grid = 1;

    cudaError_t e;
    const int nk2 = (rank + 15) / 16;
    // factor rows that are 16-byte aligned pieces go through the staged kernel
    const bool staged = aligned && rank % 2 == 0 && rank >= 2 && nk2 <= 8 && agg != FO_OUTER_LEFT_MM &&
                        !getenv("FUSEDOPS_OUTER_DIRECT");
    if (staged) {
        // FUSEDOPS_OUTER_PIPE=0 keeps the batch-at-a-time kernel (a measuring knob)
        const char *pe = getenv("FUSEDOPS_OUTER_PIPE");
        const bool pipe = !(pe && pe[0] == '0');
        if (pipe) {
            switch (nk2) {
                case 1: e = launch_outer_pipe<1>(ch, p, agg, (int)grid, st); break;
                case 2: e = launch_outer_pipe<2>(ch, p, agg, (int)grid, st); break;
                case 3: e = launch_outer_pipe<3>(ch, p, agg, (int)grid, st); break;
                case 4: e = launch_outer_pipe<4>(ch, p, agg, (int)grid, st); break;
                case 5: e = launch_outer_pipe<5>(ch, p, agg, (int)grid, st); break;
                case 6: e = launch_outer_pipe<6>(ch, p, agg, (int)grid, st); break;
                case 7: e = launch_outer_pipe<7>(ch, p, agg, (int)grid, st); break;
                default: e = launch_outer_pipe<8>(ch, p, agg, (int)grid, st); break;
            }
        } else
        if (nk2 <= 1) e = launch_outer_staged<1>(ch, p, agg, (int)grid, st);
        else if (nk2 <= 2) e = launch_outer_staged<2>(ch, p, agg, (int)grid, st);
        else if (nk2 <= 4) e = launch_outer_staged<4>(ch, p, agg, (int)grid, st);
        else if (nk2 <= 7) e = launch_outer_staged<7>(ch, p, agg, (int)grid, st);
        else e = launch_outer_staged<8>(ch, p, agg, (int)grid, st);
        return e == cudaSuccess ? FO_OK : cuda_fail(e);
    }
    if (nk2 <= 1) e = launch_outer<1>(ch, p, agg, aligned, (int)grid, st);
    else if (nk2 <= 2) e = launch_outer<2>(ch, p, agg, aligned, (int)grid, st);
    else if (nk2 <= 4) e = launch_outer<4>(ch, p, agg, aligned, (int)grid, st);
    else if (nk2 <= 7) e = launch_outer<7>(ch, p, agg, aligned, (int)grid, st);
    else if (nk2 <= 8) e = launch_outer<8>(ch, p, agg, aligned, (int)grid, st);
    else e = launch_outer<16>(ch, p, agg, aligned, (int)grid, st);
    return e == cudaSuccess ? FO_OK : cuda_fail(e);
}

}  // extern "C"
