// The kernels of the Outer template, written so that they can be compiled ahead of
// time (the chain interpreted, or one of a few inline forms) and at run time (the
// chain a generated straight-line functor, FO_JIT_OUTER defined): device code only.
#pragma once

#include "common.cuh"
#include "ptx.cuh"
#ifndef FO_JIT_OUTER
#include "chain.cuh"
#endif

namespace fo {

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
    DevSides sides;              // dense side inputs read at the stored cell (outer_kernel only)
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

#ifdef FO_JIT_OUTER
// Run-time specialised build: the chain is the generated straight-line functor.
template <bool OUT_OF_LINE = false>
__device__ __forceinline__ double outer_chain(const DevChain &ch, int, int, double a, double d)
{
    const double in[2 + kOuterMaxSides] = {a, d, 0.0, 0.0, 0.0};
    double o[1];
    JitFn::eval(in, ch.consts, o);
    return o[0];
}
template <bool GENERIC>
__device__ __forceinline__ double outer_chain_split(const DevChain &ch, int kind, int kc, double a, double d)
{
    return outer_chain(ch, kind, kc, a, d);
}
template <int KIND>
__device__ __forceinline__ double outer_chain_fixed(const DevChain &ch, int kc, double a, double d)
{
    return outer_chain(ch, KIND, kc, a, d);
}
__device__ __forceinline__ double outer_chain_sides(const DevChain &ch, double a, double d,
                                                    const double (&sv)[kOuterMaxSides])
{
    const double in[2 + kOuterMaxSides] = {a, d, sv[0], sv[1], sv[2]};
    double o[1];
    JitFn::eval(in, ch.consts, o);
    return o[0];
}
#else
// The interpreter for a chain without an inline form: R0 = a, R1 = d, R(2 + k) = side k.
__device__ __forceinline__ double outer_chain_sides(const DevChain &ch, double a, double d,
                                                    const double (&sv)[kOuterMaxSides])
{
    RegFile<kRegs, 1> f;
    f.r[0][0] = a;
    f.r[1][0] = d;
#pragma unroll
    for (int k = 0; k < kOuterMaxSides; ++k) f.r[2 + k][0] = sv[k];
    run_chain<kRegs, 1>(ch, f);
    double o[1];
    operand<kRegs, 1>(ch, f, ch.out[0], o);
    return o[0];
}

// The same, out of line: for a kernel whose main loop should not carry the
// interpreter's register file.
static __device__ __noinline__ double outer_chain_interp_call(const DevChain &ch, double a, double d)
{
    const double none[kOuterMaxSides] = {0.0, 0.0, 0.0};
    return outer_chain_sides(ch, a, d, none);
}

template <bool OUT_OF_LINE = false>
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
    if (OUT_OF_LINE) return outer_chain_interp_call(ch, a, d);
    const double none[kOuterMaxSides] = {0.0, 0.0, 0.0};
    return outer_chain_sides(ch, a, d, none);
}

// The same with the choice made at compile time: a kernel instance either carries the
// interpreter (GENERIC) or the inline forms, not both - the inline forms' instance then
// needs fewer registers.
template <bool GENERIC>
__device__ __forceinline__ double outer_chain_split(const DevChain &ch, int kind, int kc, double a, double d)
{
    if (GENERIC) {
        const double none[kOuterMaxSides] = {0.0, 0.0, 0.0};
        return outer_chain_sides(ch, a, d, none);
    }
    if (kind == kOuterXlogd) return a * slow_log(d + ch.consts[kc]);
    if (kind == kOuterMaskDot) return (a != 0.0 ? 1.0 : 0.0) * d;
    const double t0 = a != 0.0 ? 1.0 : 0.0;       // kOuterWsloss
    const double t1 = a - d;
    const double t2 = t1 * t1;
    return t0 * t2;
}

// The form of the chain fixed at compile time: the instance carries exactly one of them.
template <int KIND>
__device__ __forceinline__ double outer_chain_fixed(const DevChain &ch, int kc, double a, double d)
{
    if (KIND == kOuterGeneric) {
        const double none[kOuterMaxSides] = {0.0, 0.0, 0.0};
        return outer_chain_sides(ch, a, d, none);
    }
    if (KIND == kOuterXlogd) return a * slow_log(d + ch.consts[kc]);
    if (KIND == kOuterMaskDot) return (a != 0.0 ? 1.0 : 0.0) * d;
    const double t0 = a != 0.0 ? 1.0 : 0.0;       // kOuterWsloss
    const double t1 = a - d;
    const double t2 = t1 * t1;
    return t0 * t2;
}
#endif

// First row r in [0, rows] with rowptr[r] >= target, found by the 32 lanes of a
// warp together: 32 probes a round.
__device__ __forceinline__ long long lower_row_warp(const int *rowptr, long long rows, long long target,
                                                    int lane)
{
    long long lo = 0, hi = rows;
    while (lo < hi) {
        const long long step = (hi - lo + 31) / 32;
        const long long idx = lo + step * lane;
        const bool below = idx < hi && __ldg(rowptr + idx) < target;     // true for a prefix of the lanes
        const int c = __popc(__ballot_sync(0xffffffffu, below));
        if (c == 0) {
            hi = lo;
        } else {
            const long long nhi = lo + step * c;
            lo = lo + step * (c - 1) + 1;
            if (nhi < hi) hi = nhi;
        }
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
__device__ __forceinline__ void outer_body(const DevChain &ch, const OuterParams &p)
{
    __shared__ double s_red[32];
    __shared__ unsigned int s_flag;
    __shared__ long long s_rows[2];

    if (threadIdx.x < 64) {       // warps 0 and 1 find the CTA's first and last row, 32 probes a round
        const long long G = gridDim.x, b = blockIdx.x + (threadIdx.x >> 5);
        const long long r = (b == 0) ? 0 : (b == G) ? p.rows
                            : lower_row_warp(p.rowptr, p.rows, (p.nnz * b) / G, threadIdx.x & 31);
        if ((threadIdx.x & 31) == 0) s_rows[threadIdx.x >> 5] = r;
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
            double w;
            if (ch.side_used) {
                // side inputs at this lane's cell (i, j): a matrix at (i, j), a column vector at i,
                // a row vector at j
                double sv[kOuterMaxSides];
#pragma unroll
                for (int k = 0; k < kOuterMaxSides; ++k) {
                    sv[k] = 0.0;
                    if (valid && ((ch.side_used >> k) & 1u)) {
                        const DevSide sd = p.sides.s[k];
                        sv[k] = sd.access == FO_AT_ROW ? __ldg(sd.data + row * sd.ld)
                              : sd.access == FO_AT_COL ? __ldg(sd.data + jmine)
                                                       : __ldg(sd.data + row * sd.ld + jmine);
                    }
                }
                w = outer_chain_sides(ch, amine, dmine, sv);
            } else {
                w = outer_chain(ch, p.chain_kind, p.kconst, amine, dmine);
            }
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

constexpr int kStageRows = 16;

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc)
{
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
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
template <int NK2, int AGG, bool GENERIC>
__device__ __forceinline__ void outer_pipe_body(const DevChain &ch, const OuterParams &p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ double s_red[32];
    __shared__ unsigned int s_flag;
    __shared__ long long s_rows[2];

    if (threadIdx.x < 64) {       // warps 0 and 1 find the CTA's first and last row, 32 probes a round
        const long long G = gridDim.x, b = blockIdx.x + (threadIdx.x >> 5);
        const long long r = (b == 0) ? 0 : (b == G) ? p.rows
                            : lower_row_warp(p.rowptr, p.rows, (p.nnz * b) / G, threadIdx.x & 31);
        if ((threadIdx.x & 31) == 0) s_rows[threadIdx.x >> 5] = r;
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
        // X and U stream from HBM once: ask the L2 now for what this warp's next row will read first
        // (its U row, and the head of its cells), so that those loads find it there
        {
            const long long nrow = row + kThreads / 32;
            if (nrow < row_hi) {
                const int nb = __ldg(p.rowptr + nrow);
                const char *pu = reinterpret_cast<const char *>(p.U + nrow * p.ldu);
                const char *pc = reinterpret_cast<const char *>(p.colidx + nb);
                const char *pv = reinterpret_cast<const char *>(p.vals + nb);
                const char *what = lane < 8 ? pu + 128 * lane : lane < 12 ? pc + 128 * (lane - 8) : pv + 128 * (lane - 12);
                const bool ok = lane < 8 ? 128 * lane < rank * 8 : lane < 12 ? nb + 32 * (lane - 8) < p.nnz
                                                                 : lane < 20 && nb + 16 * (lane - 12) < p.nnz;
                if (ok) asm volatile("prefetch.global.L2 [%0];" ::"l"(what));
            }
        }
        double2 racc[AGG == kOutRight ? NK2 : 1];      // right_mm: this group's share of O_i
#pragma unroll
        for (int c = 0; c < (AGG == kOutRight ? NK2 : 1); ++c) racc[c] = make_double2(0.0, 0.0);
        // the cells of a chunk arrive a chunk ahead
        int jnext = (beg + lane < end) ? __ldg(p.colidx + beg + lane) : 0;
        double anext = (beg + lane < end) ? __ldg(p.vals + beg + lane) : 0.0;
        for (int c0 = beg; c0 < end; c0 += 32) {
            const int cnt = (end - c0 < 32) ? end - c0 : 32;
            const bool valid = lane < cnt;
            const int jmine = jnext;
            const double amine = anext;
            if (c0 + 32 + lane < end) {
                jnext = __ldg(p.colidx + c0 + 32 + lane);
                anext = __ldg(p.vals + c0 + 32 + lane);
            } else {
                jnext = 0;
                anext = 0.0;
            }
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
                    double w = outer_chain_split<GENERIC>(ch, p.chain_kind, p.kconst, a, v);
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
                const double w = outer_chain_split<GENERIC>(ch, p.chain_kind, p.kconst, amine, dmine);
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

// --------------------------------------------------------------------- bulk
// full_agg / no_agg with the factor rows landed by the bulk-copy engine.  Every warp
// owns a contiguous range of rows holding an equal share of the stored cells and
// works through it in stages of up to eight cells of one row.  A stage's V rows are
// fetched by ONE bulk copy each (a lane per copy, so one instruction starts them all)
// into a slot of the warp's private two-slot ring and counted on the slot's mbarrier;
// the warp never waits for anyone but its own copies (every wait bounded).  Column
// indices and values run ahead of the copies through a small ring in shared memory,
// filled 32 cells at a time; U_i is read at a row's first stage, having been requested
// from L2 when that stage's copies were started.
// Starting a bulk copy holds the issuing warp for about 54 cycles per row, whatever the
// row's length, so this schedule needs many warps (16 fit with rows of up to 108
// doubles, 13 at 128) and long rows; where it is chosen over the 16-byte asynchronous
// copies of outer_pipe_kernel is decided, from measurements, by the host code.
constexpr int kBulkWarps = 16;       // warps per CTA, one CTA per SM
constexpr int kBulkDepth = 2;        // slots per ring
constexpr int kBulkRing = 64;        // cells of (colidx, vals) kept per warp
constexpr int kBulkCells = 8;        // cells per stage

__host__ __device__ inline size_t bulk_warp_bytes(int rank)
{
    return (size_t)kBulkDepth * kBulkCells * rank * 8 + kBulkRing * 12 + kBulkDepth * 16;
}

template <int NK2, int AGG, int KIND>
__device__ __forceinline__ void outer_bulk_body(const DevChain &ch, const OuterParams &p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ unsigned long long s_bar[kBulkWarps * kBulkDepth];
    __shared__ double s_red[32];
    __shared__ unsigned int s_flag;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int W = blockDim.x >> 5;
    constexpr int D = kBulkDepth;
    const int l8 = lane & 7, grp = lane >> 3;
    const unsigned full = 0xffffffffu;
    const int rank = p.rank;                           // even
    const unsigned rowbytes = (unsigned)rank * 8u;
    const int slot_doubles = kBulkCells * rank;        // a stage's V rows
    unsigned char *base = smem_raw + (size_t)warp * bulk_warp_bytes(rank);
    double *slots = reinterpret_cast<double *>(base);
    double *aring = slots + (size_t)D * slot_doubles;
    int *jring = reinterpret_cast<int *>(aring + kBulkRing);
    int4 *meta = reinterpret_cast<int4 *>(jring + kBulkRing);
    unsigned long long *bar = s_bar + warp * kBulkDepth;

    if (lane == 0) {
        for (int s = 0; s < D; ++s) mbar_init(&bar[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const long long GW = (long long)gridDim.x * W, gw = (long long)blockIdx.x * W + warp;
    const long long row_lo = gw == 0 ? 0 : lower_row_warp(p.rowptr, p.rows, (p.nnz * gw) / GW, lane);
    const long long row_hi = gw == GW - 1 ? p.rows : lower_row_warp(p.rowptr, p.rows, (p.nnz * (gw + 1)) / GW, lane);
    const long long P0 = __ldg(p.rowptr + row_lo), P1 = __ldg(p.rowptr + row_hi);

    // (colidx, vals) ring: cells [.., S) relative to P0 are in shared memory, the chunk
    // [S, S + 32) is on its way in registers
    int S = 0, jn = 0;
    double an = 0.0;
    auto load_chunk = [&]() {
        const long long pp = P0 + S + lane;
        if (pp < P1) {
            jn = __ldg(p.colidx + pp);
            an = __ldg(p.vals + pp);
        }
    };
    auto store_chunk = [&]() {
        jring[(S + lane) & (kBulkRing - 1)] = jn;
        aring[(S + lane) & (kBulkRing - 1)] = an;
        S += 32;
    };
    load_chunk();
    store_chunk();
    load_chunk();
    __syncwarp();

    long long irow = row_lo, ipos = P0, iend = P0;
    bool ifirst = true;
    auto next_row = [&]() {
        while (irow < row_hi) {
            iend = __ldg(p.rowptr + irow + 1);
            if (iend > ipos) break;
            ++irow;
        }
    };
    next_row();
    auto issue = [&](int slot) {
        const int q = (int)(ipos - P0);
        const int cnt = (iend - ipos < kBulkCells) ? (int)(iend - ipos) : kBulkCells;
        if (q + cnt > S) {
            store_chunk();
            load_chunk();
            __syncwarp();
        }
        const int j = lane < cnt ? jring[(q + lane) & (kBulkRing - 1)] : 0;
        if (lane == 0) {
            meta[slot] = make_int4(q, cnt | (ifirst ? 0x100 : 0), (int)(irow - row_lo), 0);
            mbar_expect_tx(&bar[slot], (unsigned)cnt * rowbytes);
        }
        __syncwarp();
        double *sl = slots + (size_t)slot * slot_doubles;
        if (lane < cnt) bulk_g2s(sl + lane * rank, p.V + (long long)j * p.ldv, rowbytes, &bar[slot]);
        else if (ifirst && lane >= 16 && 128 * (lane - 16) < rank * 8 && irow + 1 < row_hi)
            // U streams from HBM once: ask the L2 for the NEXT row's U_i now, a row of stages ahead of its use
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char *>(p.U + (irow + 1) * p.ldu) + 128 * (lane - 16)));
        ipos += cnt;
        ifirst = false;
        if (ipos == iend) {
            ++irow;
            next_row();
            ifirst = true;
        }
    };

    if (irow < row_hi && 128 * lane < rank * 8)       // the first row's U_i
        asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char *>(p.U + irow * p.ldu) + 128 * lane));
    int issued = 0;
    while (issued < D && irow < row_hi) issue(issued++);

    double2 u[NK2];
#pragma unroll
    for (int c = 0; c < NK2; ++c) u[c] = make_double2(0.0, 0.0);
    double acc = 0.0;
    bool timed_out = false;
    // A chain that costs more than a few instructions (the interpreter, a logarithm) runs once per
    // four stages, a cell per lane: stage number sb of a batch leaves its cells' values and dot
    // products with lanes 8 sb .. 8 sb + 7.  The cheap inline forms run per stage on the lanes that
    // hold the totals (measured 2 % faster for them, 15 % slower for the logarithm).
    constexpr bool BATCH = (KIND == kOuterGeneric || KIND == kOuterXlogd);
    double pa = 0.0, pd = 0.0;
    int ppos = -1;                                    // this lane's pending cell (position behind P0), or none
    int sb = 0;
    auto flush = [&]() {
        const double w = outer_chain_fixed<KIND>(ch, p.kconst, pa, pd);
        if (AGG == kOutFull) {
            if (ppos >= 0) acc += w;
        } else {
            if (ppos >= 0) p.out[P0 + ppos] = w;
        }
        ppos = -1;
        sb = 0;
    };

    const int tcell = grp + 4 * ((lane >> 2) & 1);    // the stage's cell whose total this lane ends up with
    const bool holder = (lane & 3) == 0;
    int cslot = 0, inflight = issued;
    unsigned cphase = 0;
    while (inflight > 0) {
        const int4 m = meta[cslot];
        const int q = m.x, cnt = m.y & 0xff;
        const bool first = (m.y & 0x100) != 0;
        // the value of the cell this lane will run the chain for: cell l8 of the stage if the chain is
        // batched, else the cell whose total the lane ends up with
        const double a = aring[(q + (BATCH ? l8 : tcell)) & (kBulkRing - 1)];
        if (!__all_sync(full, mbar_wait_hint(&bar[cslot], cphase, 2000u))) {      // the whole warp leaves together
            timed_out = true;
            break;
        }
        const double *sl = slots + (size_t)cslot * slot_doubles;
        if (first) {
            const double *us = p.U + (row_lo + m.z) * p.ldu;
#pragma unroll
            for (int c = 0; c < NK2; ++c)
                if (c < NK2 - 1 || 16 * c + 2 * l8 < rank)
                    u[c] = __ldg(reinterpret_cast<const double2 *>(us + 16 * c + 2 * l8));
        }
        double dx[2] = {0.0, 0.0}, dy[2] = {0.0, 0.0};
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const double *src = sl + (grp + 4 * i) * rank + 2 * l8;
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
        // two values over the 8 lanes of a group: the lower four lanes end up with the total of
        // cell grp, the upper four with that of cell grp + 4
        const bool up = (lane & 4) != 0;
        double v = (up ? d1 : d0) + __shfl_xor_sync(full, up ? d0 : d1, 4);
        v += __shfl_xor_sync(full, v, 2);
        v += __shfl_xor_sync(full, v, 1);
        if (BATCH) {
            // cell c of the stage goes to lane 8 sb + c: its total sits in group c & 3, half c >> 2
            const double vv = __shfl_sync(full, v, 8 * (lane & 3) + 4 * ((lane >> 2) & 1));
            if ((lane >> 3) == sb) {
                pd = vv;
                pa = a;
                ppos = l8 < cnt ? q + l8 : -1;
            }
            if (++sb == 4) flush();
        } else {
            const double w = outer_chain_split<false>(ch, p.chain_kind, p.kconst, a, v);    // an inline form
            if (AGG == kOutFull) {
                if (holder && tcell < cnt) acc += w;
            } else {
                if (holder && tcell < cnt) p.out[P0 + q + tcell] = w;
            }
        }
        __syncwarp();                  // everyone is done with the slot: refill it
        --inflight;
        if (irow < row_hi) {
            issue(cslot);
            ++inflight;
        }
        if (++cslot == D) {
            cslot = 0;
            cphase ^= 1u;
        }
    }
    if (!timed_out && sb > 0) flush();
    if (timed_out) {
        // give the copies still in flight a (bounded) chance to land before the CTA's
        // shared memory is given up
        for (int k = 0; k < inflight; ++k) {
            mbar_wait(&bar[cslot], cphase);
            if (++cslot == D) {
                cslot = 0;
                cphase ^= 1u;
            }
        }
        if (lane == 0) atomicExch(&p.head->status, 1u);
    }

    if (AGG == kOutFull) {
        double v1[1] = {acc};
        block_sum<1>(v1, s_red);
        if (threadIdx.x == 0) p.partials[blockIdx.x] = v1[0];
        if (publish_and_is_last(p.head, &s_flag))
            final_sum_small(p.partials, gridDim.x, 1, p.out, s_red);
    }
}

template <int NK2, int AGG, int KIND>
__global__ void __launch_bounds__(kBulkWarps * 32, 1)
outer_bulk_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ OuterParams p)
{
    outer_bulk_body<NK2, AGG, KIND>(ch, p);
}

// -------------------------------------------------------------------- dense
// full_agg / no_agg for a main input that stores a large share of its cells
// (Section 5.2, "Outer-Product Operations": the dense end of the sparsity sweep).
// Gathering a factor row per stored cell then costs more than forming U V^T
// outright, so this schedule forms it, tile by tile, and never writes it out:
// a CTA takes a block of 64 rows (U rows in shared memory) and sweeps 32-column
// tiles of V.  Its warps have two jobs.  Eight of them form the 64 x 32 tile of
// dot products with the fp64 tensor-core instruction (mma.sync m8n8k4, a 16 x 16
// piece per warp) and leave it in one of two tile buffers in shared memory; eight
// others take the previous tile from the other buffer and evaluate its stored
// cells - a contiguous piece of each row of the CSR matrix, found with a per-row
// cursor: they pick their dot product from the buffer and run the chain.  So the
// cell work, which mostly waits for X to stream in from HBM, runs under the
// tensor-core work instead of between it.  The groups hand the buffers over with
// named barriers (full / empty per buffer: arrive on one side, sync on the
// other; both sides execute the same tile loop, so the counts always meet).  The
// V tiles are double-buffered too: the copy of the next one runs under the
// products of this one.  Work items are (row block, column range) pairs dealt
// round-robin to one CTA per SM.
constexpr int kDenseBM = 64, kDenseBN = 32;
constexpr int kDenseMmaWarps = 8, kDenseCellWarps = 8;
constexpr int kDenseThreadsAll = (kDenseMmaWarps + kDenseCellWarps) * 32;

__host__ __device__ inline int dense_ld(int rank)
{
    int ld = (rank + 3) & ~3;            // whole steps of 4
    while ((ld & 7) != 4) ld += 4;       // 4 (mod 8): the 8 x 4 fragment reads touch every bank once
    return ld;
}
__host__ __device__ inline size_t dense_smem_bytes(int rank)
{
    return (size_t)((kDenseBM + 2 * kDenseBN) * dense_ld(rank) + 2 * kDenseBM * (kDenseBN + 2)) * sizeof(double);
}

__device__ __forceinline__ void dmma_8x8x4(double &c0, double &c1, double a, double b)
{
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                 : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}

// Named barriers of the tiled kernel (0 is __syncthreads).
__device__ __forceinline__ void named_sync(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void named_arrive(int id, int threads)
{
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

struct DenseSplit {
    int row_blocks, col_splits, tiles_per_split, pad;
};

template <int AGG>
__device__ __forceinline__ void outer_dense_body(const DevChain &ch, const OuterParams &p, const DenseSplit &sp)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ double s_red[32];
    __shared__ unsigned int s_flag;

    const int rank = p.rank, ld = dense_ld(rank);
    constexpr int PLD = kDenseBN + 2;
    constexpr int kMma = kDenseMmaWarps * 32;                     // threads that form the tiles
    constexpr int kBarMma = 1, kBarFull = 2, kBarEmpty = 4;       // named barriers: + buffer number
    double *Us = reinterpret_cast<double *>(smem_raw);            // 64 x ld
    double *Vs = Us + kDenseBM * ld;                              // 2 x 32 x ld
    double *Ps = Vs + 2 * kDenseBN * ld;                          // 2 x 64 x 34

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool mma_warp = warp < kDenseMmaWarps;
    const unsigned full = 0xffffffffu;
    const int pieces = rank >> 1;                                 // 16-byte pieces of a factor row

    // columns rank .. ld - 1 of the operand buffers stay zero for good
    for (int i = threadIdx.x; i < (kDenseBM + 2 * kDenseBN) * (ld - rank); i += kDenseThreadsAll) {
        const int r = i / (ld - rank), c = rank + i % (ld - rank);
        Us[(size_t)r * ld + c] = 0.0;            // r runs over the rows of Us and then of both Vs
    }
    __syncthreads();

    double acc = 0.0;
    const long long items = (long long)sp.row_blocks * sp.col_splits;
    const long long ntiles = (p.cols + kDenseBN - 1) / kDenseBN;
    long long n = 0;                             // tiles this CTA has been through: buffer n & 1

    if (mma_warp) {
        const int g = lane >> 2, t = lane & 3;                    // fragment coordinates
        const int wm = warp >> 1, wn = warp & 1;                  // warp tile: rows 16 wm .., columns 16 wn ..
        auto copy_rows = [&](double *dst, int nrows, const double *src, long long ldsrc, long long first,
                             long long limit) {
            // rows first .. first + nrows - 1 of a factor (those below `limit`) into dst
            for (int i = threadIdx.x; i < nrows * pieces; i += kMma) {
                const int r = i / pieces, c = i % pieces;
                if (first + r < limit) cp_async16(dst + (size_t)r * ld + 2 * c, src + (first + r) * ldsrc + 2 * c);
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        for (long long item = blockIdx.x; item < items; item += gridDim.x) {
            const long long row0 = (item / sp.col_splits) * kDenseBM;
            const long long tile_lo = (item % sp.col_splits) * sp.tiles_per_split;
            const long long tile_hi = tile_lo + sp.tiles_per_split < ntiles ? tile_lo + sp.tiles_per_split : ntiles;
            named_sync(kBarMma, kMma);                            // the last products on the old U block are done
            copy_rows(Us, kDenseBM, p.U, p.ldu, row0, p.rows);
            copy_rows(Vs + (size_t)(n & 1) * kDenseBN * ld, kDenseBN, p.V, p.ldv, tile_lo * kDenseBN, p.cols);
            for (long long tile = tile_lo; tile < tile_hi; ++tile, ++n) {
                const int b = (int)(n & 1);
                asm volatile("cp.async.wait_group 0;" ::: "memory");
                named_sync(kBarMma, kMma);                        // this V tile (and U) landed; the other V buffer is free
                if (tile + 1 < tile_hi)
                    copy_rows(Vs + (size_t)(b ^ 1) * kDenseBN * ld, kDenseBN, p.V, p.ldv, (tile + 1) * kDenseBN, p.cols);
                // ---- P = U_blk V_tile^T: warp tile 16 x 16 = 2 x 2 instruction tiles
                double c[2][2][2];
#pragma unroll
                for (int i = 0; i < 2; ++i)
#pragma unroll
                    for (int j = 0; j < 2; ++j) c[i][j][0] = c[i][j][1] = 0.0;
                const double *ua = Us + (size_t)(16 * wm + g) * ld + t;
                const double *vb = Vs + (size_t)b * kDenseBN * ld + (size_t)(16 * wn + g) * ld + t;
#pragma unroll 4
                for (int k = 0; k < ld; k += 4) {
                    double a[2], bb[2];
#pragma unroll
                    for (int i = 0; i < 2; ++i) a[i] = ua[(size_t)(8 * i) * ld + k];
#pragma unroll
                    for (int j = 0; j < 2; ++j) bb[j] = vb[(size_t)(8 * j) * ld + k];
#pragma unroll
                    for (int i = 0; i < 2; ++i)
#pragma unroll
                        for (int j = 0; j < 2; ++j) dmma_8x8x4(c[i][j][0], c[i][j][1], a[i], bb[j]);
                }
                if (n >= 2) named_sync(kBarEmpty + b, kDenseThreadsAll);   // the cells of tile n - 2 are done with this buffer
                double *pb = Ps + (size_t)b * kDenseBM * PLD;
#pragma unroll
                for (int i = 0; i < 2; ++i)
#pragma unroll
                    for (int j = 0; j < 2; ++j)
                        *reinterpret_cast<double2 *>(pb + (size_t)(16 * wm + 8 * i + g) * PLD + 16 * wn + 8 * j + 2 * t) =
                            make_double2(c[i][j][0], c[i][j][1]);
                __threadfence_block();
                named_arrive(kBarFull + b, kDenseThreadsAll);     // the tile is there
            }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    } else {
        const int cw = warp - kDenseMmaWarps;                     // cell warp 0 .. 7: rows 8 cw .. 8 cw + 7
        for (long long item = blockIdx.x; item < items; item += gridDim.x) {
            const long long row0 = (item / sp.col_splits) * kDenseBM;
            const long long tile_lo = (item % sp.col_splits) * sp.tiles_per_split;
            const long long tile_hi = tile_lo + sp.tiles_per_split < ntiles ? tile_lo + sp.tiles_per_split : ntiles;
            // per-row cursors of this warp's rows (lane r keeps row r's): the first stored cell at or
            // right of the column range's start, and the row's end
            int mycur = 0, myend = 0;
            if (lane < 8) {
                const long long row = row0 + 8 * cw + lane;
                if (row < p.rows) {
                    mycur = __ldg(p.rowptr + row);
                    myend = __ldg(p.rowptr + row + 1);
                    const int want = (int)(tile_lo * kDenseBN);
                    int hi = myend;
                    while (mycur < hi) {
                        const int mid = (mycur + hi) >> 1;
                        if (__ldg(p.colidx + mid) < want) mycur = mid + 1; else hi = mid;
                    }
                }
            }
            // the cells of a tile: a lane per cell at its offset from the row's cursor.  Their loads do
            // not need the tile, and where the next tile's cells start is known as soon as this tile's
            // column indices are: so the loads run a tile ahead of the chains.
            int jj[8], jn[8], pos[8];
            double aa[8], an[8];
            auto load_cells = [&](int (&j8)[8], double (&a8)[8]) {
#pragma unroll
                for (int rr = 0; rr < 8; ++rr) {
                    const int pp = __shfl_sync(full, mycur, rr) + lane;
                    j8[rr] = 0x7fffffff;
                    a8[rr] = 0.0;
                    if (pp < __shfl_sync(full, myend, rr)) {
                        j8[rr] = __ldg(p.colidx + pp);
                        a8[rr] = __ldg(p.vals + pp);
                    }
                }
            };
            load_cells(jn, an);
            for (long long tile = tile_lo; tile < tile_hi; ++tile, ++n) {
                const int b = (int)(n & 1);
                const int n0 = (int)(tile * kDenseBN), nhi = n0 + kDenseBN;
#pragma unroll
                for (int rr = 0; rr < 8; ++rr) {
                    jj[rr] = jn[rr];
                    aa[rr] = an[rr];
                    pos[rr] = __shfl_sync(full, mycur, rr) + lane;
                    // the row's cells in this tile are a prefix of what was loaded: move the cursor past them
                    const int taken = __popc(__ballot_sync(full, jj[rr] < nhi));
                    if (lane == rr) mycur += taken;
                }
                if (tile + 1 < tile_hi) load_cells(jn, an);       // the next tile's cells, under this tile's chains
                named_sync(kBarFull + b, kDenseThreadsAll);       // tile n is in buffer b
                const double *pb = Ps + (size_t)b * kDenseBM * PLD;
#pragma unroll
                for (int rr = 0; rr < 8; ++rr) {
                    if (jj[rr] < nhi) {
                        const double w = outer_chain<true>(ch, p.chain_kind, p.kconst, aa[rr],
                                                           pb[(size_t)(8 * cw + rr) * PLD + (jj[rr] - n0)]);
                        if (AGG == kOutFull) acc += w;
                        else p.out[pos[rr]] = w;
                    }
                }
                __syncwarp();
                named_arrive(kBarEmpty + b, kDenseThreadsAll);    // done with the buffer
            }
        }
    }
    __syncthreads();

    if (AGG == kOutFull) {
        double v1[1] = {acc};
        block_sum<1>(v1, s_red);
        if (threadIdx.x == 0) p.partials[blockIdx.x] = v1[0];
        if (publish_and_is_last(p.head, &s_flag))
            final_sum_small(p.partials, gridDim.x, 1, p.out, s_red);
    }
}

template <int NK2, int AGG, bool ALIGNED>
__global__ void __launch_bounds__(kThreads, (NK2 > 8 ? 1 : 2))
outer_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ OuterParams p)
{
    outer_body<NK2, AGG, ALIGNED>(ch, p);
}

template <int NK2, int AGG, bool GENERIC>
__global__ void __launch_bounds__(kThreads, 2)
outer_pipe_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ OuterParams p)
{
    outer_pipe_body<NK2, AGG, GENERIC>(ch, p);
}

template <int AGG>
__global__ void __launch_bounds__(kDenseThreadsAll, 1)
outer_dense_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ OuterParams p,
                   const __grid_constant__ DenseSplit sp)
{
    outer_dense_body<AGG>(ch, p, sp);
}

}  // namespace fo
