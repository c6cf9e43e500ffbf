// The kernels of the Row template (dense rows through a shared-memory ring, narrow
// dense rows a thread each, CSR rows), written so that they can be compiled ahead
// of time (the chain interpreted, or one of two inline forms) and at run time (the
// chain a generated straight-line functor, FO_JIT_ROW defined): device code only.
#pragma once

#include "common.cuh"
#ifndef FO_JIT_ROW
#include "chain.cuh"
#endif
#include "ptx.cuh"

namespace fo {

struct RowParams {
    const double *X;            // dense
    const int *rowptr;          // CSR
    const int *colidx;
    const double *vals;
    long long rows, cols, ldx;
    const double *v;
    DevSides sides;
    WsHead *head;
    double *partials;
    double *out;
    int stages, rows_per_stage; // dense ring geometry
    int chain_kind;             // kChainGeneric, or a row chain the kernels evaluate inline
    int sides_in_ring;          // dense: used sides are contiguous vectors, staged with the rows
    int out_vec;                // no_agg, dense: rows of `out` can be written 16 bytes at a time
    int rb;                     // CSR: rows a warp takes at a time (32; fewer, a power of two >= 32 / G, for few rows)
};

// Row chains common enough to be evaluated inline instead of interpreted; the
// arithmetic is the same, so are the bits.
enum { kChainGeneric = 0, kChainSideTimesDot = 1, kChainDot = 2 };

enum { kRowColT = 0, kRowRow = 1, kRowFull = 2, kRowNone = 3 };

constexpr int kWarps = kThreads / 32;

#ifdef FO_JIT_ROW
// Run-time specialised build: the chain is the generated straight-line functor
// (in[0] = d, in[1 + k] = side k of the lane's row).
__device__ __forceinline__ double lane_chain(const DevChain &ch, int, double d, const double (&sv)[FO_MAX_SIDES])
{
    const double in[1 + FO_MAX_SIDES] = {d, sv[0], sv[1], sv[2], sv[3]};
    double o[1];
    JitFn::eval(in, ch.consts, o);
    return o[0];
}
#else
// The chain for one row per lane: R0 = d, R(1+k) = side k of that lane's row.
template <int NR>
__device__ __forceinline__ double lane_chain_nr(const DevChain &ch, double d, const double (&sv)[FO_MAX_SIDES])
{
    RegFile<NR, 1> f;
    f.r[0][0] = d;
#pragma unroll
    for (int k = 0; k < FO_MAX_SIDES; ++k)
        if (1 + k < NR) f.r[1 + k < NR ? 1 + k : 0][0] = sv[k];
    run_chain<NR, 1>(ch, f);
    double o[1];
    operand<NR, 1>(ch, f, ch.out[0], o);
    return o[0];
}

// A chain without an inline form runs through the interpreter, out of line: its
// register file would otherwise be counted against every kernel's main loop.
static __device__ __noinline__ double lane_chain_generic(const DevChain &ch, double d, double s0, double s1, double s2,
                                                  double s3)
{
    const double sv[FO_MAX_SIDES] = {s0, s1, s2, s3};
    if (ch.n_regs <= 4) return lane_chain_nr<4>(ch, d, sv);
    return lane_chain_nr<kRegs>(ch, d, sv);
}

__device__ __forceinline__ double lane_chain(const DevChain &ch, int kind, double d,
                                             const double (&sv)[FO_MAX_SIDES])
{
    static_assert(FO_MAX_SIDES == 4, "lane_chain_generic takes four side values");
    if (kind == kChainSideTimesDot) return sv[0] * d;
    if (kind == kChainDot) return d;
    return lane_chain_generic(ch, d, sv[0], sv[1], sv[2], sv[3]);
}
#endif

// ------------------------------------------------------------------ dense
// 512 threads = 16 warps.  W warps form a group that works on R rows at a time;
// warp w of a group owns the 64-column chunks c * W + w (c < NCH) of those rows,
// of v and of the output accumulator - all in registers - so cols <= 64*NCH*W.
// Per stage of the ring: every warp reads its pieces of the R rows, forms R
// partial dot products, reduces them over its lanes (R values in one butterfly)
// and leaves them in shared memory; after ONE CTA barrier - at which point the
// ring slot is free again, the rows being held in registers - lane r of every
// warp adds the W partials of row r in a fixed order, evaluates the chain for
// that row, and the warp adds t_r * X_r into its accumulator columns.
// STAGED: rows arrive through the shared-memory ring; otherwise lanes load
// their pairs straight from global memory (any alignment, any cols).
constexpr int kDenseThreads = 512;                 // compute threads
constexpr int kDenseWarps = kDenseThreads / 32;
constexpr int kDenseBlock = kDenseThreads + 32;    // plus the warp that feeds the ring
constexpr int kDenseMaxSlots = 64;                 // ring slots of all groups together

template <int NCH, int W, int R, int AGG, bool STAGED>
__device__ __forceinline__ void row_dense_body(const DevChain &ch, const RowParams &p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ unsigned long long s_full[kDenseMaxSlots], s_empty[kDenseMaxSlots];
    __shared__ double s_part[2][kDenseWarps][8];     // [parity][warp][row of the group]
    __shared__ double s_red[32];
    __shared__ unsigned int s_flag;

    // The 16 compute warps form GROUPS independent groups of W warps.  A group has
    // its own ring slots, barriers and sequence of tiles (R rows each), so the
    // groups drift apart and one group's barrier and reduction latency is covered
    // by the others' work.
    constexpr int GROUPS = kDenseWarps / W;
    constexpr int SH = 5 - Log2<R>::value;           // lane l holds row (l >> SH) after the butterfly
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool feeder = warp == kDenseWarps;         // warp 16 only moves data
    const int w = warp % W;
    // a feeder lane serves the group of its lane number
    const int grp = feeder ? (lane < GROUPS ? lane : 0) : warp / W;
    const int n = (int)p.cols;
    const int S = p.stages;                          // ring slots per group
    double *ring = reinterpret_cast<double *>(smem_raw) + (size_t)grp * S * R * n;
    // side ring: [group][slot][side][R] doubles behind all the row rings (STAGED only)
    double *side_ring = reinterpret_cast<double *>(smem_raw) + (size_t)GROUPS * S * R * n
                        + (size_t)grp * S * FO_MAX_SIDES * R;
    unsigned long long *full = s_full + grp * S, *empty = s_empty + grp * S;
    const bool ring_sides = STAGED && p.sides_in_ring != 0;

    // tiles of R rows are dealt round-robin to the (CTA, group) pairs
    const long long ntiles = (p.rows + R - 1) / R;
    const long long me = (long long)blockIdx.x * GROUPS + grp, stride = (long long)gridDim.x * GROUPS;
    const long long my_tiles = (ntiles > me) ? (ntiles - me + stride - 1) / stride : 0;

    // this lane's columns: pair (col, col + 1) of chunk c
    double2 vreg[NCH], q[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
        const int col = 64 * (c * W + w) + 2 * lane;
        vreg[c].x = (!feeder && col < n) ? __ldg(p.v + col) : 0.0;
        vreg[c].y = (!feeder && col + 1 < n) ? __ldg(p.v + col + 1) : 0.0;
        q[c] = make_double2(0.0, 0.0);
    }
    double tsum = 0.0;
    bool timed_out = false;

    auto issue = [&](long long it) {
        const int slot = (int)(it % S);
        const long long r0 = (me + it * stride) * R;
        const int nr = (int)((p.rows - r0 < R) ? p.rows - r0 : R);
        double *dst = ring + (size_t)slot * R * n;
        // a ragged last tile with an odd row count cannot be a 16-byte multiple:
        // its side values are read directly (see load_tile_sides)
        const bool with_sides = ring_sides && (nr % 2 == 0);
        unsigned bytes = (unsigned)(nr * n * 8);
        if (with_sides) {
#pragma unroll
            for (int k = 0; k < FO_MAX_SIDES; ++k)
                if ((ch.side_used >> k) & 1u) bytes += (unsigned)(nr * 8);
        }
        mbar_expect_tx(&full[slot], bytes);
        if (p.ldx == n) {
            bulk_g2s(dst, p.X + r0 * p.ldx, (unsigned)(nr * n * 8), &full[slot]);
        } else {
            for (int r = 0; r < nr; ++r)
                bulk_g2s(dst + (size_t)r * n, p.X + (r0 + r) * p.ldx, (unsigned)(n * 8), &full[slot]);
        }
        if (with_sides) {
#pragma unroll
            for (int k = 0; k < FO_MAX_SIDES; ++k)
                if ((ch.side_used >> k) & 1u)
                    bulk_g2s(side_ring + ((size_t)slot * FO_MAX_SIDES + k) * R, p.sides.s[k].data + r0,
                             (unsigned)(nr * 8), &full[slot]);
        }
    };
    // side values of the row this lane evaluates the chain for (lanes 0..R-1),
    // read straight from global memory
    auto load_tile_sides = [&](long long it, double (&sv)[FO_MAX_SIDES]) {
        const long long row = (me + it * stride) * R + lane;
#pragma unroll
        for (int k = 0; k < FO_MAX_SIDES; ++k)
            sv[k] = (lane < R && it < my_tiles && row < p.rows && ((ch.side_used >> k) & 1u))
                        ? __ldg(p.sides.s[k].data + row * p.sides.s[k].ld) : 0.0;
    };

    if (STAGED) {
        if (threadIdx.x == 0) {
            for (int s = 0; s < GROUPS * S; ++s) {
                mbar_init(&s_full[s], 1);
                mbar_init(&s_empty[s], W);
            }
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        __syncthreads();
        // the feeding warp, one lane per group: refill a slot as soon as every warp
        // of the group has taken its pieces of the slot's rows into registers
        if (feeder && lane < GROUPS) {
            for (long long it = 0; it < my_tiles; ++it) {
                if (it >= S && !mbar_wait(&empty[it % S], (unsigned)(((it / S) - 1) & 1))) timed_out = true;
                issue(it);
            }
        }
    }

    for (long long it = 0; it < my_tiles && !feeder; ++it) {
        const long long r0 = (me + it * stride) * R;
        const int slot = (int)(it % S);
        const int par = (int)(it & 1);
        double sv[FO_MAX_SIDES];
        const int nr = (int)((p.rows - r0 < R) ? p.rows - r0 : R);
        // strided or unaligned side vectors (and a ragged odd last tile) cannot ride
        // in the ring: their values are requested here, ahead of the wait
        if (!(ring_sides && nr % 2 == 0)) load_tile_sides(it, sv);
        if (STAGED) {
            if (!mbar_wait(&full[slot], (unsigned)((it / S) & 1))) timed_out = true;
        }
        if (ring_sides && nr % 2 == 0) {
#pragma unroll
            for (int k = 0; k < FO_MAX_SIDES; ++k)
                sv[k] = (lane < R && ((ch.side_used >> k) & 1u))
                            ? side_ring[((size_t)slot * FO_MAX_SIDES + k) * R + lane] : 0.0;
        }
        // rows of this tile into registers, partial dot products
        double2 x[R][NCH];
        double part[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const bool have = r0 + r < p.rows;
            double d0 = 0.0, d1 = 0.0;
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                const int col = 64 * (c * W + w) + 2 * lane;
                if (STAGED) {
                    const double *rowp = ring + ((size_t)slot * R + r) * n;
                    x[r][c] = (have && col < n) ? *reinterpret_cast<const double2 *>(rowp + col)
                                                : make_double2(0.0, 0.0);
                } else {
                    const double *rowp = p.X + (r0 + r) * p.ldx;
                    x[r][c].x = (have && col < n) ? ld_stream1(rowp + col) : 0.0;
                    x[r][c].y = (have && col + 1 < n) ? ld_stream1(rowp + col + 1) : 0.0;
                }
                d0 = fma(x[r][c].x, vreg[c].x, d0);
                d1 = fma(x[r][c].y, vreg[c].y, d1);
            }
            part[r] = d0 + d1;
        }
        // rows and side values are in registers: hand the slot back to the feeder
        if (STAGED) {
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[slot]);
        }
        warp_sum_multi<R>(part, lane);
        if ((lane & ((1 << SH) - 1)) == 0) s_part[par][warp][lane >> SH] = part[0];
        if (W > 1) {
            asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "n"(W * 32) : "memory");   // the group's warps
        } else {
            __syncwarp();
        }
        // lane r: dot product of row r (warps of the group in order), then the chain
        double d = 0.0;
        if (lane < R) {
#pragma unroll
            for (int k = 0; k < W; ++k) d += s_part[par][grp * W + k][lane];
        }
        // (one instance for inline and general chains alike: splitting them, as the CSR kernels do,
        // measured 6 % slower here - 1.23 against 1.16 ms on the same GPU)
        double t;
        if (p.chain_kind == kChainSideTimesDot) {
            t = sv[0] * d;
        } else if (p.chain_kind == kChainDot) {
            t = d;
        } else {
#ifdef FO_JIT_ROW
            t = lane_chain(ch, p.chain_kind, d, sv);      // lane r: the generated chain on row r's values
#else
            // general chain: one warp-wide evaluation per row (lane 0 holds d, lane 1 + k side k)
            t = 0.0;
            for (int r = 0; r < R; ++r) {
                double mine = __shfl_sync(0xffffffffu, d, r);
#pragma unroll
                for (int k = 0; k < FO_MAX_SIDES; ++k) {
                    const double sk = __shfl_sync(0xffffffffu, sv[k], r);
                    if (lane == 1 + k) mine = sk;
                }
                const double tr = warp_chain(ch, mine, lane);
                if (lane == r) t = tr;
            }
#endif
        }
        if (AGG == kRowColT) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const double tr = __shfl_sync(0xffffffffu, t, r);
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    q[c].x = fma(tr, x[r][c].x, q[c].x);
                    q[c].y = fma(tr, x[r][c].y, q[c].y);
                }
            }
        } else if (AGG == kRowNone) {
            // out_i = t_i * X_i, written from the registers that hold the row
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const double tr = __shfl_sync(0xffffffffu, t, r);
                double *orow = p.out + (r0 + r) * (long long)n;
                if (r0 + r < p.rows) {
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        const int col = 64 * (c * W + w) + 2 * lane;
                        if (p.out_vec) {
                            if (col < n)
                                *reinterpret_cast<double2 *>(orow + col) = make_double2(tr * x[r][c].x, tr * x[r][c].y);
                        } else {
                            if (col < n) orow[col] = tr * x[r][c].x;
                            if (col + 1 < n) orow[col + 1] = tr * x[r][c].y;
                        }
                    }
                }
            }
        } else {
            const long long row = r0 + lane;
            if (w == 0 && lane < R && row < p.rows) {
                if (AGG == kRowRow) p.out[row] = t;
                else tsum += t;
            }
        }
    }

    if (STAGED && timed_out) atomicExch(&p.head->status, 1u);

    if (AGG == kRowColT) {
        // groups -> CTA: fixed order over groups, through shared memory
        __syncthreads();
        double *qs = reinterpret_cast<double *>(smem_raw);      // GROUPS * n doubles
        const int cgrp = warp / W;
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            const int col = 64 * (c * W + w) + 2 * lane;
            if (!feeder && col < n) qs[(size_t)cgrp * n + col] = q[c].x;
            if (!feeder && col + 1 < n) qs[(size_t)cgrp * n + col + 1] = q[c].y;
        }
        __syncthreads();
        for (int j = threadIdx.x; j < n; j += kDenseBlock) {
            double s = 0.0;
#pragma unroll
            for (int g = 0; g < GROUPS; ++g) s += qs[(size_t)g * n + j];
            p.partials[(size_t)blockIdx.x * n + j] = s;
        }
        reduce_columns_two_level(p.head, p.partials, p.partials + (size_t)gridDim.x * n, n, p.out,
                                 &s_flag);
    } else if (AGG == kRowFull) {
        double v1[1] = {tsum};
        block_sum<1>(v1, s_red);
        if (threadIdx.x == 0) p.partials[blockIdx.x] = v1[0];
        if (publish_and_is_last(p.head, &s_flag))
            final_sum_small(p.partials, gridDim.x, 1, p.out, s_red);
    }
}

// ----------------------------------------------------------- dense, narrow
// Rows of at most NC <= 32 columns (the tall, narrow matrices of the paper's
// end-to-end runs: 10^8 x 10): a row is too short to spread over a warp, so a
// thread takes whole rows.  It loads its row (16-byte loads when the layout
// allows), forms the dot product with v (in registers up to 16 columns, from the
// cache beyond), evaluates the chain
// and keeps the n output sums in registers; the CTA adds them up in a fixed order
// at the end.  Neighbouring lanes read neighbouring rows, so a warp's loads cover
// one contiguous piece of X between them and every fetched sector is used.
constexpr int kNarrowMax = 32;

template <int NC, int AGG, bool VEC>
__device__ __forceinline__ void row_narrow_body(const DevChain &ch, const RowParams &p)
{
    __shared__ double s_red[NC * 32];
    __shared__ unsigned int s_flag;
    const int n = (int)p.cols;
    constexpr bool VREG = NC <= 16;               // beyond that v is read through the cache (one address per warp)
    double v[VREG ? NC : 1], q[NC];
#pragma unroll
    for (int j = 0; j < NC; ++j) {
        if (VREG) v[VREG ? j : 0] = j < n ? __ldg(p.v + j) : 0.0;
        q[j] = 0.0;
    }
    double tsum = 0.0;
    const long long stride = (long long)gridDim.x * kThreads;
    for (long long row = (long long)blockIdx.x * kThreads + threadIdx.x; row < p.rows; row += stride) {
        const double *xr = p.X + row * p.ldx;
        double x[NC];
        if (VEC) {
#pragma unroll
            for (int j = 0; j < NC; j += 2) {
                double2 t2 = make_double2(0.0, 0.0);
                // n even: the pair is inside the row.  Cached in L1 on purpose: a 32-byte sector
                // holds two of these pairs, and the second request should not go back to L2
                if (j < n) t2 = __ldg(reinterpret_cast<const double2 *>(xr + j));
                x[j] = t2.x;
                x[j + 1] = t2.y;
            }
        } else {
#pragma unroll
            for (int j = 0; j < NC; ++j) x[j] = j < n ? ld_stream1(xr + j) : 0.0;
        }
        double sv[FO_MAX_SIDES];
#pragma unroll
        for (int k = 0; k < FO_MAX_SIDES; ++k)
            sv[k] = ((ch.side_used >> k) & 1u) ? __ldg(p.sides.s[k].data + row * p.sides.s[k].ld) : 0.0;
        double d0 = 0.0, d1 = 0.0;
#pragma unroll
        for (int j = 0; j < NC; j += 2) {
            const double va = VREG ? v[VREG ? j : 0] : (j < n ? __ldg(p.v + j) : 0.0);
            const double vb = VREG ? v[VREG ? j + 1 : 0] : (j + 1 < n ? __ldg(p.v + j + 1) : 0.0);
            d0 = fma(x[j], va, d0);
            d1 = fma(x[j + 1], vb, d1);
        }
        const double t = lane_chain(ch, p.chain_kind, d0 + d1, sv);
        if (AGG == kRowColT) {
#pragma unroll
            for (int j = 0; j < NC; ++j) q[j] = fma(t, x[j], q[j]);
        } else if (AGG == kRowRow) {
            p.out[row] = t;
        } else if (AGG == kRowFull) {
            tsum += t;
        } else {
            double *orow = p.out + row * (long long)n;
#pragma unroll
            for (int j = 0; j < NC; ++j)
                if (j < n) orow[j] = t * x[j];
        }
    }
    if (AGG == kRowColT) {
        block_sum<NC>(q, s_red);
        if (threadIdx.x == 0) {
#pragma unroll
            for (int j = 0; j < NC; ++j)
                if (j < n) p.partials[(size_t)blockIdx.x * n + j] = q[j];
        }
        reduce_columns_two_level(p.head, p.partials, p.partials + (size_t)gridDim.x * n, n, p.out, &s_flag);
    } else if (AGG == kRowFull) {
        double v1[1] = {tsum};
        block_sum<1>(v1, s_red);
        if (threadIdx.x == 0) p.partials[blockIdx.x] = v1[0];
        if (publish_and_is_last(p.head, &s_flag))
            final_sum_small(p.partials, gridDim.x, 1, p.out, s_red);
    }
}

// -------------------------------------------------------------------- CSR
// col_t_agg / col_agg.  A warp takes blocks of 32 consecutive rows.  Row
// offsets, side values and the chain are handled one row per lane (coalesced loads, one chain evaluation for
// 32 rows); the block's stored cells - one contiguous piece of colidx / vals -
// are first copied into the warp's slice of shared memory with coalesced loads.
// Then G lanes share a row (G = 2 .. 32 by the matrix's mean row length, so
// that a row takes a few trips): 32 / G rows at a time, every group walks its
// row with the same, warp-uniform trip count - dot product against v (shared
// memory), then the scatter  acc[col] += t * val  into the CTA's shared
// accumulator.  Two lanes may hit the same column at the same time, so
// the scatter uses shared-memory atomics (their order is not fixed).
constexpr int kCsrStage = 512;            // stored cells a warp can stage per block of rows

template <int G, bool GENERIC>
__device__ __forceinline__ void row_csr_body(const DevChain &ch, const RowParams &p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ unsigned int s_flag;
    const long long n = p.cols;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lg = lane & (G - 1), grp = lane / G;

    double *vs = reinterpret_cast<double *>(smem_raw);
    double *qs = vs + n;
    double *sx = vs + 2 * n + (size_t)warp * kCsrStage;
    int *sc = reinterpret_cast<int *>(vs + 2 * n + (size_t)kWarps * kCsrStage) + (size_t)warp * kCsrStage;
    for (long long j = threadIdx.x; j < n; j += kThreads) {
        vs[j] = __ldg(p.v + j);
        qs[j] = 0.0;
    }
    __syncthreads();

    const int RB = p.rb;
    const int nit = G * RB / 32;                     // >= 1: RB >= 32 / G
    const long long nblocks = (p.rows + RB - 1) / RB;
    const long long warp0 = (long long)blockIdx.x * kWarps + warp;
    const long long nwarps = (long long)gridDim.x * kWarps;

    for (long long blk = warp0; blk < nblocks; blk += nwarps) {
        const long long myrow = blk * RB + lane;
        const bool have = lane < RB && myrow < p.rows;
        const int beg_l = have ? __ldg(p.rowptr + myrow) : 0;
        const int end_l = have ? __ldg(p.rowptr + myrow + 1) : beg_l;
        double sv[FO_MAX_SIDES];
#pragma unroll
        for (int k = 0; k < FO_MAX_SIDES; ++k)
            sv[k] = (have && ((ch.side_used >> k) & 1u))
                        ? __ldg(p.sides.s[k].data + myrow * p.sides.s[k].ld) : 0.0;

        // stage the block's stored cells (skipped, and read from global memory
        // below, when the block holds more than the slice can take)
        const int base = __shfl_sync(0xffffffffu, beg_l, 0);
        const int last_end = __shfl_sync(0xffffffffu, end_l, (int)((p.rows - blk * RB < RB) ? p.rows - blk * RB - 1 : RB - 1));
        const int total = last_end - base;
        const bool staged = total <= kCsrStage;
        if (staged) {
            for (int e = lane; e < total; e += 32) {
                sc[e] = __ldg(p.colidx + base + e);
                sx[e] = __ldg(p.vals + base + e);
            }
        }
        __syncwarp();

        // G lanes per row: 32 / G rows at a time, G trips
        double dmine = 0.0;
#pragma unroll 1
        for (int it = 0; it < nit; ++it) {
            const int rr = it * (32 / G) + grp;
            const int beg = __shfl_sync(0xffffffffu, beg_l, rr);
            const int end = __shfl_sync(0xffffffffu, end_l, rr);
            double d = 0.0;
            if (staged) {
                // the same trip count in all groups: no divergent loop
                const int trips = __reduce_max_sync(0xffffffffu, (end - beg + G - 1) / G);
                int q0 = beg - base + lg;
                const int qe = end - base;
                for (int s = 0; s < trips; ++s, q0 += G) {
                    const bool ok = q0 < qe;
                    const int qq = ok ? q0 : 0;
                    const double x = ok ? sx[qq] : 0.0;
                    d = fma(x, vs[sc[qq]], d);
                }
            } else {
                for (int q0 = beg + lg; q0 < end; q0 += G)
                    d = fma(__ldg(p.vals + q0), vs[__ldg(p.colidx + q0)], d);
            }
#pragma unroll
            for (int o = G / 2; o >= 1; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
            // row rr's dot product sits in group (rr mod groups); lane rr keeps it
            const double dall = __shfl_sync(0xffffffffu, d, (lane & (32 / G - 1)) * G);
            if (lane / (32 / G) == it) dmine = dall;
        }
        // (an instance either carries the interpreter or the two inline forms)
        const double t = GENERIC ? lane_chain(ch, kChainGeneric, dmine, sv)
                                 : (p.chain_kind == kChainDot ? dmine : sv[0] * dmine);
#pragma unroll 1
        for (int it = 0; it < nit; ++it) {
            const int rr = it * (32 / G) + grp;
            const int beg = __shfl_sync(0xffffffffu, beg_l, rr);
            const int end = __shfl_sync(0xffffffffu, end_l, rr);
            const double tt = __shfl_sync(0xffffffffu, t, rr);
            if (staged) {
                const int trips = __reduce_max_sync(0xffffffffu, (end - beg + G - 1) / G);
                int q0 = beg - base + lg;
                const int qe = end - base;
                for (int s = 0; s < trips; ++s, q0 += G)
                    if (q0 < qe) atomicAdd(&qs[sc[q0]], tt * sx[q0]);
            } else {
                for (int q0 = beg + lg; q0 < end; q0 += G)
                    atomicAdd(&qs[__ldg(p.colidx + q0)], tt * __ldg(p.vals + q0));
            }
        }
        __syncwarp();          // the slice is reused by the next block
    }

    __syncthreads();
    for (long long j = threadIdx.x; j < n; j += kThreads)
        p.partials[(size_t)blockIdx.x * n + j] = qs[j];
    reduce_columns_two_level(p.head, p.partials, p.partials + (size_t)gridDim.x * n, n, p.out, &s_flag);
}

// row_agg / full_agg / no_agg: the stored cells kept in registers instead of a staged
// slice.  G lanes share a row and 32 / G rows are worked on at a time, as above,
// but every lane loads its cells of the row (every G-th one, up to kCsrRegCells of
// them) straight from global memory into registers - neighbouring rows are
// neighbours in colidx / vals, so the warp's loads cover one contiguous piece and
// the sectors it touches are used up over the trips - forms its share of the dot
// product from v in shared memory, and after the group's sum and the chain
// (evaluated by every lane of the group for its row) writes t, adds it up, or
// writes  t * val  from the same registers.  Nothing is staged and nothing is read
// twice; longer rows finish in a loop that reads global memory again.  (For the
// column scatter this form measured slower than the staged one above: 0.87 against
// 0.82 ms on 1e7 x 1000 at density 0.01.)
constexpr int kCsrRegCells = 8;

template <int AGG, int G, bool GENERIC>
__device__ __forceinline__ void row_csr_reg_body(const DevChain &ch, const RowParams &p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ double s_red[32];
    __shared__ unsigned int s_flag;
    const long long n = p.cols;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lg = lane & (G - 1), grp = lane / G;
    const unsigned full = 0xffffffffu;

    double *vs = reinterpret_cast<double *>(smem_raw);
    for (long long j = threadIdx.x; j < n; j += kThreads) vs[j] = __ldg(p.v + j);
    __syncthreads();

    const int RB = p.rb;
    const int nit = G * RB / 32;                     // >= 1: RB >= 32 / G
    const long long nblocks = (p.rows + RB - 1) / RB;
    const long long warp0 = (long long)blockIdx.x * kWarps + warp;
    const long long nwarps = (long long)gridDim.x * kWarps;
    double tsum = 0.0;

    for (long long blk = warp0; blk < nblocks; blk += nwarps) {
        const long long myrow = blk * RB + lane;
        const bool have = lane < RB && myrow < p.rows;
        const int beg_l = have ? __ldg(p.rowptr + myrow) : 0;
        const int end_l = have ? __ldg(p.rowptr + myrow + 1) : beg_l;
        double sv[FO_MAX_SIDES];
#pragma unroll
        for (int k = 0; k < FO_MAX_SIDES; ++k)
            sv[k] = (have && ((ch.side_used >> k) & 1u))
                        ? __ldg(p.sides.s[k].data + myrow * p.sides.s[k].ld) : 0.0;
        // a set of 32 / G rows: its cells in registers
        struct Cells {
            int beg, end, trips;
            int cj[kCsrRegCells];
            double cx[kCsrRegCells];
        };
        auto load_cells = [&](int it, Cells &c) {
            const int rr = it * (32 / G) + grp;
            c.beg = __shfl_sync(full, beg_l, rr);
            c.end = __shfl_sync(full, end_l, rr);
            // the same trip count in all groups: no divergent loop
            c.trips = __reduce_max_sync(full, (c.end - c.beg + G - 1) / G);
            if (c.trips > kCsrRegCells) c.trips = kCsrRegCells;
#pragma unroll
            for (int s = 0; s < kCsrRegCells; ++s) {
                c.cj[s] = 0;
                c.cx[s] = 0.0;
                if (s < c.trips) {                   // uniform
                    const int q = c.beg + lg + G * s;
                    if (q < c.end) {
                        c.cj[s] = __ldg(p.colidx + q);
                        c.cx[s] = __ldg(p.vals + q);
                    }
                }
            }
        };
        auto process = [&](int it, const Cells &c) {
            const int rr = it * (32 / G) + grp;
            const int beg = c.beg, end = c.end, trips = c.trips;
            double d = 0.0;
#pragma unroll
            for (int s = 0; s < kCsrRegCells; ++s)
                if (s < trips) d = fma(c.cx[s], vs[c.cj[s]], d);
            for (int q = beg + lg + G * kCsrRegCells; q < end; q += G)
                d = fma(__ldg(p.vals + q), vs[__ldg(p.colidx + q)], d);
#pragma unroll
            for (int o = G / 2; o >= 1; o >>= 1) d += __shfl_xor_sync(full, d, o);
            // every lane of the group runs the chain for the group's row
            double svr[FO_MAX_SIDES];
#pragma unroll
            for (int k = 0; k < FO_MAX_SIDES; ++k)
                svr[k] = ((ch.side_used >> k) & 1u) ? __shfl_sync(full, sv[k], rr) : 0.0;
            const double t = GENERIC ? lane_chain(ch, kChainGeneric, d, svr)
                                     : (p.chain_kind == kChainDot ? d : svr[0] * d);
            const bool live = rr < RB && blk * RB + rr < p.rows;
            if (AGG == kRowRow) {
                if (live && lg == 0) p.out[blk * RB + rr] = t;
            } else if (AGG == kRowFull) {
                if (live && lg == 0) tsum += t;
            } else {
                // out has X's pattern: stored cell q of row i becomes t_i * vals[q]
#pragma unroll
                for (int s = 0; s < kCsrRegCells; ++s)
                    if (s < trips && beg + lg + G * s < end) p.out[beg + lg + G * s] = t * c.cx[s];
                for (int q = beg + lg + G * kCsrRegCells; q < end; q += G) p.out[q] = t * __ldg(p.vals + q);
            }
        };
#pragma unroll 1
        for (int it = 0; it < nit; ++it) {
            Cells a;
            load_cells(it, a);
            process(it, a);
        }
    }

    if (AGG == kRowFull) {
        double v1[1] = {tsum};
        block_sum<1>(v1, s_red);
        if (threadIdx.x == 0) p.partials[blockIdx.x] = v1[0];
        if (publish_and_is_last(p.head, &s_flag))
            final_sum_small(p.partials, gridDim.x, 1, p.out, s_red);
    }
}

template <int NCH, int W, int R, int AGG, bool STAGED>
__global__ void __launch_bounds__(kDenseBlock, 1)
row_dense_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ RowParams p)
{
    row_dense_body<NCH, W, R, AGG, STAGED>(ch, p);
}

template <int NC, int AGG, bool VEC>
__global__ void __launch_bounds__(kThreads)
row_narrow_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ RowParams p)
{
    row_narrow_body<NC, AGG, VEC>(ch, p);
}

template <int G, bool GENERIC>
__global__ void __launch_bounds__(kThreads, 3)
row_csr_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ RowParams p)
{
    row_csr_body<G, GENERIC>(ch, p);
}

template <int AGG, int G, bool GENERIC>
__global__ void __launch_bounds__(kThreads, 3)
row_csr_reg_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ RowParams p)
{
    row_csr_reg_body<AGG, G, GENERIC>(ch, p);
}

}  // namespace fo
