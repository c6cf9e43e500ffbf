// Row template with matrix-valued row intermediates (Table 1: no_agg_B1 /
// col_agg_B1; Eq. 2 and its row-wise listing in Section 2.2; Section 5.2 "Row
// Operations", t(X) %*% (X %*% V)).  Per row i of a dense X and a side matrix
// B (n x k):  D_i = X_i B  (k values),  s_i = sum_c pre(D_ic),  T_ic = post(D_ic, s_i),
// then  out += X_i^T T_i  (n x k)  or  out[i] = T_i.
// Four kernels: tensor-core tiles (row_b1_mma_kernel), multiply-add tiles
// (row_b1_kernel, described next), a thread per row for narrow matrices
// (row_b1_narrow_kernel) and CSR rows (row_b1_csr_kernel).
//
// The row is read from HBM once.  A CTA's 16 warps form independent groups; a
// group streams its tiles of R rows through its own shared-memory ring with
// bulk asynchronous copies (bounded waits): once the group's barrier of a tile
// has been passed every warp holds its pieces of the tile in registers, so one
// elected lane refills that slot right away - nobody waits for a free slot.  Inside a group W warps
// split the columns and KW warps split the k classes into slices of KL; a lane
// keeps its column pairs of the tile's rows in registers for both uses, takes
// B (transposed, zero-padded) from shared memory, and owns the output
// accumulators of (its columns) x (its class slice) in registers.
#include <stdio.h>
#include <stdlib.h>

#include <type_traits>

#include "chain.cuh"
#include "ptx.cuh"

namespace fo {

namespace {

struct B1Params {
    const double *X;
    long long rows, cols, ldx;
    const double *B;            // n x k, row-major
    long long ldb;
    int k;
    DevSides sides;
    WsHead *head;
    double *partials;
    double *out;
    int stages;                 // ring slots per group
    int W, KW;                  // warps of a group across columns / across class slices
    int ns;                     // tensor-core variant: row stride of a tile in shared memory
    int chain_kind;
    int has_pre;
    unsigned side_used;         // sides read by either chain
};

// Chains evaluated inline (same arithmetic, same order, same bits as the interpreter).
enum { kB1Generic = 0, kB1Identity = 1, kB1Mlogreg = 2 };
enum { kB1ColT = 0, kB1None = 1 };

constexpr int kB1Warps = 16;
constexpr int kB1Block = kB1Warps * 32;            // 4 warps per SM sub-partition: 128 registers a thread
constexpr int kB1MaxSlots = 64;
constexpr int kB1MaxTile = 64;                     // R * (padded k) values of one tile

// The chain for one (row, class) value per lane: R0 = d, R(1 + j) = side j.
// Out of line: the interpreter's register file must not weigh on the streaming
// loop, which the common chains (evaluated inline) never leave.
__device__ __noinline__ double b1_lane_chain(const DevChain &ch, double d, double s0, double s1, double s2,
                                             double s3)
{
    RegFile<kRegs, 1> f;
    f.r[0][0] = d;
    f.r[1][0] = s0;
    f.r[2][0] = s1;
    f.r[3][0] = s2;
    f.r[4][0] = s3;
    run_chain<kRegs, 1>(ch, f);
    double o[1];
    operand<kRegs, 1>(ch, f, ch.out[0], o);
    return o[0];
}

// GENERIC: the chains go through the interpreter; otherwise only the chains
// evaluated inline exist in the kernel, and no call weighs on the streaming loop.
template <int NCH, int R, int KL, int AGG, bool STAGED, bool GENERIC>
__global__ void __launch_bounds__(kB1Block, 1)
row_b1_kernel(const __grid_constant__ DevChain pre, const __grid_constant__ DevChain post,
              const __grid_constant__ B1Params p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ unsigned long long s_full[kB1MaxSlots];
    __shared__ __align__(16) double s_part[2][kB1Warps * R * KL];  // [parity][warp][row, local class]
    __shared__ __align__(16) double s_T[kB1Warps][kB1MaxTile];     // every warp's copy of the tile's T
    __shared__ unsigned int s_flag;

    constexpr int M = R * KL;                        // partial sums a warp forms per tile
    constexpr int SH = 5 - Log2<M>::value;           // lane l holds value (l >> SH) after the butterfly
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int W = p.W, KW = p.KW, GW = W * KW;       // warps per group
    const int GROUPS = kB1Warps / GW;
    const int KP = KL * KW;                          // padded class count
    const int MT = R * KP;                           // T values per tile
    const int grp = warp / GW;
    const int wig = warp % GW, w_cls = wig / W, w_col = wig % W;
    const int n = (int)p.cols, k = p.k;
    const int nB = 64 * NCH * W;                     // padded row length of B^T
    const int S = p.stages;

    double *ring = reinterpret_cast<double *>(smem_raw) + (size_t)grp * S * R * n;
    double *BT = reinterpret_cast<double *>(smem_raw) + (size_t)GROUPS * S * R * n;   // KP x nB
    unsigned long long *full = s_full + grp * S;

    const long long ntiles = (p.rows + R - 1) / R;
    const long long me = (long long)blockIdx.x * GROUPS + grp, stride = (long long)gridDim.x * GROUPS;
    const long long my_tiles = (ntiles > me) ? (ntiles - me + stride - 1) / stride : 0;

    // B^T, zero beyond n columns and k classes
    for (int e = threadIdx.x; e < KP * nB; e += kB1Block) {
        const int c = e / nB, j = e - c * nB;
        BT[e] = (c < k && j < n) ? __ldg(p.B + (long long)j * p.ldb + c) : 0.0;
    }

    double2 q[KL][NCH];
#pragma unroll
    for (int cl = 0; cl < KL; ++cl)
#pragma unroll
        for (int c = 0; c < NCH; ++c) q[cl][c] = make_double2(0.0, 0.0);
    bool timed_out = false;

    auto issue = [&](long long it) {
        const int slot = (int)(it % S);
        const long long r0 = (me + it * stride) * R;
        const int nr = (int)((p.rows - r0 < R) ? p.rows - r0 : R);
        double *dst = ring + (size_t)slot * R * n;
        mbar_expect_tx(&full[slot], (unsigned)(nr * n * 8));
        if (p.ldx == n) {
            bulk_g2s(dst, p.X + r0 * p.ldx, (unsigned)(nr * n * 8), &full[slot]);
        } else {
            for (int r = 0; r < nr; ++r)
                bulk_g2s(dst + (size_t)r * n, p.X + (r0 + r) * p.ldx, (unsigned)(n * 8), &full[slot]);
        }
    };

    if (STAGED) {
        if (threadIdx.x == 0) {
            for (int s = 0; s < GROUPS * S; ++s) mbar_init(&s_full[s], 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
    }
    __syncthreads();
    const bool elected = wig == 0 && lane == 0;      // the lane that feeds its group's ring
    if (STAGED && elected)
        for (long long it = 0; it < my_tiles && it < S; ++it) issue(it);

    // what does not change from tile to tile: this lane's columns, and the two
    // (row, class) entries of a tile - entries lane and lane + 32 - it evaluates
    // the chains for
    int colv[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) colv[c] = 64 * (c * W + w_col) + 2 * lane;
    int er[2], ec[2], esrc[2];
    bool ein[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const int idx = lane + 32 * u;
        er[u] = idx / KP;
        ec[u] = idx - er[u] * KP;
        ein[u] = idx < MT;
        esrc[u] = ein[u] ? (grp * GW + (ec[u] / KL) * W) * M + er[u] * KL + (ec[u] % KL) : 0;
    }
    const double *bt_mine = BT + (size_t)(w_cls * KL) * nB;
    const double *t_mine = &s_T[warp][w_cls * KL];

    int slot = 0;
    unsigned phase = 0;
    long long r0 = me * R;
    const long long r0_step = stride * R;
    for (long long it = 0; it < my_tiles; ++it, r0 += r0_step) {
        const int par = (int)(it & 1);

        // side values of this lane's entries, requested ahead of the wait
        double sv[2][FO_MAX_SIDES];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int j = 0; j < FO_MAX_SIDES; ++j) sv[u][j] = 0.0;
        if (p.side_used != 0) {
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const long long row = r0 + er[u];
                const bool ok = ein[u] && ec[u] < k && row < p.rows;
#pragma unroll
                for (int j = 0; j < FO_MAX_SIDES; ++j) {
                    if (ok && ((p.side_used >> j) & 1u)) {
                        const DevSide &sd = p.sides.s[j];
                        const long long off = sd.access == FO_AT_CELL ? row * sd.ld + ec[u]
                                              : sd.access == FO_AT_ROW ? row * sd.ld : (long long)ec[u];
                        sv[u][j] = __ldg(sd.data + off);
                    }
                }
            }
        }

        if (STAGED) {
            if (!mbar_wait(&full[slot], phase)) timed_out = true;
        }
        // this lane's column pairs of the tile's rows
        double2 x[R][NCH];
        const double *tile = ring + (size_t)slot * R * n;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const bool have = r0 + r < p.rows;
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                const int col = colv[c];
                if (STAGED) {
                    x[r][c] = (have && col < n) ? *reinterpret_cast<const double2 *>(tile + (size_t)r * n + col)
                                                : make_double2(0.0, 0.0);
                } else {
                    const double *rowp = p.X + (r0 + r) * p.ldx;
                    x[r][c].x = (have && col < n) ? ld_stream1(rowp + col) : 0.0;
                    x[r][c].y = (have && col + 1 < n) ? ld_stream1(rowp + col + 1) : 0.0;
                }
            }
        }

        // partial products with this warp's class slice of B
        double part[M];
#pragma unroll
        for (int i = 0; i < M; ++i) part[i] = 0.0;
#pragma unroll
        for (int cl = 0; cl < KL; ++cl) {
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                const double2 b = *reinterpret_cast<const double2 *>(bt_mine + (size_t)cl * nB + colv[c]);
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    part[r * KL + cl] = fma(x[r][c].x, b.x, part[r * KL + cl]);
                    part[r * KL + cl] = fma(x[r][c].y, b.y, part[r * KL + cl]);
                }
            }
        }
        warp_sum_multi<M>(part, lane);
        double *mypart = &s_part[par][0];
        if ((lane & ((1 << SH) - 1)) == 0) mypart[warp * M + (lane >> SH)] = part[0];
        if (GW > 1) {
            asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "r"(GW * 32) : "memory");
        } else {
            __syncwarp();
        }
        // the tile now lives in the group's registers: its slot takes the tile S ahead
        if (STAGED && elected && it + S < my_tiles) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            issue(it + S);
        }
        if (++slot == S) { slot = 0; phase ^= 1u; }

        // every warp of the group: D of the whole tile (column warps in order), the
        // two chains, T into the warp's own copy
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (32 * u < MT) {                        // uniform
                const bool ok = ein[u] && ec[u] < k && r0 + er[u] < p.rows;
                double d = 0.0;
                if (ein[u]) {
                    const double *src = mypart + esrc[u];
                    for (int wc = 0; wc < W; ++wc) d += src[wc * M];
                }
                double t;
                if (p.chain_kind == kB1Identity) {
                    t = d;
                } else {
                    double rowsum = 0.0;
                    if (p.has_pre) {
                        double pv;
                        if (!GENERIC || p.chain_kind == kB1Mlogreg) pv = sv[u][0] * d;
                        else pv = b1_lane_chain(pre, d, sv[u][0], sv[u][1], sv[u][2], sv[u][3]);
                        rowsum = ok ? pv : 0.0;
                        // classes of a row sit in KP consecutive lanes
                        for (int o = 1; o < KP && o < 32; o <<= 1)
                            rowsum += __shfl_xor_sync(0xffffffffu, rowsum, o);
                    }
                    if (!GENERIC || p.chain_kind == kB1Mlogreg) {
                        t = sv[u][0] * d - sv[u][0] * rowsum;
                    } else {
                        double s2[FO_MAX_SIDES];
#pragma unroll
                        for (int j = 0; j < FO_MAX_SIDES; ++j)
                            s2[j] = (p.has_pre && j == p.sides.n) ? rowsum : sv[u][j];
                        t = b1_lane_chain(post, d, s2[0], s2[1], s2[2], s2[3]);
                    }
                }
                t = ok ? t : 0.0;
                if (ein[u]) s_T[warp][lane + 32 * u] = t;
                if (AGG == kB1None && wig == 0 && ok) p.out[(r0 + er[u]) * k + ec[u]] = t;
            }
        }

        if (AGG == kB1ColT) {
            __syncwarp();
#pragma unroll
            for (int r = 0; r < R; ++r) {
#pragma unroll
                for (int cl = 0; cl < KL; cl += 2) {
                    const double2 tt = *reinterpret_cast<const double2 *>(t_mine + r * KP + cl);
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        q[cl][c].x = fma(tt.x, x[r][c].x, q[cl][c].x);
                        q[cl][c].y = fma(tt.x, x[r][c].y, q[cl][c].y);
                        q[cl + 1][c].x = fma(tt.y, x[r][c].x, q[cl + 1][c].x);
                        q[cl + 1][c].y = fma(tt.y, x[r][c].y, q[cl + 1][c].y);
                    }
                }
            }
        }
    }

    if (STAGED && timed_out) atomicExch(&p.head->status, 1u);

    if (AGG == kB1ColT) {
        // groups -> CTA through shared memory, groups in index order; then the
        // CTA's n x k tile goes to the workspace and the last CTAs add them up
        double *qs = reinterpret_cast<double *>(smem_raw);
        for (int g = 0; g < GROUPS; ++g) {
            __syncthreads();
            if (warp / GW == g) {
#pragma unroll
                for (int cl = 0; cl < KL; ++cl) {
                    const int c = w_cls * KL + cl;
#pragma unroll
                    for (int ch = 0; ch < NCH; ++ch) {
                        const int col = 64 * (ch * W + w_col) + 2 * lane;
                        if (c < k && col < n) {
                            double *dst = qs + (size_t)col * k + c;
                            *dst = (g == 0) ? q[cl][ch].x : *dst + q[cl][ch].x;
                        }
                        if (c < k && col + 1 < n) {
                            double *dst = qs + (size_t)(col + 1) * k + c;
                            *dst = (g == 0) ? q[cl][ch].y : *dst + q[cl][ch].y;
                        }
                    }
                }
            }
        }
        __syncthreads();
        const long long width = (long long)n * k;
        for (long long j = threadIdx.x; j < width; j += kB1Block)
            p.partials[(size_t)blockIdx.x * width + j] = qs[j];
        reduce_columns_two_level(p.head, p.partials, p.partials + (size_t)gridDim.x * width, width, p.out,
                                 &s_flag);
    }
}

// ------------------------------------------------------- tensor-core variant
// The two products of a tile - D = X_tile B (8 rows x 8 classes, summed over the
// columns) and H += X_tile^T T (8 columns x 8 classes, summed over the 8 rows) -
// are small dense fp64 contractions, so they run as m8n8k4 double-precision
// matrix multiply-accumulates: one instruction does the work of eight warp-wide
// multiply-adds and sums over its k dimension by itself, which removes the
// partial-sum exchange that bounds the kernel above once k > 2.
//
// 8 warps per CTA.  A group of W x KB warps shares a ring of 8-row tiles; warp
// (w, cb) owns the columns [w * 8 NCB, (w + 1) * 8 NCB) and the classes
// [8 cb, 8 cb + 8): its fragments of B (one register per 4-column step) and its
// tile of the output (two registers per 8-column block) stay in registers.
// Rows sit in shared memory with a stride of ns doubles, ns = 4 (mod 8), so
// that both ways of reading a tile - 8 rows x 4 columns, 4 rows x 8 columns -
// touch every bank once.  Rows beyond the matrix and columns beyond n read
// zeros or stale finite values whose partner operand is zero.
__device__ __forceinline__ void dmma_8x8x4(double &c0, double &c1, double a, double b)
{
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                 : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}

constexpr int kMmaMaxWarps = 16;
constexpr int kMmaMaxSlots = 32;

// NW warps per CTA (8 are compiled: up to 255 registers a thread).
template <int NW, int NCB, int AGG, bool GENERIC>
__global__ void __launch_bounds__(NW * 32, 1)
row_b1_mma_kernel(const __grid_constant__ DevChain pre, const __grid_constant__ DevChain post,
                  const __grid_constant__ B1Params p)
{
    constexpr int kMmaWarps = NW, kMmaBlock = NW * 32;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ unsigned long long s_full[kMmaMaxSlots];
    __shared__ __align__(16) double s_D[2][kMmaWarps][64];    // partial D of every warp (W > 1)
    __shared__ double s_rs[2][kMmaWarps][8];                  // row sums of every class block (KB > 1)
    __shared__ double s_T[kMmaWarps][64];
    __shared__ unsigned int s_flag;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int W = p.W, KB = p.KW, GW = W * KB, GROUPS = kMmaWarps / GW;
    const int grp = warp / GW, wig = warp % GW, cb = wig / W, w = wig % W;
    const int n = (int)p.cols, k = p.k, ns = p.ns, S = p.stages;
    const int lq = lane >> 2, lr = lane & 3;                   // fragment coordinates
    const int col0 = w * NCB * 8;

    double *ring = reinterpret_cast<double *>(smem_raw) + (size_t)grp * S * 8 * ns;
    unsigned long long *full = s_full + grp * S;
    const long long ntiles = (p.rows + 7) / 8;
    const long long me = (long long)blockIdx.x * GROUPS + grp, stride = (long long)gridDim.x * GROUPS;
    const long long my_tiles = (ntiles > me) ? (ntiles - me + stride - 1) / stride : 0;

    // fragments of B: step s covers columns col0 + 4 s .. + 3
    double bfrag[2 * NCB];
#pragma unroll
    for (int s = 0; s < 2 * NCB; ++s) {
        const int j = col0 + 4 * s + lr, c = cb * 8 + lq;
        bfrag[s] = (j < n && c < k) ? __ldg(p.B + (long long)j * p.ldb + c) : 0.0;
    }
    double acc[NCB][2];
#pragma unroll
    for (int jb = 0; jb < NCB; ++jb) acc[jb][0] = acc[jb][1] = 0.0;

    // the rings start as zeros: padding columns and the rows of a ragged last
    // tile are never written by a copy
    {
        double *all = reinterpret_cast<double *>(smem_raw);
        const int total = GROUPS * S * 8 * ns + 8;               // and the slack behind the last tile
        for (int e = threadIdx.x; e < total; e += kMmaBlock) all[e] = 0.0;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < GROUPS * S; ++s) mbar_init(&s_full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();

    bool timed_out = false;
    auto issue = [&](long long it, int slot) {
        const long long r0 = (me + it * stride) * 8;
        const int nr = (int)((p.rows - r0 < 8) ? p.rows - r0 : 8);
        double *dst = ring + (size_t)slot * 8 * ns;
        mbar_expect_tx(&full[slot], (unsigned)(nr * n * 8));
        if (p.ldx == n && ns == n) {
            bulk_g2s(dst, p.X + r0 * p.ldx, (unsigned)(nr * n * 8), &full[slot]);
        } else {
            for (int r = 0; r < nr; ++r)
                bulk_g2s(dst + (size_t)r * ns, p.X + (r0 + r) * p.ldx, (unsigned)(n * 8), &full[slot]);
        }
    };
    const bool elected = wig == 0 && lane == 0;
    if (elected)
        for (int it = 0; it < S && it < my_tiles; ++it) issue(it, it);

    const int c0 = cb * 8 + 2 * lr;                            // this lane's two classes (c0, c0 + 1)
    // side values of the entries (row lq, classes c0 and c0 + 1) of the tile at tile_r0;
    // the inline chains only ever read side 0
    constexpr int NS = GENERIC ? FO_MAX_SIDES : 1;
    auto load_sides = [&](long long tile_r0, double (&a)[NS], double (&b)[NS]) {
#pragma unroll
        for (int j = 0; j < NS; ++j) a[j] = b[j] = 0.0;
        if (p.side_used == 0) return;
        const long long row = tile_r0 + lq;
        const bool okr = row < p.rows;
#pragma unroll
        for (int j = 0; j < NS; ++j) {
            if ((p.side_used >> j) & 1u) {
                const DevSide &sd = p.sides.s[j];
                const long long base = sd.access == FO_AT_CELL ? row * sd.ld + c0
                                       : sd.access == FO_AT_ROW ? row * sd.ld : (long long)c0;
                const int step = sd.access == FO_AT_ROW ? 0 : 1;
                if (okr && c0 < k) a[j] = __ldg(sd.data + base);
                if (okr && c0 + 1 < k) b[j] = __ldg(sd.data + base + step);
            }
        }
    };
    double nsv0[NS], nsv1[NS];
    load_sides(me * 8, nsv0, nsv1);
    int slot = 0, prev_slot = 0;
    unsigned phase = 0;
    long long r0 = me * 8;
    const long long r0_step = stride * 8;
    for (long long it = 0; it < my_tiles; ++it, r0 += r0_step) {
        const int par = (int)(it & 1);
        const long long row = r0 + lq;
        const bool ok0 = row < p.rows && c0 < k, ok1 = row < p.rows && c0 + 1 < k;

        // side values of this tile (requested while the previous tile was worked on)
        double sv0[NS], sv1[NS];
#pragma unroll
        for (int j = 0; j < NS; ++j) {
            sv0[j] = nsv0[j];
            sv1[j] = nsv1[j];
        }
        load_sides(r0 + r0_step, nsv0, nsv1);

        if (!mbar_wait(&full[slot], phase)) timed_out = true;
        const double *tile = ring + (size_t)slot * 8 * ns;

        // D = X_tile B over this warp's columns
        // (four independent accumulator pairs: consecutive steps do not wait for each other)
        double d0, d1;
        {
            double da[4][2];
#pragma unroll
            for (int i = 0; i < 4; ++i) da[i][0] = da[i][1] = 0.0;
            const double *arow = tile + (size_t)lq * ns + col0 + lr;
#pragma unroll
            for (int s = 0; s < 2 * NCB; ++s)
                if (col0 + 4 * s < n) dmma_8x8x4(da[s & 3][0], da[s & 3][1], arow[4 * s], bfrag[s]);
            d0 = (da[0][0] + da[1][0]) + (da[2][0] + da[3][0]);
            d1 = (da[0][1] + da[1][1]) + (da[2][1] + da[3][1]);
        }
        if (W > 1) *reinterpret_cast<double2 *>(&s_D[par][warp][2 * lane]) = make_double2(d0, d1);
        if (GW > 1) {
            asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "r"(GW * 32) : "memory");
            // every warp of the group is past its use of the previous tile
            if (elected && it > 0 && it - 1 + S < my_tiles) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                issue(it - 1 + S, prev_slot);
            }
        }
        if (W > 1) {
            d0 = d1 = 0.0;
            for (int ww = 0; ww < W; ++ww) {
                const double2 v = *reinterpret_cast<const double2 *>(&s_D[par][grp * GW + cb * W + ww][2 * lane]);
                d0 += v.x;
                d1 += v.y;
            }
        }

        double t0, t1;
        if (p.chain_kind == kB1Identity) {
            t0 = d0;
            t1 = d1;
        } else {
            double rowsum = 0.0;
            if (p.has_pre) {
                double p0, p1;
                if (!GENERIC || p.chain_kind == kB1Mlogreg) {
                    p0 = sv0[0] * d0;
                    p1 = sv1[0] * d1;
                } else {
                    p0 = b1_lane_chain(pre, d0, sv0[0], sv0[NS > 1 ? 1 : 0], sv0[NS > 2 ? 2 : 0], sv0[NS > 3 ? 3 : 0]);
                    p1 = b1_lane_chain(pre, d1, sv1[0], sv1[NS > 1 ? 1 : 0], sv1[NS > 2 ? 2 : 0], sv1[NS > 3 ? 3 : 0]);
                }
                rowsum = (ok0 ? p0 : 0.0) + (ok1 ? p1 : 0.0);
                rowsum += __shfl_xor_sync(0xffffffffu, rowsum, 1);
                rowsum += __shfl_xor_sync(0xffffffffu, rowsum, 2);
                if (KB > 1) {
                    if (w == 0 && lr == 0) s_rs[par][grp * KB + cb][lq] = rowsum;
                    asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "r"(GW * 32) : "memory");
                    rowsum = 0.0;
                    for (int b = 0; b < KB; ++b) rowsum += s_rs[par][grp * KB + b][lq];
                }
            }
            if (!GENERIC || p.chain_kind == kB1Mlogreg) {
                t0 = sv0[0] * d0 - sv0[0] * rowsum;
                t1 = sv1[0] * d1 - sv1[0] * rowsum;
            } else {
                double a0[FO_MAX_SIDES], a1[FO_MAX_SIDES];
#pragma unroll
                for (int j = 0; j < FO_MAX_SIDES; ++j) {
                    const bool rs = p.has_pre && j == p.sides.n;
                    a0[j] = rs ? rowsum : sv0[j < NS ? j : 0];
                    a1[j] = rs ? rowsum : sv1[j < NS ? j : 0];
                }
                t0 = b1_lane_chain(post, d0, a0[0], a0[1], a0[2], a0[3]);
                t1 = b1_lane_chain(post, d1, a1[0], a1[1], a1[2], a1[3]);
            }
        }
        t0 = ok0 ? t0 : 0.0;
        t1 = ok1 ? t1 : 0.0;

        if (AGG == kB1None) {
            if (w == 0 && ok0) p.out[row * k + c0] = t0;
            if (w == 0 && ok1) p.out[row * k + c0 + 1] = t1;
        } else {
            // T from accumulator layout (row lq, classes 2 lr, 2 lr + 1) to operand
            // layout (rows lr and lr + 4, class lq) through the warp's own scratch
            s_T[warp][lq * 8 + 2 * lr] = t0;
            s_T[warp][lq * 8 + 2 * lr + 1] = t1;
            __syncwarp();
            const double tf0 = s_T[warp][lr * 8 + lq], tf1 = s_T[warp][(4 + lr) * 8 + lq];
            const double *a0p = tile + (size_t)lr * ns + col0 + lq;
            const double *a1p = a0p + (size_t)4 * ns;
#pragma unroll
            for (int jb = 0; jb < NCB; ++jb) {
                if (col0 + 8 * jb < n) {
                    dmma_8x8x4(acc[jb][0], acc[jb][1], a0p[8 * jb], tf0);
                    dmma_8x8x4(acc[jb][0], acc[jb][1], a1p[8 * jb], tf1);
                }
            }
        }
        if (GW == 1) {
            __syncwarp();
            if (elected && it + S < my_tiles) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                issue(it + S, slot);
            }
        }
        prev_slot = slot;
        if (++slot == S) { slot = 0; phase ^= 1u; }
    }

    if (timed_out) atomicExch(&p.head->status, 1u);

    if (AGG == kB1ColT) {
        double *qs = reinterpret_cast<double *>(smem_raw);
        for (int g = 0; g < GROUPS; ++g) {
            __syncthreads();
            if (grp == g) {
#pragma unroll
                for (int jb = 0; jb < NCB; ++jb) {
                    const int j = col0 + 8 * jb + lq;
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const int c = c0 + i;
                        if (j < n && c < k) {
                            double *dst = qs + (size_t)j * k + c;
                            *dst = (g == 0) ? acc[jb][i] : *dst + acc[jb][i];
                        }
                    }
                }
            }
        }
        __syncthreads();
        const long long width = (long long)n * k;
        for (long long j = threadIdx.x; j < width; j += kMmaBlock)
            p.partials[(size_t)blockIdx.x * width + j] = qs[j];
        reduce_columns_two_level(p.head, p.partials, p.partials + (size_t)gridDim.x * width, width, p.out,
                                 &s_flag);
    }
}

// ----------------------------------------------------------------- narrow
// Rows of at most NC <= 16 columns and at most KC <= 8 classes, NC * KC <= 64
// (Eq. 2 on the tall, narrow matrices of the paper's end-to-end runs): a thread
// takes whole rows.  It loads its row, forms the k products with B (shared
// memory, every lane the same address), sums the first chain over the classes by
// itself, and keeps the n x k output sums in registers; the CTA adds them up in
// a fixed order at the end.
constexpr int kB1NarrowThreads = 256;

template <int NC, int KC, int AGG, bool VEC>
__global__ void __launch_bounds__(kB1NarrowThreads)
row_b1_narrow_kernel(const __grid_constant__ DevChain pre, const __grid_constant__ DevChain post,
                     const __grid_constant__ B1Params p)
{
    __shared__ double s_B[NC * KC];
    __shared__ double s_red[NC * KC * 32];
    __shared__ unsigned int s_flag;
    const int n = (int)p.cols, k = p.k;
    for (int e = threadIdx.x; e < NC * KC; e += kB1NarrowThreads) {
        const int j = e / KC, c = e - j * KC;
        s_B[e] = (j < n && c < k) ? __ldg(p.B + (long long)j * p.ldb + c) : 0.0;
    }
    __syncthreads();
    double h[NC * KC];
#pragma unroll
    for (int e = 0; e < NC * KC; ++e) h[e] = 0.0;

    const long long stride = (long long)gridDim.x * kB1NarrowThreads;
    for (long long row = (long long)blockIdx.x * kB1NarrowThreads + threadIdx.x; row < p.rows; row += stride) {
        const double *xr = p.X + row * p.ldx;
        double x[NC];
        if (VEC) {
#pragma unroll
            for (int j = 0; j < NC; j += 2) {
                double2 t2 = make_double2(0.0, 0.0);
                if (j < n) t2 = __ldg(reinterpret_cast<const double2 *>(xr + j));     // n even
                x[j] = t2.x;
                x[j + 1] = t2.y;
            }
        } else {
#pragma unroll
            for (int j = 0; j < NC; ++j) x[j] = j < n ? __ldg(xr + j) : 0.0;
        }
        double d[KC], t[KC], sv[KC][FO_MAX_SIDES];
#pragma unroll
        for (int c = 0; c < KC; ++c) {
            d[c] = 0.0;
#pragma unroll
            for (int j = 0; j < FO_MAX_SIDES; ++j) {
                sv[c][j] = 0.0;
                if (c < k && ((p.side_used >> j) & 1u)) {
                    const DevSide &sd = p.sides.s[j];
                    const long long off = sd.access == FO_AT_CELL ? row * sd.ld + c
                                          : sd.access == FO_AT_ROW ? row * sd.ld : (long long)c;
                    sv[c][j] = __ldg(sd.data + off);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < NC; ++j)
#pragma unroll
            for (int c = 0; c < KC; ++c) d[c] = fma(x[j], s_B[j * KC + c], d[c]);

        if (p.chain_kind == kB1Identity) {
#pragma unroll
            for (int c = 0; c < KC; ++c) t[c] = d[c];
        } else {
            double rowsum = 0.0;
            if (p.has_pre) {
#pragma unroll
                for (int c = 0; c < KC; ++c) {
                    const double pv = p.chain_kind == kB1Mlogreg
                                          ? sv[c][0] * d[c]
                                          : b1_lane_chain(pre, d[c], sv[c][0], sv[c][1], sv[c][2], sv[c][3]);
                    rowsum += c < k ? pv : 0.0;
                }
            }
#pragma unroll
            for (int c = 0; c < KC; ++c) {
                if (p.chain_kind == kB1Mlogreg) {
                    t[c] = sv[c][0] * d[c] - sv[c][0] * rowsum;
                } else {
                    double s2[FO_MAX_SIDES];
#pragma unroll
                    for (int j = 0; j < FO_MAX_SIDES; ++j) s2[j] = (p.has_pre && j == p.sides.n) ? rowsum : sv[c][j];
                    t[c] = b1_lane_chain(post, d[c], s2[0], s2[1], s2[2], s2[3]);
                }
            }
        }
        if (AGG == kB1None) {
#pragma unroll
            for (int c = 0; c < KC; ++c)
                if (c < k) p.out[row * k + c] = t[c];
        } else {
#pragma unroll
            for (int j = 0; j < NC; ++j)
#pragma unroll
                for (int c = 0; c < KC; ++c) h[j * KC + c] = fma(x[j], c < k ? t[c] : 0.0, h[j * KC + c]);
        }
    }
    if (AGG == kB1ColT) {
        block_sum<NC * KC>(h, s_red);
        const long long width = (long long)n * k;
        if (threadIdx.x == 0) {
#pragma unroll
            for (int j = 0; j < NC; ++j)
#pragma unroll
                for (int c = 0; c < KC; ++c)
                    if (j < n && c < k) p.partials[(size_t)blockIdx.x * width + (size_t)j * k + c] = h[j * KC + c];
        }
        reduce_columns_two_level(p.head, p.partials, p.partials + (size_t)gridDim.x * width, width, p.out,
                                 &s_flag);
    }
}

// ------------------------------------------------------------------- CSR
// The same operator over the stored cells of a CSR X (the listing's
// genexecSparse).  A warp takes blocks of 32 consecutive rows and stages their
// cells - one contiguous piece of colidx / vals - in its slice of shared memory;
// then one row after the other: the 32 lanes are (cell slot, class) pairs,
// 32 / KP slots x KP classes, every lane adds val * B[col][class] over its slot's
// cells, slots are combined by shuffles, the chains run once per class, and for
// col_agg_B1_T every (cell, class) adds val * T_class into the CTA's n x KP
// output tile in shared memory (atomics: several warps share the tile).
constexpr int kB1CsrThreads = 256;
constexpr int kB1CsrWarps = kB1CsrThreads / 32;
constexpr int kB1CsrStage = 512;           // stored cells a warp can stage per block of rows

struct B1CsrParams {
    const int *rowptr;
    const int *colidx;
    const double *vals;
    long long rows, cols;
    const double *B;
    long long ldb;
    int k;
    DevSides sides;
    WsHead *head;
    double *partials;
    double *out;
    int chain_kind, has_pre;
    unsigned side_used;
};

template <int KP, int AGG, bool GENERIC>
__global__ void __launch_bounds__(kB1CsrThreads)
row_b1_csr_kernel(const __grid_constant__ DevChain pre, const __grid_constant__ DevChain post,
                  const __grid_constant__ B1CsrParams p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ unsigned int s_flag;
    constexpr int CS = 32 / KP;                       // cell slots of a warp
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c = lane % KP, slot = lane / KP;
    const int n = (int)p.cols, k = p.k;

    double *Bs = reinterpret_cast<double *>(smem_raw);                   // n x KP
    double *Hs = Bs + (size_t)n * KP;                                    // n x KP (col_agg_B1_T)
    double *sx = Bs + (size_t)(AGG == kB1ColT ? 2 : 1) * n * KP + (size_t)warp * kB1CsrStage;
    int *sc = reinterpret_cast<int *>(Bs + (size_t)(AGG == kB1ColT ? 2 : 1) * n * KP + (size_t)kB1CsrWarps * kB1CsrStage)
              + (size_t)warp * kB1CsrStage;
    for (int e = threadIdx.x; e < n * KP; e += kB1CsrThreads) {
        const int j = e / KP, cc = e - j * KP;
        Bs[e] = cc < k ? __ldg(p.B + (long long)j * p.ldb + cc) : 0.0;
        if (AGG == kB1ColT) Hs[e] = 0.0;
    }
    __syncthreads();

    const long long nblocks = (p.rows + 31) >> 5;
    const long long warp0 = (long long)blockIdx.x * kB1CsrWarps + warp;
    const long long nwarps = (long long)gridDim.x * kB1CsrWarps;
    for (long long blk = warp0; blk < nblocks; blk += nwarps) {
        const long long myrow = (blk << 5) + lane;
        const bool have = myrow < p.rows;
        const int beg_l = have ? __ldg(p.rowptr + myrow) : 0;
        const int end_l = have ? __ldg(p.rowptr + myrow + 1) : beg_l;
        const int nrows = (int)((p.rows - (blk << 5) < 32) ? p.rows - (blk << 5) : 32);
        const int base = __shfl_sync(0xffffffffu, beg_l, 0);
        const int total = __shfl_sync(0xffffffffu, end_l, nrows - 1) - base;
        const bool staged = total <= kB1CsrStage;
        if (staged) {
            for (int e = lane; e < total; e += 32) {
                sc[e] = __ldg(p.colidx + base + e);
                sx[e] = __ldg(p.vals + base + e);
            }
        }
        __syncwarp();

        for (int rr = 0; rr < nrows; ++rr) {
            const long long row = (blk << 5) + rr;
            const int beg = __shfl_sync(0xffffffffu, beg_l, rr);
            const int end = __shfl_sync(0xffffffffu, end_l, rr);
            const bool ok = c < k;
            // side values of (row, class)
            double sv[FO_MAX_SIDES];
#pragma unroll
            for (int j = 0; j < FO_MAX_SIDES; ++j) {
                sv[j] = 0.0;
                if (ok && ((p.side_used >> j) & 1u)) {
                    const DevSide &sd = p.sides.s[j];
                    const long long off = sd.access == FO_AT_CELL ? row * sd.ld + c
                                          : sd.access == FO_AT_ROW ? row * sd.ld : (long long)c;
                    sv[j] = __ldg(sd.data + off);
                }
            }
            // D_c = sum over the row's cells of val * B[col][c]
            double d = 0.0;
            for (int q = beg + slot; q < end; q += CS) {
                const double val = staged ? sx[q - base] : __ldg(p.vals + q);
                const int col = staged ? sc[q - base] : __ldg(p.colidx + q);
                d = fma(val, Bs[(size_t)col * KP + c], d);
            }
#pragma unroll
            for (int o = KP; o < 32; o <<= 1) d += __shfl_xor_sync(0xffffffffu, d, o);

            double t;
            if (p.chain_kind == kB1Identity) {
                t = d;
            } else {
                double rowsum = 0.0;
                if (p.has_pre) {
                    double pv;
                    if (!GENERIC || p.chain_kind == kB1Mlogreg) pv = sv[0] * d;
                    else pv = b1_lane_chain(pre, d, sv[0], sv[1], sv[2], sv[3]);
                    rowsum = ok ? pv : 0.0;
#pragma unroll
                    for (int o = 1; o < KP; o <<= 1) rowsum += __shfl_xor_sync(0xffffffffu, rowsum, o);
                }
                if (!GENERIC || p.chain_kind == kB1Mlogreg) {
                    t = sv[0] * d - sv[0] * rowsum;
                } else {
                    double s2[FO_MAX_SIDES];
#pragma unroll
                    for (int j = 0; j < FO_MAX_SIDES; ++j) s2[j] = (p.has_pre && j == p.sides.n) ? rowsum : sv[j];
                    t = b1_lane_chain(post, d, s2[0], s2[1], s2[2], s2[3]);
                }
            }
            if (AGG == kB1None) {
                if (ok && slot == 0) p.out[row * k + c] = t;
            } else if (ok) {
                for (int q = beg + slot; q < end; q += CS) {
                    const double val = staged ? sx[q - base] : __ldg(p.vals + q);
                    const int col = staged ? sc[q - base] : __ldg(p.colidx + q);
                    atomicAdd(&Hs[(size_t)col * KP + c], val * t);
                }
            }
        }
        __syncwarp();          // the slice is reused by the next block
    }

    if (AGG == kB1ColT) {
        __syncthreads();
        const long long width = (long long)n * k;
        for (long long e = threadIdx.x; e < width; e += kB1CsrThreads) {
            const long long j = e / k, cc = e - j * k;
            p.partials[(size_t)blockIdx.x * width + e] = Hs[j * KP + cc];
        }
        reduce_columns_two_level(p.head, p.partials, p.partials + (size_t)gridDim.x * width, width, p.out,
                                 &s_flag);
    }
}

__global__ void b1_fill_zero_kernel(double *out, long long n)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
         i += (long long)gridDim.x * blockDim.x)
        out[i] = 0.0;
}

// ------------------------------------------------------------------- host
constexpr size_t kB1SmemBudget = 200 * 1024;       // dynamic shared memory of one CTA
constexpr long long kB1MaxOutTile = 24576;         // n * k doubles of a CTA's output tile (192 KB)
constexpr long long kB1CsrMaxTile = 9600;          // CSR X: n * (padded k); B and the output tile share 150 KB

int b1_grid_cap() { return 148 * 2; }              // bound used for workspace sizing

size_t b1_ws_bytes(long long cols, int k, int agg)
{
    if (agg == FO_ROW_COL_AGG_B1_T)
        return sizeof(WsHead) + (size_t)(b1_grid_cap() + b1_grid_cap() / kGroup + 1) * (size_t)cols * (size_t)k * sizeof(double);
    return sizeof(WsHead);
}

// Kernel shape for n columns and k classes: column pairs per lane (nch), rows
// per tile (r), classes per warp (kl) - the compiled combinations - and the
// group layout (w warps across columns, kw across class slices).
struct B1Shape {
    int nch, r, kl, w, kw;
};

const int kB1Compiled[][3] = {{1, 8, 2}, {2, 4, 2}, {4, 2, 2}, {1, 4, 4}, {2, 2, 4}, {1, 2, 8}};

int pow2_at_least(long long v)
{
    int p = 1;
    while (p < v) p <<= 1;
    return p;
}

// Fills in w and kw for a compiled (nch, r, kl); false if the shape cannot hold the problem.
bool b1_complete(B1Shape &s, long long n, int k)
{
    const int kp = pow2_at_least(k < 2 ? 2 : k);
    if (s.kl > kp) return false;
    s.kw = kp / s.kl;
    s.w = pow2_at_least((n + 64 * s.nch - 1) / (64 * s.nch));
    if (s.w < 1) s.w = 1;
    if (s.w * s.kw > kB1Warps) return false;
    if (s.r * s.kl * s.kw > kB1MaxTile) return false;
    // B^T plus at least two ring slots per group must fit in shared memory
    const size_t bt = (size_t)s.kl * s.kw * 64 * s.nch * s.w * 8, slot = (size_t)s.r * n * 8;
    if (bt + 2 * slot * (kB1Warps / (s.w * s.kw)) > kB1SmemBudget) return false;
    return true;
}

bool b1_shape(long long n, int k, B1Shape *out)
{
    // the knob b1.shape = "nch,r,kl" picks a compiled shape
    char e[48];
    if (tune_get("b1.shape", e, sizeof(e))) {
        int a = 0, b = 0, c = 0;
        if (sscanf(e, "%d,%d,%d", &a, &b, &c) == 3)
            for (const auto &t : kB1Compiled)
                if (t[0] == a && t[1] == b && t[2] == c) {
                    B1Shape s = {a, b, c, 0, 0};
                    if (b1_complete(s, n, k)) { *out = s; return true; }
                }
    }
    const int kp = pow2_at_least(k < 2 ? 2 : k);
    // measured on B200 (t(X) (X V) and the Eq. 2 chain; 100, 500 and 1000 columns,
    // k = 2 .. 32): two column pairs per lane beat one (half as many partial sums
    // to combine per multiply-add); two classes: {2,4,2}; more: {2,2,4}, and
    // {4,2,2} for 8 classes over more than 512 columns
    const int pref2[][3] = {{2, 4, 2}, {4, 2, 2}, {1, 8, 2}};
    const int pref4[][3] = {{2, 2, 4}, {2, 4, 2}, {1, 4, 4}};
    const int pref8w[][3] = {{4, 2, 2}, {2, 2, 4}, {1, 2, 8}};
    const int (*pref)[3] = kp <= 2 ? pref2 : (kp == 8 && n > 512) ? pref8w : pref4;
    if (kp <= 2 && n <= 64) {
        B1Shape s = {1, 8, 2, 0, 0};
        if (b1_complete(s, n, k)) { *out = s; return true; }
    }
    for (int i = 0; i < 3; ++i) {
        B1Shape s = {pref[i][0], pref[i][1], pref[i][2], 0, 0};
        if (b1_complete(s, n, k)) { *out = s; return true; }
    }
    for (const auto &t : kB1Compiled) {
        B1Shape s = {t[0], t[1], t[2], 0, 0};
        if (b1_complete(s, n, k)) { *out = s; return true; }
    }
    return false;
}

template <int NCH, int R, int KL>
cudaError_t b1_launch_shape(const DevChain &pre, const DevChain &post, const B1Params &p, int agg,
                            bool staged, int grid, size_t smem, cudaStream_t st)
{
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<grid, kB1Block, smem, st>>>(pre, post, p);
        return cudaGetLastError();
    };
    const bool generic = p.chain_kind == kB1Generic;
    if (agg == FO_ROW_COL_AGG_B1_T) {
        if (generic)
            return staged ? go(row_b1_kernel<NCH, R, KL, kB1ColT, true, true>)
                          : go(row_b1_kernel<NCH, R, KL, kB1ColT, false, true>);
        return staged ? go(row_b1_kernel<NCH, R, KL, kB1ColT, true, false>)
                      : go(row_b1_kernel<NCH, R, KL, kB1ColT, false, false>);
    }
    if (generic)
        return staged ? go(row_b1_kernel<NCH, R, KL, kB1None, true, true>)
                      : go(row_b1_kernel<NCH, R, KL, kB1None, false, true>);
    return staged ? go(row_b1_kernel<NCH, R, KL, kB1None, true, false>)
                  : go(row_b1_kernel<NCH, R, KL, kB1None, false, false>);
}

// Tensor-core variant: column blocks per warp (compiled: 8, 14, 16, 20), warps
// across the columns and class blocks of 8; w * kb <= 8 warps.
struct MmaShape {
    int ncb, w, kb;
};

bool b1_mma_shape(long long n, int k, int nw, MmaShape *out)
{
    const int kb = pow2_at_least((k + 7) / 8);
    if (kb > nw || n < 2) return false;
    // the knob b1.mma_shape = "ncb,w"
    char e[48];
    if (tune_get("b1.mma_shape", e, sizeof(e))) {
        int a = 0, b = 0;
        if (sscanf(e, "%d,%d", &a, &b) == 2 && (a == 8 || a == 14 || a == 16 || a == 20) && b >= 1 &&
            (b & (b - 1)) == 0 && b * kb <= nw && (long long)8 * a * b >= n) {
            *out = MmaShape{a, b, kb};
            return true;
        }
    }
    const int ncbs[] = {8, 14, 16, 20};
    for (int w = 1; w * kb <= nw; w *= 2)
        for (int ncb : ncbs)
            if ((long long)8 * ncb * w >= n) {
                *out = MmaShape{ncb, w, kb};
                return true;
            }
    return false;
}

// Row stride of a tile in shared memory: the smallest ns >= n with ns = 4 (mod 8).
int b1_mma_stride(long long n) { return (int)(n + ((4 - n % 8) + 8) % 8); }

template <int NW, int NCB>
cudaError_t b1_mma_launch(const DevChain &pre, const DevChain &post, const B1Params &p, int agg,
                          int grid, size_t smem, cudaStream_t st)
{
    constexpr int kMmaBlock = NW * 32;
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<grid, kMmaBlock, smem, st>>>(pre, post, p);
        return cudaGetLastError();
    };
    const bool generic = p.chain_kind == kB1Generic;
    if (agg == FO_ROW_COL_AGG_B1_T)
        return generic ? go(row_b1_mma_kernel<NW, NCB, kB1ColT, true>) : go(row_b1_mma_kernel<NW, NCB, kB1ColT, false>);
    return generic ? go(row_b1_mma_kernel<NW, NCB, kB1None, true>) : go(row_b1_mma_kernel<NW, NCB, kB1None, false>);
}

bool b1_aligned16(const void *q) { return ((uintptr_t)q & 15u) == 0; }

}  // namespace

}  // namespace fo

extern "C" {

size_t fused_row_b1_workspace_bytes(const fo_mat *X, int k, int agg)
{
    if (!X || (X->kind != FO_DENSE && X->kind != FO_CSR) || k < 1 || k > FO_B1_MAX_K) return 0;
    if (agg != FO_ROW_COL_AGG_B1_T && agg != FO_ROW_NO_AGG_B1) return 0;
    const long long cols = X->kind == FO_CSR ? X->csr.cols : X->dense.cols;
    if (cols < 0) return 0;
    return fo::b1_ws_bytes(cols, k, agg);
}

int fused_row_b1(const fo_chain *pre, const fo_chain *post, const fo_mat *X, const fo_dense *B,
                 const fo_side *sides, int n_sides, const double *scalars, int n_scalars,
                 int agg, double *out, void *ws, size_t ws_bytes, void *stream)
{
    using namespace fo;
    if (!post || !X || !B) return FO_ERR_NULL;
    if (n_sides > 0 && !sides) return FO_ERR_NULL;
    if (agg != FO_ROW_COL_AGG_B1_T && agg != FO_ROW_NO_AGG_B1) return FO_ERR_UNSUPPORTED;
    if (X->kind != FO_DENSE && X->kind != FO_CSR) return FO_ERR_SHAPE;
    const bool csr = X->kind == FO_CSR;
    const long long rows = csr ? X->csr.rows : X->dense.rows, cols = csr ? X->csr.cols : X->dense.cols;
    if (rows < 0 || cols < 0) return FO_ERR_SHAPE;
    if (csr) {
        if (X->csr.nnz < 0 || X->csr.nnz >= (1ll << 31)) return FO_ERR_UNSUPPORTED;
        if (!X->csr.rowptr) return FO_ERR_NULL;
        if (X->csr.nnz > 0 && (!X->csr.colidx || !X->csr.vals)) return FO_ERR_NULL;
    } else {
        if (X->dense.ld < cols) return FO_ERR_SHAPE;
        if (rows > 0 && cols > 0 && !X->dense.data) return FO_ERR_NULL;
    }
    if (B->rows != cols || B->cols < 1 || B->ld < B->cols) return FO_ERR_SHAPE;
    if (B->cols > FO_B1_MAX_K) return FO_ERR_UNSUPPORTED;
    if (cols > 0 && !B->data) return FO_ERR_NULL;
    const int k = (int)B->cols;
    if (!out && (agg == FO_ROW_COL_AGG_B1_T ? cols : rows) > 0) return FO_ERR_NULL;
    if (n_sides < 0 || n_sides > FO_MAX_SIDES) return FO_ERR_UNSUPPORTED;
    if (pre && n_sides + 1 > FO_MAX_SIDES) return FO_ERR_UNSUPPORTED;

    // the second chain sees the row sum of the first as one more side input
    DevChain chpre, chpost;
    memset(&chpre, 0, sizeof(chpre));
    int rc;
    if (pre) {
        rc = translate_chain(pre, kUseRow, n_sides, scalars, n_scalars, 1, 1, &chpre);
        if (rc != FO_OK) return rc;
    }
    rc = translate_chain(post, kUseRow, n_sides + (pre ? 1 : 0), scalars, n_scalars, 1, 1, &chpost);
    if (rc != FO_OK) return rc;

    B1Params p;
    memset(&p, 0, sizeof(p));
    p.rows = rows; p.cols = cols;
    if (!csr) { p.X = X->dense.data; p.ldx = X->dense.ld; }
    p.B = B->data; p.ldb = B->ld; p.k = k;
    p.has_pre = pre ? 1 : 0;
    p.sides.n = n_sides;
    for (int j = 0; j < n_sides; ++j) {
        const fo_side &s = sides[j];
        if (s.sparse) return FO_ERR_UNSUPPORTED;       // sparse sides: CSR main input of Cell / MAgg only
        if (s.access == FO_AT_CELL) {
            if (s.m.rows != rows || s.m.cols != k || s.m.ld < k) return FO_ERR_SHAPE;
        } else if (s.access == FO_AT_ROW) {
            if (s.m.rows != rows || s.m.cols != 1 || s.m.ld < 1) return FO_ERR_SHAPE;
        } else if (s.access == FO_AT_COL) {
            if (s.m.rows != 1 || s.m.cols != k) return FO_ERR_SHAPE;
        } else {
            return FO_ERR_SHAPE;
        }
        if (rows > 0 && !s.m.data) return FO_ERR_NULL;
        p.sides.s[j].data = s.m.data;
        p.sides.s[j].ld = s.m.ld;
        p.sides.s[j].access = s.access;
    }
    p.side_used = (chpre.side_used | chpost.side_used) & ((1u << n_sides) - 1u);

    if (agg == FO_ROW_COL_AGG_B1_T && cols * k > kB1MaxOutTile) return FO_ERR_UNSUPPORTED;
    B1Shape sh = {0, 0, 0, 0, 0};
    if (!csr && !b1_shape(cols, k, &sh)) return FO_ERR_UNSUPPORTED;
    const int kp_csr = pow2_at_least(k < 2 ? 2 : k);
    if (csr && cols * kp_csr > kB1CsrMaxTile) return FO_ERR_UNSUPPORTED;

    // chains evaluated inline: the identity (t(X) (X B)) and the inner loop of Eq. 2
    p.chain_kind = kB1Generic;
    if (!pre && chpost.n_ops == 0 && chpost.out[0] == 0) p.chain_kind = kB1Identity;
    if (pre && n_sides == 1 && sides[0].access == FO_AT_CELL) {
        char e1[96], e2[96];
        if (chain_expression(chpre, 0, e1, sizeof(e1)) == 0 && chain_expression(chpost, 0, e2, sizeof(e2)) == 0) {
            const bool pre_ok = !strcmp(e1, "mul(r1,r0)") || !strcmp(e1, "mul(r0,r1)");
            const bool post_ok = !strcmp(e2, "sub(mul(r1,r0),mul(r1,r2))") || !strcmp(e2, "sub(mul(r0,r1),mul(r1,r2))") ||
                                 !strcmp(e2, "sub(mul(r1,r0),mul(r2,r1))") || !strcmp(e2, "sub(mul(r0,r1),mul(r2,r1))");
            if (pre_ok && post_ok) p.chain_kind = kB1Mlogreg;
        }
    }

    rc = check_workspace(ws, ws_bytes, b1_ws_bytes(cols, k, agg));
    if (rc != FO_OK) return rc;
    p.head = (WsHead *)ws;
    p.partials = (double *)((char *)ws + sizeof(WsHead));
    p.out = out;
    cudaStream_t st = (cudaStream_t)stream;

    if (rows == 0 || (cols == 0 && agg == FO_ROW_COL_AGG_B1_T)) {
        const long long nout = agg == FO_ROW_COL_AGG_B1_T ? cols * k : 0;
        if (nout > 0) {
            const long long b = (nout + 255) / 256;
            b1_fill_zero_kernel<<<(unsigned)(b > 1024 ? 1024 : b), 256, 0, st>>>(out, nout);
        }
        const cudaError_t e = cudaGetLastError();
        return e == cudaSuccess ? FO_OK : cuda_fail(e);
    }

    const int sms = sm_count();
    if (sms <= 0) return cuda_fail(cudaErrorNoDevice);
    if (csr) {
        B1CsrParams q;
        memset(&q, 0, sizeof(q));
        q.rowptr = X->csr.rowptr; q.colidx = X->csr.colidx; q.vals = X->csr.vals;
        q.rows = rows; q.cols = cols; q.B = B->data; q.ldb = B->ld; q.k = k;
        q.sides = p.sides; q.head = p.head; q.partials = p.partials; q.out = out;
        q.chain_kind = p.chain_kind; q.has_pre = p.has_pre; q.side_used = p.side_used;
        const size_t smem = (size_t)cols * kp_csr * 8 * (agg == FO_ROW_COL_AGG_B1_T ? 2 : 1)
                            + (size_t)kB1CsrWarps * kB1CsrStage * 12;
        long long grid = (rows + kB1CsrThreads - 1) / kB1CsrThreads;
        const long long cap = (long long)sms * (smem <= 100 * 1024 ? 2 : 1);
        if (grid > cap) grid = cap;
        if (grid > b1_grid_cap()) grid = b1_grid_cap();
        if (grid < 1) grid = 1;
        auto go = [&](auto kern) -> cudaError_t {
            cudaError_t e2 = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e2 != cudaSuccess) return e2;
            kern<<<(unsigned)grid, kB1CsrThreads, smem, st>>>(chpre, chpost, q);
            return cudaGetLastError();
        };
        const bool generic = p.chain_kind == kB1Generic;
        auto by_kp = [&](auto kpc) -> cudaError_t {
            constexpr int KP = decltype(kpc)::value;
            if (agg == FO_ROW_COL_AGG_B1_T)
                return generic ? go(row_b1_csr_kernel<KP, kB1ColT, true>) : go(row_b1_csr_kernel<KP, kB1ColT, false>);
            return generic ? go(row_b1_csr_kernel<KP, kB1None, true>) : go(row_b1_csr_kernel<KP, kB1None, false>);
        };
        cudaError_t e2;
        if (kp_csr == 2) e2 = by_kp(std::integral_constant<int, 2>());
        else if (kp_csr == 4) e2 = by_kp(std::integral_constant<int, 4>());
        else if (kp_csr == 8) e2 = by_kp(std::integral_constant<int, 8>());
        else if (kp_csr == 16) e2 = by_kp(std::integral_constant<int, 16>());
        else e2 = by_kp(std::integral_constant<int, 32>());
        return e2 == cudaSuccess ? FO_OK : cuda_fail(e2);
    }
    const bool staged = b1_aligned16(p.X) && (p.ldx % 2 == 0) && (cols % 2 == 0) && cols >= 2;
    // narrow rows: a thread per row (the knob b1.narrow = 0 switches it off)
    {
        const int nc = cols <= 8 ? 8 : 16, kc = k <= 2 ? 2 : k <= 4 ? 4 : 8;
        if (tune_int("b1.narrow", 1) != 0 && cols <= 16 && k <= 8 && nc * kc <= 64) {
            const bool vec = b1_aligned16(p.X) && (p.ldx % 2 == 0) && (cols % 2 == 0);
            long long grid = (rows + kB1NarrowThreads - 1) / kB1NarrowThreads;
            const long long cap = (long long)sms * 2 < b1_grid_cap() ? (long long)sms * 2 : b1_grid_cap();
            if (grid > cap) grid = cap;
            if (grid < 1) grid = 1;
            auto gon = [&](auto ncc, auto kcc) -> cudaError_t {
                constexpr int NC = decltype(ncc)::value, KC = decltype(kcc)::value;
                if (agg == FO_ROW_COL_AGG_B1_T) {
                    if (vec) row_b1_narrow_kernel<NC, KC, kB1ColT, true><<<(unsigned)grid, kB1NarrowThreads, 0, st>>>(chpre, chpost, p);
                    else row_b1_narrow_kernel<NC, KC, kB1ColT, false><<<(unsigned)grid, kB1NarrowThreads, 0, st>>>(chpre, chpost, p);
                } else {
                    if (vec) row_b1_narrow_kernel<NC, KC, kB1None, true><<<(unsigned)grid, kB1NarrowThreads, 0, st>>>(chpre, chpost, p);
                    else row_b1_narrow_kernel<NC, KC, kB1None, false><<<(unsigned)grid, kB1NarrowThreads, 0, st>>>(chpre, chpost, p);
                }
                return cudaGetLastError();
            };
            using I2 = std::integral_constant<int, 2>;
            using I4 = std::integral_constant<int, 4>;
            using I8 = std::integral_constant<int, 8>;
            using I16 = std::integral_constant<int, 16>;
            cudaError_t en;
            if (nc == 8) en = kc == 2 ? gon(I8(), I2()) : kc == 4 ? gon(I8(), I4()) : gon(I8(), I8());
            else en = kc == 2 ? gon(I16(), I2()) : gon(I16(), I4());
            return en == cudaSuccess ? FO_OK : cuda_fail(en);
        }
    }
    // tensor-core variant where its layout fits (the knob b1.mma = 0 / 1 forces the choice)
    {
        MmaShape ms;
        const int forced = tune_int("b1.mma", -1);
        const bool want = forced >= 0 ? forced != 0 : (k > 2 || cols <= 160);
        // 8 warps (two per scheduler, up to 255 registers each) measured faster than 16
        // warps of 128 registers in every layout tried: 0.81 against 1.06 ms at best for
        // 5 000 000 x 100, k = 8
        const int nw = 8;
        if (want && staged && b1_mma_shape(cols, k, nw, &ms)) {
            const int groups = nw / (ms.w * ms.kb);
            const int ns = b1_mma_stride(cols);
            const size_t slot_bytes = (size_t)8 * ns * 8;
            const size_t budget = 208 * 1024;
            int stages = (int)((budget - 64) / (slot_bytes * groups));
            if (stages > 6) stages = 6;
            if (stages * groups > kMmaMaxSlots) stages = kMmaMaxSlots / groups;
            if (stages >= 2) {
                p.W = ms.w; p.KW = ms.kb; p.ns = ns; p.stages = stages;
                size_t smem = slot_bytes * groups * stages + 64;      // 8 doubles of slack behind the rings
                const size_t qs_bytes = agg == FO_ROW_COL_AGG_B1_T ? (size_t)cols * k * 8 : 0;
                if (smem < qs_bytes) smem = qs_bytes;
                const long long ntiles = (rows + 7) / 8;
                long long grid = (ntiles + groups - 1) / groups;
                if (grid > sms) grid = sms;
                if (grid < 1) grid = 1;
                cudaError_t e = cudaErrorInvalidValue;
                if (ms.ncb == 8) e = b1_mma_launch<8, 8>(chpre, chpost, p, agg, (int)grid, smem, st);
                else if (ms.ncb == 14) e = b1_mma_launch<8, 14>(chpre, chpost, p, agg, (int)grid, smem, st);
                else if (ms.ncb == 16) e = b1_mma_launch<8, 16>(chpre, chpost, p, agg, (int)grid, smem, st);
                else if (ms.ncb == 20) e = b1_mma_launch<8, 20>(chpre, chpost, p, agg, (int)grid, smem, st);
                return e == cudaSuccess ? FO_OK : cuda_fail(e);
            }
        }
    }
    const int groups = kB1Warps / (sh.w * sh.kw);
    p.W = sh.w; p.KW = sh.kw;
    const size_t bt_bytes = (size_t)sh.kl * sh.kw * 64 * sh.nch * sh.w * 8;
    const size_t slot_bytes = (size_t)sh.r * cols * 8;
    int stages = 0;
    if (staged) {
        if (bt_bytes + 2 * slot_bytes * groups > kB1SmemBudget) return FO_ERR_UNSUPPORTED;
        stages = (int)((kB1SmemBudget - bt_bytes) / (slot_bytes * groups));
        if (stages > 8) stages = 8;
        if (stages * groups > kB1MaxSlots) stages = kB1MaxSlots / groups;
    }
    p.stages = stages;
    size_t smem = bt_bytes + slot_bytes * groups * stages;
    const size_t qs_bytes = agg == FO_ROW_COL_AGG_B1_T ? (size_t)cols * k * 8 : 0;
    if (smem < qs_bytes) smem = qs_bytes;
    const long long ntiles = (rows + sh.r - 1) / sh.r;
    long long grid = (ntiles + groups - 1) / groups;
    if (grid > sms) grid = sms;
    if (grid > b1_grid_cap()) grid = b1_grid_cap();
    if (grid < 1) grid = 1;

    cudaError_t e = cudaErrorInvalidValue;
#define FO_B1(A, B_, C) \
    if (sh.nch == A && sh.r == B_ && sh.kl == C) \
        e = b1_launch_shape<A, B_, C>(chpre, chpost, p, agg, staged, (int)grid, smem, st);
    FO_B1(1, 8, 2) FO_B1(2, 4, 2) FO_B1(4, 2, 2) FO_B1(1, 4, 4) FO_B1(2, 2, 4) FO_B1(1, 2, 8)
#undef FO_B1
    return e == cudaSuccess ? FO_OK : cuda_fail(e);
}

}  // extern "C"
