// Outer template (Table 1; Fig. 1(d); Eq. 1 and the outer-product listing of
// Section 2.2): for every stored cell (i, j) of the CSR matrix X evaluate
// w = chain(a = X_ij, d = U_i . V_j) and aggregate.  U V^T is never formed.
//
// Schedule: CTAs own contiguous row ranges holding equal shares of the stored
// cells (binary search on rowptr); inside a CTA a warp owns a row at a time.
// The row U_i sits in registers, spread over the 8 lanes of a group; the four
// groups of a warp take stored cells p, p+1, p+2, p+3 of the row and gather
// their V_j rows with 128-bit loads (V is read many times and stays in L2).
#include "chain.cuh"

namespace fo {

namespace {

struct OuterParams {
    const int *rowptr;
    const int *colidx;
    const double *vals;
    long long rows, cols, nnz;
    int rank, pad;
    const double *U;
    long long ldu;
    const double *V;
    long long ldv;
    WsHead *head;
    double *partials;
    double *out;
};

enum { kOutFull = 0, kOutNone = 1, kOutRight = 2 };

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

__device__ __forceinline__ double outer_chain(const DevChain &ch, double a, double d)
{
    RegFile<kRegs, 1> f;
    f.r[0][0] = a;
    f.r[1][0] = d;
    run_chain<kRegs, 1>(ch, f);
    double o[1];
    operand<kRegs, 1>(ch, f, ch.out[0], o);
    return o[0];
}

__device__ __forceinline__ double group_sum(double v, unsigned gmask)
{
    v += __shfl_xor_sync(gmask, v, 4);
    v += __shfl_xor_sync(gmask, v, 2);
    v += __shfl_xor_sync(gmask, v, 1);
    return v;
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
template <int NK2, int AGG, bool ALIGNED>
__global__ void __launch_bounds__(kThreads)
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
    const unsigned gmask = 0xffu << (lane & 24);
    const int rank = p.rank;
    double acc = 0.0;

    for (long long row = row_lo + warp; row < row_hi; row += kThreads / 32) {
        const int beg = __ldg(p.rowptr + row), end = __ldg(p.rowptr + row + 1);
        if (beg == end) {
            if (AGG == kOutRight) {
                for (int c = lane; c < rank; c += 32) p.out[row * rank + c] = 0.0;
            }
            continue;
        }
        double2 u[NK2], racc[NK2];
        const double *urow = p.U + row * p.ldu;
#pragma unroll
        for (int c = 0; c < NK2; ++c) {
            u[c] = ld_pair_cached<ALIGNED>(urow, 16 * c + 2 * l8, rank);
            racc[c] = make_double2(0.0, 0.0);
        }
        for (int q0 = beg + grp; q0 < end; q0 += 8) {
            // two stored cells per group and trip: q0 and q0 + 4
            const int q1 = q0 + 4;
            const bool two = q1 < end;
            const int j0 = __ldg(p.colidx + q0);
            const int j1 = two ? __ldg(p.colidx + q1) : j0;
            const double a0 = __ldg(p.vals + q0);
            const double a1 = two ? __ldg(p.vals + q1) : 0.0;
            const double *v0 = p.V + (long long)j0 * p.ldv;
            const double *v1 = p.V + (long long)j1 * p.ldv;
            double2 x0[NK2], x1[NK2];
#pragma unroll
            for (int c = 0; c < NK2; ++c) {
                x0[c] = ld_pair_cached<ALIGNED>(v0, 16 * c + 2 * l8, rank);
                x1[c] = ld_pair_cached<ALIGNED>(v1, 16 * c + 2 * l8, rank);
            }
            double d0 = 0.0, d1 = 0.0;
#pragma unroll
            for (int c = 0; c < NK2; ++c) {
                d0 = fma(u[c].x, x0[c].x, d0);
                d0 = fma(u[c].y, x0[c].y, d0);
                d1 = fma(u[c].x, x1[c].x, d1);
                d1 = fma(u[c].y, x1[c].y, d1);
            }
            d0 = group_sum(d0, gmask);
            d1 = group_sum(d1, gmask);
            // lane 0 of the group evaluates cell q0, lane 1 cell q1 (one pass of the chain)
            const double a = (l8 == 1) ? a1 : a0;
            const double d = (l8 == 1) ? d1 : d0;
            const double w = outer_chain(ch, a, d);
            if (AGG == kOutFull) {
                if (l8 == 0 || (l8 == 1 && two)) acc += w;
            } else if (AGG == kOutNone) {
                if (l8 == 0) p.out[q0] = w;
                if (l8 == 1 && two) p.out[q1] = w;
            } else {
                const double w0 = __shfl_sync(gmask, w, (lane & 24) + 0);
                const double w1 = two ? __shfl_sync(gmask, w, (lane & 24) + 1) : 0.0;
#pragma unroll
                for (int c = 0; c < NK2; ++c) {
                    racc[c].x = fma(w0, x0[c].x, racc[c].x);
                    racc[c].y = fma(w0, x0[c].y, racc[c].y);
                    racc[c].x = fma(w1, x1[c].x, racc[c].x);
                    racc[c].y = fma(w1, x1[c].y, racc[c].y);
                }
            }
        }
        if (AGG == kOutRight) {
            // the four groups hold partial rows: add them in a fixed order
#pragma unroll
            for (int c = 0; c < NK2; ++c) {
                racc[c].x += __shfl_xor_sync(0xffffffffu, racc[c].x, 8);
                racc[c].y += __shfl_xor_sync(0xffffffffu, racc[c].y, 8);
                racc[c].x += __shfl_xor_sync(0xffffffffu, racc[c].x, 16);
                racc[c].y += __shfl_xor_sync(0xffffffffu, racc[c].y, 16);
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
    else FO_GO(kOutRight);
#undef FO_GO
    return cudaGetLastError();
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
    if (agg == FO_OUTER_LEFT_MM) return FO_ERR_UNSUPPORTED;
    if (agg != FO_OUTER_FULL_AGG && agg != FO_OUTER_NO_AGG && agg != FO_OUTER_RIGHT_MM)
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
    cudaStream_t st = (cudaStream_t)stream;

    if (X->nnz == 0 || X->rows == 0) {
        const long long nout = agg == FO_OUTER_FULL_AGG ? 1
                             : agg == FO_OUTER_RIGHT_MM ? X->rows * rank : 0;
        if (nout > 0) {
            const long long b = (nout + 255) / 256;
            outer_fill_zero_kernel<<<(unsigned)(b > 1024 ? 1024 : b), 256, 0, st>>>(out, nout);
        }
        const cudaError_t e = cudaGetLastError();
        return e == cudaSuccess ? FO_OK : cuda_fail(e);
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
    if (nk2 <= 1) e = launch_outer<1>(ch, p, agg, aligned, (int)grid, st);
    else if (nk2 <= 2) e = launch_outer<2>(ch, p, agg, aligned, (int)grid, st);
    else if (nk2 <= 4) e = launch_outer<4>(ch, p, agg, aligned, (int)grid, st);
    else if (nk2 <= 7) e = launch_outer<7>(ch, p, agg, aligned, (int)grid, st);
    else if (nk2 <= 8) e = launch_outer<8>(ch, p, agg, aligned, (int)grid, st);
    else e = launch_outer<16>(ch, p, agg, aligned, (int)grid, st);
    return e == cudaSuccess ? FO_OK : cuda_fail(e);
}

}  // extern "C"
