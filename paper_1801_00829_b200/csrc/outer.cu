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

#include <atomic>

#include "jit.h"
#include "outer_kernels.cuh"

namespace fo {

namespace {

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

// full_agg / no_agg / right_mm through the pipelined kernel; NK2 is exactly ceil(rank / 16).
template <int NK2, int AGG, bool GENERIC>
cudaError_t launch_outer_pipe_gen(const DevChain &ch, const OuterParams &p, int grid, cudaStream_t st)
{
    const size_t smem = (size_t)(kThreads / 32) * kStageRows * p.rank * sizeof(double);
    // the attribute sticks to the function: raise it when a call needs more than any before
    static std::atomic<size_t> granted[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || granted[dev].load(std::memory_order_relaxed) < smem) {
        e = cudaFuncSetAttribute(outer_pipe_kernel<NK2, AGG, GENERIC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) granted[dev].store(smem, std::memory_order_relaxed);
    }
    outer_pipe_kernel<NK2, AGG, GENERIC><<<grid, kThreads, smem, st>>>(ch, p);
    return cudaGetLastError();
}

// an instance with the interpreter for chains without an inline form, one without it for the rest
template <int NK2, int AGG>
cudaError_t launch_outer_pipe_one(const DevChain &ch, const OuterParams &p, int grid, cudaStream_t st)
{
    return p.chain_kind == kOuterGeneric ? launch_outer_pipe_gen<NK2, AGG, true>(ch, p, grid, st)
                                         : launch_outer_pipe_gen<NK2, AGG, false>(ch, p, grid, st);
}

template <int NK2>
cudaError_t launch_outer_pipe(const DevChain &ch, const OuterParams &p, int agg, int grid, cudaStream_t st)
{
    if (agg == FO_OUTER_FULL_AGG) return launch_outer_pipe_one<NK2, kOutFull>(ch, p, grid, st);
    if (agg == FO_OUTER_NO_AGG) return launch_outer_pipe_one<NK2, kOutNone>(ch, p, grid, st);
    return launch_outer_pipe_one<NK2, kOutRight>(ch, p, grid, st);
}

// full_agg / no_agg through the bulk-copy kernel; NK2 is exactly ceil(rank / 16) (at most 7 here).

template <int NK2, int AGG, int KIND>
cudaError_t launch_outer_bulk_one(const DevChain &ch, const OuterParams &p, int grid, int warps, size_t smem,
                                  cudaStream_t st)
{
    static std::atomic<size_t> granted[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || granted[dev].load(std::memory_order_relaxed) < smem) {
        e = cudaFuncSetAttribute(outer_bulk_kernel<NK2, AGG, KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) granted[dev].store(smem, std::memory_order_relaxed);
    }
    outer_bulk_kernel<NK2, AGG, KIND><<<grid, warps * 32, smem, st>>>(ch, p);
    return cudaGetLastError();
}

// three instances: the interpreter and the logarithm chain (evaluated once per four stages), and the
// cheap inline forms (evaluated per stage)
template <int NK2, int AGG>
cudaError_t launch_outer_bulk_agg(const DevChain &ch, const OuterParams &p, int grid, int warps, size_t smem,
                                  cudaStream_t st)
{
    switch (p.chain_kind) {
        case kOuterGeneric: return launch_outer_bulk_one<NK2, AGG, kOuterGeneric>(ch, p, grid, warps, smem, st);
        case kOuterXlogd: return launch_outer_bulk_one<NK2, AGG, kOuterXlogd>(ch, p, grid, warps, smem, st);
        default: return launch_outer_bulk_one<NK2, AGG, kOuterWsloss>(ch, p, grid, warps, smem, st);   // the cheap inline forms
    }
}

template <int NK2>
cudaError_t launch_outer_bulk(const DevChain &ch, const OuterParams &p, int agg, int grid, int warps, size_t smem,
                              cudaStream_t st)
{
    if (agg == FO_OUTER_FULL_AGG) return launch_outer_bulk_agg<NK2, kOutFull>(ch, p, grid, warps, smem, st);
    return launch_outer_bulk_agg<NK2, kOutNone>(ch, p, grid, warps, smem, st);
}

// Work split of the tiled schedule: column ranges so that there are enough work items for a
// few rounds over the SMs (the last round a small share), and the grid.
bool dense_plan(const OuterParams &p, int sms, DenseSplit *sp, long long *grid)
{
    const long long ntiles = (p.cols + kDenseBN - 1) / kDenseBN;
    const long long rb = (p.rows + kDenseBM - 1) / kDenseBM;
    long long splits = (8ll * sms + rb - 1) / rb;
    if (splits < 1) splits = 1;
    if (splits > ntiles) splits = ntiles;
    const long long per = (ntiles + splits - 1) / splits;
    splits = (ntiles + per - 1) / per;
    if (rb > 0x7fffffffll / splits) return false;
    sp->row_blocks = (int)rb;
    sp->col_splits = (int)splits;
    sp->tiles_per_split = (int)per;
    sp->pad = 0;
    *grid = rb * splits;
    if (*grid > sms) *grid = sms;
    return true;
}

// full_agg / no_agg through the tiled schedule for densely stored inputs.
template <int AGG>
cudaError_t launch_outer_dense_one(const DevChain &ch, const OuterParams &p, int sms, cudaStream_t st)
{
    const size_t smem = dense_smem_bytes(p.rank);
    static std::atomic<size_t> granted[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || granted[dev].load(std::memory_order_relaxed) < smem) {
        e = cudaFuncSetAttribute(outer_dense_kernel<AGG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) granted[dev].store(smem, std::memory_order_relaxed);
    }
    DenseSplit sp;
    long long grid = 0;
    if (!dense_plan(p, sms, &sp, &grid)) return cudaErrorInvalidValue;
    outer_dense_kernel<AGG><<<(unsigned)grid, kDenseThreadsAll, smem, st>>>(ch, p, sp);
    return cudaGetLastError();
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
                const fo_side *sides, int n_sides, const double *scalars, int n_scalars, int agg, double *out,
                long long *out_nnz, void *ws, size_t ws_bytes, void *stream)
{
    using namespace fo;
    if (!chain || !X || !U || !V || !out) return FO_ERR_NULL;
    if (n_sides > 0 && !sides) return FO_ERR_NULL;
    if (agg != FO_OUTER_FULL_AGG && agg != FO_OUTER_NO_AGG && agg != FO_OUTER_RIGHT_MM &&
        agg != FO_OUTER_LEFT_MM)
        return FO_ERR_UNSUPPORTED;
    if (out_nnz && agg != FO_OUTER_NO_AGG) return FO_ERR_UNSUPPORTED;     // a count needs an elementwise result
    if (X->rows < 0 || X->cols < 0 || X->nnz < 0) return FO_ERR_SHAPE;
    if (X->nnz >= (1ll << 31)) return FO_ERR_UNSUPPORTED;
    if (U->rows != X->rows || V->rows != X->cols || U->cols != V->cols) return FO_ERR_SHAPE;
    if (U->ld < U->cols || V->ld < V->cols) return FO_ERR_SHAPE;
    const int rank = (int)U->cols;
    if (U->cols > 256) return FO_ERR_UNSUPPORTED;
    if (!X->rowptr) return FO_ERR_NULL;
    if (X->nnz > 0 && (!X->colidx || !X->vals)) return FO_ERR_NULL;
    if (rank > 0 && ((X->rows > 0 && !U->data) || (X->cols > 0 && !V->data))) return FO_ERR_NULL;
    if (out_nnz) {
        // the elementwise result first, then one more pass over it for the count
        const int rc0 = fused_outer(chain, X, U, V, sides, n_sides, scalars, n_scalars, agg, out, nullptr, ws,
                                    ws_bytes, stream);
        if (rc0 != FO_OK) return rc0;
        const cudaError_t ce = launch_count_nonzero(out, X->nnz, out_nnz, (cudaStream_t)stream);
        return ce == cudaSuccess ? FO_OK : cuda_fail(ce);
    }

    DevChain ch;
    int rc = translate_chain(chain, kUseOuter, n_sides, scalars, n_scalars, 1, 1, &ch);
    if (rc != FO_OK) return rc;
    rc = check_workspace(ws, ws_bytes, fused_outer_workspace_bytes(X, rank, agg));
    if (rc != FO_OK) return rc;

    OuterParams p;
    memset(&p, 0, sizeof(p));
    p.sides.n = n_sides;
    for (int k = 0; k < n_sides; ++k) {
        const fo_side &sd = sides[k];
        if (sd.sparse) return FO_ERR_UNSUPPORTED;            // dense side inputs only
        if (sd.m.rows < 0 || sd.m.cols < 0 || sd.m.ld < sd.m.cols) return FO_ERR_SHAPE;
        const bool fits = sd.access == FO_AT_CELL ? (sd.m.rows == X->rows && sd.m.cols == X->cols)
                        : sd.access == FO_AT_ROW ? (sd.m.rows == X->rows && sd.m.cols == 1)
                        : sd.access == FO_AT_COL ? (sd.m.rows == 1 && sd.m.cols == X->cols) : false;
        if (!fits) return FO_ERR_SHAPE;
        if (sd.m.rows > 0 && sd.m.cols > 0 && !sd.m.data) return FO_ERR_NULL;
        p.sides.s[k].data = sd.m.data;
        p.sides.s[k].ld = sd.m.ld;
        p.sides.s[k].access = sd.access;
    }
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
    // factor rows that are whole 16-byte pieces can be copied asynchronously into shared memory
    // (a chain that reads side inputs runs through the kernel that gathers into registers:
    // it is the one that knows every cell's row and column where the chain is evaluated)
    const bool copyable = aligned && rank % 2 == 0 && rank >= 2 && nk2 <= 8 && agg != FO_OUTER_LEFT_MM &&
                          ch.side_used == 0;
    char which[48] = "";
    tune_get("outer.kernel", which, sizeof(which));
    const bool want_direct = strcmp(which, "direct") == 0;
    // densely stored inputs: forming the tiles of U V^T beats a gathered row per stored cell
    // once about one cell in seven is stored (measured crossover on this part)
    const bool want_dense = strcmp(which, "dense") == 0;
    const bool dense_ok = copyable && agg != FO_OUTER_RIGHT_MM && rank >= 8 &&
                          dense_smem_bytes(rank) <= 220u * 1024u;
    const double stored_share = (double)X->nnz / ((double)X->rows * (double)X->cols);
    // a chain without an inline form: the same kernels compiled for it at run time, else interpreted
    const bool try_jit = p.chain_kind == kOuterGeneric && !force_interpreter();
    const int kagg = agg == FO_OUTER_FULL_AGG ? kOutFull : agg == FO_OUTER_NO_AGG ? kOutNone
                     : agg == FO_OUTER_RIGHT_MM ? kOutRight : kOutLeft;
    if (dense_ok && (want_dense || (which[0] == 0 && stored_share >= 0.15 && X->rows >= 64 && X->cols >= 64))) {
        if (try_jit) {
            DenseSplit sp;
            long long g = 0;
            if (dense_plan(p, sms, &sp, &g)) {
                const JitSpec js = {kJitOuterDense, kagg, 0, 0};
                const int jrc = jit_launch(js, ch, &p, (unsigned)g, 1, st, jit_first_use(), true,
                                           dense_smem_bytes(rank), &sp, kDenseThreadsAll);
                if (jrc == FO_OK) return FO_OK;
                if (jrc != kJitUnavailable) return jrc;
            }
        }
        e = agg == FO_OUTER_FULL_AGG ? launch_outer_dense_one<kOutFull>(ch, p, sms, st)
                                     : launch_outer_dense_one<kOutNone>(ch, p, sms, st);
        return e == cudaSuccess ? FO_OK : cuda_fail(e);
    }
    // full_agg / no_agg: factor rows landed by bulk copies where that measured faster than 16-byte copies -
    // long rows whose 16-byte pieces straddle 128-byte lines (rank 97 .. 112 with a leading dimension that is
    // not a multiple of 16 doubles: 0.58 against 0.66 ms at rank 100), and rows so long that only one CTA of
    // the 16-byte-copy kernel fits on an SM (rank above 112: 0.67 against 0.90 ms at rank 120).  Below rank 97
    // a row is too short to be worth the ~54 cycles its copy holds the warp (rank 80: 0.58 against 0.43 ms).
    const bool want_bulk = strcmp(which, "bulk") == 0, want_pipe = strcmp(which, "pipe") == 0;
    int bulk_warps = (int)((225u * 1024u) / bulk_warp_bytes(rank));
    if (bulk_warps > kBulkWarps) bulk_warps = kBulkWarps;
    const bool bulk_pays = bulk_warps >= 12 && (rank > 112 || (rank > 96 && V->ld % 16 != 0));
    if (copyable && !want_direct && !want_pipe && agg != FO_OUTER_RIGHT_MM && bulk_warps >= 8 &&
        (want_bulk || bulk_pays)) {
        const size_t smem = (size_t)bulk_warps * bulk_warp_bytes(rank);
        long long g = sms;
        const long long by_cells = (X->nnz + 8ll * bulk_warps - 1) / (8ll * bulk_warps);    // a stage per warp at least
        if (g > by_cells) g = by_cells;
        if (g < 1) g = 1;
        if (try_jit) {
            const JitSpec js = {kJitOuterBulk, nk2, kagg, 0};
            const int jrc = jit_launch(js, ch, &p, (unsigned)g, 1, st, jit_first_use(), true, smem, nullptr,
                                       bulk_warps * 32);
            if (jrc == FO_OK) return FO_OK;
            if (jrc != kJitUnavailable) return jrc;
        }
        switch (nk2) {
            case 1: e = launch_outer_bulk<1>(ch, p, agg, (int)g, bulk_warps, smem, st); break;
            case 2: e = launch_outer_bulk<2>(ch, p, agg, (int)g, bulk_warps, smem, st); break;
            case 3: e = launch_outer_bulk<3>(ch, p, agg, (int)g, bulk_warps, smem, st); break;
            case 4: e = launch_outer_bulk<4>(ch, p, agg, (int)g, bulk_warps, smem, st); break;
            case 5: e = launch_outer_bulk<5>(ch, p, agg, (int)g, bulk_warps, smem, st); break;
            case 6: e = launch_outer_bulk<6>(ch, p, agg, (int)g, bulk_warps, smem, st); break;
            case 7: e = launch_outer_bulk<7>(ch, p, agg, (int)g, bulk_warps, smem, st); break;
            default: e = launch_outer_bulk<8>(ch, p, agg, (int)g, bulk_warps, smem, st); break;
        }
        return e == cudaSuccess ? FO_OK : cuda_fail(e);
    }
    if (copyable && !want_direct) {
        if (try_jit) {
            const JitSpec js = {kJitOuterPipe, nk2 > 8 ? 8 : nk2, kagg, 0};
            const int jrc = jit_launch(js, ch, &p, (unsigned)grid, 1, st, jit_first_use(), true,
                                       (size_t)(kThreads / 32) * kStageRows * rank * sizeof(double));
            if (jrc == FO_OK) return FO_OK;
            if (jrc != kJitUnavailable) return jrc;
        }
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
        return e == cudaSuccess ? FO_OK : cuda_fail(e);
    }
    if (try_jit) {
        const int cap = nk2 <= 1 ? 1 : nk2 <= 2 ? 2 : nk2 <= 4 ? 4 : nk2 <= 7 ? 7 : nk2 <= 8 ? 8 : 16;
        const JitSpec js = {kJitOuterDirect, cap, kagg, aligned ? 1 : 0};
        const int jrc = jit_launch(js, ch, &p, (unsigned)grid, 1, st, jit_first_use(), true);
        if (jrc == FO_OK) return FO_OK;
        if (jrc != kJitUnavailable) return jrc;
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
