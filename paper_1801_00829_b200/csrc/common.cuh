// Shared device/host helpers of the fused-operator kernels (sm_100a).
#pragma once

// This header is also compiled at run time (NVRTC) as part of specialised
// kernels; there the system headers are not available, so the few fixed-width
// types and the FO_* limits are supplied by the generated source instead.
#ifndef __CUDACC_RTC__
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "../../include/fusedops.h"
#include "../../include/fusedops_tools.h"
#endif

namespace fo {

// ---------------------------------------------------------------- workspace
// Head of every workspace: control words, then the per-CTA partials.  All
// counters are zero between calls: whoever takes the last ticket resets it.
struct WsHead {
    unsigned int ticket;        // CTAs (or groups) that have published; reset by the last one
    unsigned int status;        // 0, or 1 once a bounded device-side wait ran out
    unsigned int pad[62];
    unsigned int group[4032];   // tickets of CTA groups / column tiles
};
static_assert(sizeof(WsHead) == 16384, "workspace head is 16 KB");
constexpr int kMaxGroups = 4032;
constexpr int kGroup = 16;      // CTAs per group in the two-level column reduction

constexpr int kMaxPartials = 2048;   // upper bound on CTAs that publish partials
constexpr int kThreads = 256;        // CTA size of the reduction kernels

// ------------------------------------------------------------- device chain
// The chain as the kernels see it: operands renumbered into one flat register
// file R[0..kRegs) plus a constant table (scalars and immediates merged).
//
// Register layout (inputs sit at fixed places so the kernels fill them without
// a run-time index; temporaries follow, packed by live range):
//   Cell / MAgg : R0 = a,  R(1+k) = side k
//   Row         : R0 = d,  R(1+k) = side k
//   Outer       : R0 = a,  R1 = d,  R(2+k) = side k  (at most kOuterMaxSides sides)
constexpr int kRegs = 13;            // 1 + FO_MAX_SIDES + FO_MAX_TMPS
constexpr int kOuterMaxSides = 3;    // 2 + sides + FO_MAX_TMPS registers must fit kRegs
constexpr int kConsts = 40;          // FO_MAX_SCALARS + FO_MAX_OPS

struct DevOp {
    uint8_t opcode, dst, a, b, c;    // dst: register; a/b/c: register, or 0x80|const index
    uint8_t pad[3];
};

struct DevChain {
    int32_t n_ops;
    int32_t n_out;
    int32_t n_regs;                  // registers in use (upper bound on every index)
    uint32_t side_used;              // bit k: the chain reads side k
    int32_t tmp_base;                // first temporary register (inputs sit below it)
    int32_t pad0;
    uint8_t out[FO_MAX_OUT];         // operand bytes (register or constant)
    DevOp ops[FO_MAX_OPS];
    double consts[kConsts];
};

struct DevSide {
    const double *data;
    long long ld;
    int access;
    int pad;
};

struct DevSides {
    int n;
    int pad;
    DevSide s[FO_MAX_SIDES];
};

#ifndef __CUDACC_RTC__
// Host: validate a chain for a template and translate it (chain_host.cu).
enum ChainUse { kUseCell, kUseRow, kUseOuter };
int translate_chain(const fo_chain *chain, ChainUse use, int n_sides,
                    const double *scalars, int n_scalars, int min_out, int max_out,
                    DevChain *out);

// Host: the k-th result of a translated chain written out as an expression over
// its inputs, e.g. "mul(ne(r0,k0),mul(sub(r0,r1),sub(r0,r1)))": rN is input
// register N, kN entry N of the constant table; sq(x) is written mul(x,x).  Two
// chains with the same text do the same arithmetic in the same order, whatever
// temporaries they were written with.  Writes at most cap - 1 characters;
// returns 0, or -1 if the text does not fit.
int chain_expression(const DevChain &ch, int k, char *text, size_t cap);

// True while fo_set_force_interpreter(1) is in effect: every chain goes through
// the general interpreter (cell.cu).
bool force_interpreter();

// Measurement knobs set through fo_tune (fusedops_tools.h): false / `fallback` unless set.
bool tune_get(const char *name, char *value, size_t cap);
int tune_int(const char *name, int fallback);

int check_workspace(const void *ws, size_t ws_bytes, size_t need);

// *out_nnz (device) = number of values[0..n) that are not zero: one more pass over an
// elementwise result, asynchronous on `st` (cell.cu).
cudaError_t launch_count_nonzero(const double *values, long long n, long long *out_nnz, cudaStream_t st);
int cuda_fail(cudaError_t e);
int sm_count();
#endif

#ifdef __CUDACC__
// ------------------------------------------------------------ device helpers
__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Streaming 128-bit load of read-once data: no L1 allocation.
__device__ __forceinline__ double2 ld_stream2(const double *p)
{
    double2 r;
    asm volatile("ld.global.nc.L1::no_allocate.v2.f64 {%0, %1}, [%2];"
                 : "=d"(r.x), "=d"(r.y) : "l"(p));
    return r;
}
__device__ __forceinline__ double ld_stream1(const double *p)
{
    double r;
    asm volatile("ld.global.nc.L1::no_allocate.f64 %0, [%1];" : "=d"(r) : "l"(p));
    return r;
}

// CTA-wide sum of NV values per thread, in a fixed order: lanes by xor-shuffle
// tree, then warps 0..W-1 sequentially.  Result valid in thread 0.
template <int NV>
__device__ __forceinline__ void block_sum(double (&v)[NV], double *smem /* NV * 32 */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nwarps = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int k = 0; k < NV; ++k) v[k] = warp_sum(v[k]);
    __syncthreads();
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < NV; ++k) smem[k * 32 + warp] = v[k];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            double s = 0.0;
            for (int w = 0; w < nwarps; ++w) s += smem[k * 32 + w];
            v[k] = s;
        }
    }
}

// Takes a ticket; true for the CTA that took the last of `count`.  Every CTA's
// global writes made before the call are visible to that last CTA.
__device__ __forceinline__ bool take_ticket(unsigned int *counter, unsigned int count,
                                            unsigned int *s_flag)
{
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int prev = atomicAdd(counter, 1u);
        const bool last = (prev == count - 1);
        if (last) *counter = 0u;         // ready for the next call
        *s_flag = last ? 1u : 0u;
        __threadfence();
    }
    __syncthreads();
    return *s_flag != 0u;
}

// Tells whether this CTA is the last of the grid to arrive (see take_ticket).
__device__ __forceinline__ bool publish_and_is_last(WsHead *head, unsigned int *s_flag)
{
    return take_ticket(&head->ticket, gridDim.x * gridDim.y, s_flag);
}

// Final stage of a scalar (or k-vector) sum: the last CTA adds the G partials
// of each of `width` outputs in index order and writes out[0..width).
__device__ __forceinline__ void final_sum_small(const double *partials, int G, int width,
                                                double *out, double *smem /* 32 */)
{
    for (int k = 0; k < width; ++k) {
        double s = 0.0;
        for (int g = threadIdx.x; g < G; g += blockDim.x)
            s += __ldcg(partials + (size_t)g * width + k);
        double v[1] = {s};
        block_sum<1>(v, smem);
        if (threadIdx.x == 0) out[k] = v[0];
        __syncthreads();
    }
}

// out[j] = sum_g src[g * width + j], g ascending, for the columns this CTA's
// threads cover.  128-bit loads when `width` is even and src is 16-byte aligned.
__device__ __forceinline__ void sum_columns(const double *src, int G, long long width, double *out)
{
    for (long long j = threadIdx.x; j < width; j += blockDim.x) {
        double s = 0.0;
        int g = 0;
        for (; g + 8 <= G; g += 8) {
            double t[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) t[u] = __ldcg(src + (size_t)(g + u) * width + j);
#pragma unroll
            for (int u = 0; u < 8; ++u) s += t[u];
        }
        for (; g < G; ++g) s += __ldcg(src + (size_t)g * width + j);
        out[j] = s;
    }
}

// Two-level, fixed-order sum of the G per-CTA vectors in `partials` (G x width,
// CTA-major; G <= kGroup * kMaxGroups): the last CTA of each group of kGroup
// CTAs adds that group's vectors into `gpart` (groups x width), the last group
// to finish adds the group vectors into `out`.  Nobody waits.
__device__ __forceinline__ void reduce_columns_two_level(WsHead *head, const double *partials,
                                                         double *gpart, long long width,
                                                         double *out, unsigned int *s_flag)
{
    const int G = gridDim.x, cta = blockIdx.x;
    const int ngroups = (G + kGroup - 1) / kGroup;
    const int gid = cta / kGroup;
    const int gsize = (G - gid * kGroup < kGroup) ? G - gid * kGroup : kGroup;
    if (!take_ticket(&head->group[gid], (unsigned)gsize, s_flag)) return;
    if (ngroups == 1) {
        sum_columns(partials, gsize, width, out);
        return;
    }
    sum_columns(partials + (size_t)gid * kGroup * width, gsize, width, gpart + (size_t)gid * width);
    if (!take_ticket(&head->ticket, (unsigned)ngroups, s_flag)) return;
    sum_columns(gpart, ngroups, width, out);
}
#endif  // __CUDACC__

}  // namespace fo
