// Shared device/host helpers of the fused-operator kernels (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "../../include/fusedops.h"

namespace fo {

// ---------------------------------------------------------------- workspace
// Head of every workspace: control words, then the per-CTA partials.
struct WsHead {
    unsigned int ticket;     // CTAs that have published their partial; reset by the last one
    unsigned int status;     // 0, or 1 once a bounded device-side wait ran out
    unsigned int pad[62];
};
static_assert(sizeof(WsHead) == 256, "workspace head is 256 bytes");

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
//   Outer       : R0 = a,  R1 = d
constexpr int kRegs = 13;            // 1 + FO_MAX_SIDES + FO_MAX_TMPS
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

// Host: validate a chain for a template and translate it (chain_host.cu).
enum ChainUse { kUseCell, kUseRow, kUseOuter };
int translate_chain(const fo_chain *chain, ChainUse use, int n_sides,
                    const double *scalars, int n_scalars, int min_out, int max_out,
                    DevChain *out);

int check_workspace(const void *ws, size_t ws_bytes, size_t need);
int cuda_fail(cudaError_t e);
int sm_count();

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

// Publishes this CTA's partial vector (`width` doubles already written to
// partials[blockIdx.x * width ..]) and tells whether this CTA is the last one.
// The last CTA sees every other CTA's partial.  Nobody waits.
__device__ __forceinline__ bool publish_and_is_last(WsHead *head, unsigned int *s_flag)
{
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int prev = atomicAdd(&head->ticket, 1u);
        const bool last = (prev == gridDim.x * gridDim.y - 1);
        if (last) head->ticket = 0u;     // ready for the next call
        *s_flag = last ? 1u : 0u;
        __threadfence();
    }
    __syncthreads();
    return *s_flag != 0u;
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

// Final stage of a vector sum: out[j] = sum_g partials[g * width + j], g ascending.
__device__ __forceinline__ void final_sum_columns(const double *partials, int G, long long width,
                                                  double *out)
{
    for (long long j = threadIdx.x; j < width; j += blockDim.x) {
        double s = 0.0;
        int g = 0;
        for (; g + 8 <= G; g += 8) {
            double t[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) t[u] = __ldcg(partials + (size_t)(g + u) * width + j);
#pragma unroll
            for (int u = 0; u < 8; ++u) s += t[u];
        }
        for (; g < G; ++g) s += __ldcg(partials + (size_t)g * width + j);
        out[j] = s;
    }
}
#endif  // __CUDACC__

}  // namespace fo
