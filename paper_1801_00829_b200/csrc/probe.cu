// Two machine-rate probes for the roofline of the Outer template: how fast
// whole factor rows can be gathered at random from a matrix that fits in L2, and
// how fast fp64 fused multiply-adds issue from registers.  They compute nothing
// the fused operators need; the benchmark divides the Outer kernel's gather
// bytes and FMA count by these rates.
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"
#include "fusedops_tools.h"

namespace fo {
namespace {

constexpr int kProbeCtasPerSm = 8;

// An 8-lane group per gathered row (the access shape of the Outer kernels),
// four rows per group in flight; every lane adds up what it loaded.
__global__ void __launch_bounds__(kThreads)
probe_gather_kernel(const double *__restrict__ V, long long ldv, int half, const int *__restrict__ idx,
                    long long n, double *__restrict__ out)
{
    const int lane = threadIdx.x & 31, l8 = lane & 7;
    const long long group = ((long long)blockIdx.x * kThreads + threadIdx.x) >> 3;
    const long long ngroups = ((long long)gridDim.x * kThreads) >> 3;
    double acc = 0.0;
    for (long long i = group * 4; i < n; i += ngroups * 4) {
        const double2 *row[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long r = i + u < n ? __ldg(idx + i + u) : __ldg(idx + i);
            row[u] = reinterpret_cast<const double2 *>(V + r * ldv);
        }
        for (int k = l8; k < half; k += 8) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const double2 x = __ldg(row[u] + k);
                acc += x.x + x.y;
            }
        }
    }
    out[(long long)blockIdx.x * kThreads + threadIdx.x] = acc;
}

// Eight independent multiply-add chains per thread.
__global__ void __launch_bounds__(kThreads)
probe_fma_kernel(long long iters, double a, double b, double *__restrict__ out)
{
    double x[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) x[k] = (double)(threadIdx.x + k) * 1e-3;
    for (long long i = 0; i < iters; ++i) {
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = fma(x[k], a, b);
    }
    double s = 0.0;
#pragma unroll
    for (int k = 0; k < 8; ++k) s += x[k];
    out[(long long)blockIdx.x * kThreads + threadIdx.x] = s;
}

}  // namespace
}  // namespace fo

using namespace fo;

extern "C" size_t fo_probe_out_len(void)
{
    const int sms = sm_count();
    return sms > 0 ? (size_t)sms * kProbeCtasPerSm * kThreads : 0;
}

extern "C" int fo_probe_l2_gather(const fo_dense *V, const int *idx, long long n, double *out, void *stream)
{
    if (!V || !out || (n > 0 && !idx)) return FO_ERR_NULL;
    if (V->rows <= 0 || V->cols <= 0 || V->ld < V->cols || n < 0) return FO_ERR_SHAPE;
    if (!V->data) return FO_ERR_NULL;
    if ((V->cols & 1) || (V->ld & 1) || ((uintptr_t)V->data & 15u)) return FO_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return cuda_fail(cudaErrorNoDevice);
    probe_gather_kernel<<<sms * kProbeCtasPerSm, kThreads, 0, (cudaStream_t)stream>>>(
        V->data, V->ld, (int)(V->cols / 2), idx, n, out);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? FO_OK : cuda_fail(e);
}

extern "C" int fo_probe_fp64_fma(long long iters, double *out, void *stream)
{
    if (!out) return FO_ERR_NULL;
    if (iters < 0) return FO_ERR_SHAPE;
    const int sms = sm_count();
    if (sms <= 0) return cuda_fail(cudaErrorNoDevice);
    probe_fma_kernel<<<sms * kProbeCtasPerSm, kThreads, 0, (cudaStream_t)stream>>>(iters, 0.999999, 1e-6, out);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? FO_OK : cuda_fail(e);
}
