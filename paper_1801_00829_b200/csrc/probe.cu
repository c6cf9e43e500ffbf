// Two machine-rate probes for the roofline of the Outer template: how fast
// whole factor rows can be gathered at random from a matrix that fits in L2, and
// how fast fp64 fused multiply-adds issue from registers.  They compute nothing
// the fused operators need; the benchmark divides the Outer kernel's gather
// bytes and FMA count by these rates.
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"
#include "fusedops_tools.h"
#include "ptx.cuh"

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


// The same gather through the bulk-copy engine instead of per-lane loads: a warp keeps
// two slots of 16 rows in flight, every row landed in shared memory by one bulk copy
// that one of its lanes starts.  Nothing of the access pattern is shared with the
// per-lane probe or with the Outer kernels.  One CTA of 8 warps per SM.
constexpr int kBulkProbeRows = 16;

__global__ void __launch_bounds__(kThreads, 1)
probe_bulk_gather_kernel(const double *__restrict__ V, long long ldv, int cols, const int *__restrict__ idx,
                         long long n, double *__restrict__ out, unsigned int *status)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ unsigned long long s_bar[(kThreads / 32) * 2];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned rowbytes = (unsigned)cols * 8u;
    double *slot = reinterpret_cast<double *>(smem_raw) + (size_t)warp * 2 * kBulkProbeRows * cols;
    unsigned long long *bar = s_bar + warp * 2;
    if (lane == 0) {
        mbar_init(&bar[0], 1);
        mbar_init(&bar[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    const long long nwarps = (long long)gridDim.x * (kThreads / 32);
    const long long w0 = (long long)blockIdx.x * (kThreads / 32) + warp;
    const long long nbatch = (n + kBulkProbeRows - 1) / kBulkProbeRows;
    auto issue = [&](long long batch, int s) {
        const long long first = batch * kBulkProbeRows;
        const int cnt = n - first < kBulkProbeRows ? (int)(n - first) : kBulkProbeRows;
        if (lane == 0) mbar_expect_tx(&bar[s], (unsigned)cnt * rowbytes);
        __syncwarp();
        if (lane < cnt)
            bulk_g2s(slot + (size_t)(s * kBulkProbeRows + lane) * cols, V + (long long)__ldg(idx + first + lane) * ldv,
                     rowbytes, &bar[s]);
    };
    double acc = 0.0;
    bool gave_up = false;
    long long mine = 0;                          // batches of this warp issued so far
    for (long long b = w0; b < nbatch && mine < 2; b += nwarps, ++mine) issue(b, (int)(mine & 1));
    long long done = 0;
    for (long long b = w0; b < nbatch; b += nwarps, ++done) {
        const int s = (int)(done & 1);
        if (!__all_sync(0xffffffffu, mbar_wait(&bar[s], (unsigned)((done >> 1) & 1)))) {
            gave_up = true;
            break;
        }
        acc += slot[(size_t)(s * kBulkProbeRows) * cols + lane % cols];       // touch what landed
        __syncwarp();
        const long long next = b + 2 * nwarps;
        if (next < nbatch) issue(next, s);
    }
    if (gave_up && lane == 0) atomicExch(status, 1u);
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

extern "C" int fo_probe_bulk_gather(const fo_dense *V, const int *idx, long long n, double *out, void *stream)
{
    if (!V || !out || (n > 0 && !idx)) return FO_ERR_NULL;
    if (V->rows <= 0 || V->cols <= 0 || V->ld < V->cols || n < 0) return FO_ERR_SHAPE;
    if (!V->data) return FO_ERR_NULL;
    if ((V->cols & 1) || (V->ld & 1) || ((uintptr_t)V->data & 15u)) return FO_ERR_UNSUPPORTED;
    const size_t smem = (size_t)(kThreads / 32) * 2 * kBulkProbeRows * V->cols * sizeof(double);
    if (smem > 220u * 1024u) return FO_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return cuda_fail(cudaErrorNoDevice);
    cudaError_t e = cudaFuncSetAttribute(probe_bulk_gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e);
    // out's last double doubles as the give-up flag of the bounded waits: it is written by
    // the kernel's last thread anyway, so the flag lives one slot beyond what the kernel writes
    unsigned int *flag = reinterpret_cast<unsigned int *>(out + (size_t)sms * kThreads);
    e = cudaMemsetAsync(flag, 0, sizeof(double), (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e);
    probe_bulk_gather_kernel<<<sms, kThreads, smem, (cudaStream_t)stream>>>(V->data, V->ld, (int)V->cols, idx, n,
                                                                          out, flag);
    e = cudaGetLastError();
    return e == cudaSuccess ? FO_OK : cuda_fail(e);
}
