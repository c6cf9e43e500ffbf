// The flat streaming kernel of the Cell / MAgg templates, written so that it can
// be compiled ahead of time (nvcc, with the interpreter or a built-in
// specialisation as EVAL) and at run time (NVRTC, with a generated EVAL): it
// depends on common.cuh only.
#pragma once

#include "common.cuh"

namespace fo {

constexpr int kIn = 1 + FO_MAX_SIDES;      // input slots: a, side0..side3

struct CellParams {
    const double *X;
    long long rows, cols, ldx;
    DevSides sides;
    WsHead *head;
    double *partials;
    double *out;
    int panels;           // cell_cols_kernel: number of row panels
    int cx;               // cell_cols_kernel: column pairs per CTA
    unsigned long long *stamps;   // flat kernel: where to record phase times (measurement), or NULL
};

// Time stamps of the flat kernel's phases, in nanoseconds of the GPU's global timer,
// kept in the workspace head when a measurement asks for them: [0] the complement of
// the earliest CTA start, [1] the latest end of a CTA's scan, [2] the latest
// publication of a partial sum, [3] the final result written.
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

constexpr int kV = 4;     // cells per thread per chain evaluation

enum { kAggNone = 0, kAggRow = 1, kAggFull = 3 };

// Adds the chain's results for four cells to the running sums (invalid cells count 0).
template <int NOUT>
__device__ __forceinline__ void add_outputs(const double (&o)[NOUT][kV], const bool (&valid)[kV],
                                            double (&acc)[NOUT])
{
#pragma unroll
    for (int k = 0; k < NOUT; ++k) {
        double s = 0.0;
#pragma unroll
        for (int i = 0; i < kV; ++i) s += valid[i] ? o[k][i] : 0.0;
        acc[k] += s;
    }
}

__device__ __forceinline__ void put4(double (&dst)[kV], double2 m0, double2 m1)
{
    dst[0] = m0.x; dst[1] = m0.y; dst[2] = m1.x; dst[3] = m1.y;
}

// ------------------------------------------------------------------ flat
template <class EVAL, int NOUT, bool STORE>
__device__ __forceinline__ void cell_flat_body(const DevChain &ch, const CellParams &p)
{
    __shared__ double s_red[NOUT * 32];
    __shared__ unsigned int s_flag;
    double acc[NOUT];
#pragma unroll
    for (int k = 0; k < NOUT; ++k) acc[k] = 0.0;

    const long long ncells = p.rows * p.cols;
    const long long ntiles = ncells >> 10;          // full tiles of 1024 cells
    const int t = threadIdx.x;
    if (p.stamps && t == 0) atomicMax(&p.stamps[0], ~global_ns());

    // two tiles a trip while they last: twice the loads in flight per thread, which is what
    // a small input (a few tiles per CTA in all) has to hide the memory latency with
    // (straight-line chains only: the interpreter's register file does not fit twice)
    long long tile = blockIdx.x;
    for (; !EVAL::kInterp && tile + gridDim.x < ntiles; tile += 2ll * gridDim.x) {
        const long long a0 = (tile << 10) + 2 * t, a1 = a0 + 512;
        const long long b0 = ((tile + gridDim.x) << 10) + 2 * t, b1 = b0 + 512;
        double in[kIn][kV], in2[kIn][kV];
        put4(in[0], ld_stream2(p.X + a0), ld_stream2(p.X + a1));
        put4(in2[0], ld_stream2(p.X + b0), ld_stream2(p.X + b1));
#pragma unroll
        for (int k = 0; k < FO_MAX_SIDES; ++k) {
            if (EVAL::uses_side(ch, k)) {
                const double *sp = p.sides.s[k].data;
                put4(in[1 + k], ld_stream2(sp + a0), ld_stream2(sp + a1));
                put4(in2[1 + k], ld_stream2(sp + b0), ld_stream2(sp + b1));
            }
        }
        double o[NOUT][kV], o2[NOUT][kV];
        EVAL::template run<kV, NOUT>(ch, in, o);
        EVAL::template run<kV, NOUT>(ch, in2, o2);
        if (STORE) {
            *reinterpret_cast<double2 *>(p.out + a0) = make_double2(o[0][0], o[0][1]);
            *reinterpret_cast<double2 *>(p.out + a1) = make_double2(o[0][2], o[0][3]);
            *reinterpret_cast<double2 *>(p.out + b0) = make_double2(o2[0][0], o2[0][1]);
            *reinterpret_cast<double2 *>(p.out + b1) = make_double2(o2[0][2], o2[0][3]);
        } else {
            const bool valid[kV] = {true, true, true, true};
            add_outputs<NOUT>(o, valid, acc);
            add_outputs<NOUT>(o2, valid, acc);
        }
    }
    for (; tile < ntiles; tile += gridDim.x) {
        const long long o0 = (tile << 10) + 2 * t, o1 = o0 + 512;
        double in[kIn][kV];
        put4(in[0], ld_stream2(p.X + o0), ld_stream2(p.X + o1));
#pragma unroll
        for (int k = 0; k < FO_MAX_SIDES; ++k) {
            if (EVAL::uses_side(ch, k)) {
                const double *sp = p.sides.s[k].data;
                put4(in[1 + k], ld_stream2(sp + o0), ld_stream2(sp + o1));
            }
        }
        double o[NOUT][kV];
        EVAL::template run<kV, NOUT>(ch, in, o);
        if (STORE) {
            *reinterpret_cast<double2 *>(p.out + o0) = make_double2(o[0][0], o[0][1]);
            *reinterpret_cast<double2 *>(p.out + o1) = make_double2(o[0][2], o[0][3]);
        } else {
            const bool valid[kV] = {true, true, true, true};
            add_outputs<NOUT>(o, valid, acc);
        }
    }

    // ragged tail (< 1024 cells): one CTA, scalar loads
    const long long tail0 = ntiles << 10;
    if (tail0 < ncells && blockIdx.x == (unsigned)(ntiles % gridDim.x)) {
        double in[kIn][kV];
        bool valid[kV];
        long long idx[kV];
#pragma unroll
        for (int i = 0; i < kV; ++i) {
            idx[i] = tail0 + t + i * kThreads;
            valid[i] = idx[i] < ncells;
            in[0][i] = valid[i] ? ld_stream1(p.X + idx[i]) : 0.0;
        }
#pragma unroll
        for (int k = 0; k < FO_MAX_SIDES; ++k) {
            if (EVAL::uses_side(ch, k)) {
#pragma unroll
                for (int i = 0; i < kV; ++i)
                    in[1 + k][i] = valid[i] ? ld_stream1(p.sides.s[k].data + idx[i]) : 0.0;
            }
        }
        double o[NOUT][kV];
        EVAL::template run<kV, NOUT>(ch, in, o);
        if (STORE) {
#pragma unroll
            for (int i = 0; i < kV; ++i)
                if (valid[i]) p.out[idx[i]] = o[0][i];
        } else {
            add_outputs<NOUT>(o, valid, acc);
        }
    }

    if (!STORE) {
        if (p.stamps && t == 0) atomicMax(&p.stamps[1], global_ns());
        block_sum<NOUT>(acc, s_red);
        if (t == 0) {
#pragma unroll
            for (int k = 0; k < NOUT; ++k)
                if (k < ch.n_out) p.partials[(size_t)blockIdx.x * ch.n_out + k] = acc[k];
        }
        const bool last = publish_and_is_last(p.head, &s_flag);
        if (p.stamps && t == 0) atomicMax(&p.stamps[2], global_ns());
        if (last) {
            final_sum_small(p.partials, gridDim.x, ch.n_out, p.out, s_red);
            if (p.stamps && t == 0) p.stamps[3] = global_ns();
        }
    }
}


template <class EVAL, int NOUT, bool STORE>
__global__ void __launch_bounds__(kThreads)
cell_flat_kernel(const __grid_constant__ DevChain ch, const __grid_constant__ CellParams p)
{
    cell_flat_body<EVAL, NOUT, STORE>(ch, p);
}

// EVAL for a chain written out as straight-line code.  Fn provides
//   kSideMask  bit k set if it reads side k,
//   kOut       number of results,
//   eval(in, consts, out)  with in[0] = a, in[1 + k] = side k.
template <class Fn>
struct EvalFn {
    static constexpr bool kInterp = false;
    static constexpr int kOutMax = Fn::kOut;
    __device__ __forceinline__ static bool uses_side(const DevChain &, int k) { return (Fn::kSideMask >> k) & 1u; }
    template <int V, int NOUT>
    __device__ __forceinline__ static void run(const DevChain &ch, const double (&in)[kIn][V],
                                               double (&o)[NOUT][V])
    {
        static_assert(NOUT >= Fn::kOut, "accumulator count");
#pragma unroll
        for (int i = 0; i < V; ++i) {
            double x[kIn], y[Fn::kOut];
#pragma unroll
            for (int k = 0; k < kIn; ++k) x[k] = (k == 0 || ((Fn::kSideMask >> (k - 1)) & 1u)) ? in[k][i] : 0.0;
            Fn::eval(x, ch.consts, y);
#pragma unroll
            for (int k = 0; k < NOUT; ++k) o[k][i] = (k < Fn::kOut) ? y[k < Fn::kOut ? k : 0] : 0.0;
        }
    }
};

}  // namespace fo
