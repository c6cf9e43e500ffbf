// Device-side evaluation of a scalar operator chain on V values per thread.
//
// The chain is warp-uniform data in kernel-parameter (constant) space; each
// thread holds a register file R[NR][V] of doubles.  Register numbers are only
// known at run time, so reads and writes of R go through switch statements
// whose cases name the registers statically: R stays in hardware registers
// and the branches are uniform across the warp.  Working on V cells per
// dispatch spreads the decode cost over V results.
#pragma once

#include "common.cuh"

namespace fo {

// Long-latency library functions stay out of line: inlined V times each they
// would dominate the register budget of kernels whose usual chains never call them.
static __device__ __noinline__ double slow_exp(double a) { return exp(a); }
static __device__ __noinline__ double slow_log(double a) { return log(a); }
static __device__ __noinline__ double slow_pow(double a, double b) { return pow(a, b); }
static __device__ __noinline__ double slow_div(double a, double b) { return a / b; }
static __device__ __noinline__ double slow_sqrt(double a) { return sqrt(a); }

template <int NR, int V>
struct RegFile {
    double r[NR][V];
};

template <int NR, int V>
__device__ __forceinline__ void reg_read(const RegFile<NR, V> &f, int idx, double (&dst)[V])
{
#define FO_RD(k)                                            \
    case k:                                                 \
        if (k < NR) {                                       \
            _Pragma("unroll") for (int i = 0; i < V; ++i) dst[i] = f.r[k < NR ? k : 0][i]; \
        }                                                   \
        break;
    switch (idx) {
        FO_RD(0) FO_RD(1) FO_RD(2) FO_RD(3) FO_RD(4) FO_RD(5) FO_RD(6)
        FO_RD(7) FO_RD(8) FO_RD(9) FO_RD(10) FO_RD(11) FO_RD(12) FO_RD(13)
        default: break;
    }
#undef FO_RD
}

template <int NR, int V>
__device__ __forceinline__ void reg_write(RegFile<NR, V> &f, int idx, const double (&src)[V])
{
#define FO_WR(k)                                            \
    case k:                                                 \
        if (k < NR) {                                       \
            _Pragma("unroll") for (int i = 0; i < V; ++i) f.r[k < NR ? k : 0][i] = src[i]; \
        }                                                   \
        break;
    switch (idx) {
        FO_WR(0) FO_WR(1) FO_WR(2) FO_WR(3) FO_WR(4) FO_WR(5) FO_WR(6)
        FO_WR(7) FO_WR(8) FO_WR(9) FO_WR(10) FO_WR(11) FO_WR(12) FO_WR(13)
        default: break;
    }
#undef FO_WR
}

// Operand byte: register index, or 0x80 | constant index.
template <int NR, int V>
__device__ __forceinline__ void operand(const DevChain &ch, const RegFile<NR, V> &f, int opnd,
                                        double (&dst)[V])
{
    if (opnd & 0x80) {
        const double c = ch.consts[opnd & 0x7f];
#pragma unroll
        for (int i = 0; i < V; ++i) dst[i] = c;
    } else {
        reg_read<NR, V>(f, opnd, dst);
    }
}

// Runs every step of the chain on the register file.
template <int NR, int V>
__device__ __forceinline__ void run_chain(const DevChain &ch, RegFile<NR, V> &f)
{
    const int n = ch.n_ops;
    for (int s = 0; s < n; ++s) {
        const DevOp op = ch.ops[s];
        double a[V], b[V], r[V];
        operand<NR, V>(ch, f, op.a, a);
        if (op.opcode >= FO_OP_ADD) operand<NR, V>(ch, f, op.b, b);
#define FO_EACH(expr)                                       \
    _Pragma("unroll") for (int i = 0; i < V; ++i) { r[i] = (expr); }
        switch (op.opcode) {
            case FO_OP_MOV: FO_EACH(a[i]) break;
            case FO_OP_NEG: FO_EACH(-a[i]) break;
            case FO_OP_ABS: FO_EACH(fabs(a[i])) break;
            case FO_OP_SQRT: FO_EACH(slow_sqrt(a[i])) break;
            case FO_OP_EXP: FO_EACH(slow_exp(a[i])) break;
            case FO_OP_LOG: FO_EACH(slow_log(a[i])) break;
            case FO_OP_SQ: FO_EACH(a[i] * a[i]) break;
            case FO_OP_ADD: FO_EACH(a[i] + b[i]) break;
            case FO_OP_SUB: FO_EACH(a[i] - b[i]) break;
            case FO_OP_MUL: FO_EACH(a[i] * b[i]) break;
            case FO_OP_DIV: FO_EACH(slow_div(a[i], b[i])) break;
            case FO_OP_MIN: FO_EACH(fmin(a[i], b[i])) break;
            case FO_OP_MAX: FO_EACH(fmax(a[i], b[i])) break;
            case FO_OP_POW: FO_EACH(slow_pow(a[i], b[i])) break;
            case FO_OP_EQ: FO_EACH(a[i] == b[i] ? 1.0 : 0.0) break;
            case FO_OP_NE: FO_EACH(a[i] != b[i] ? 1.0 : 0.0) break;
            case FO_OP_LT: FO_EACH(a[i] < b[i] ? 1.0 : 0.0) break;
            case FO_OP_LE: FO_EACH(a[i] <= b[i] ? 1.0 : 0.0) break;
            case FO_OP_GT: FO_EACH(a[i] > b[i] ? 1.0 : 0.0) break;
            case FO_OP_GE: FO_EACH(a[i] >= b[i] ? 1.0 : 0.0) break;
            case FO_OP_SEL: {
                double c[V];
                operand<NR, V>(ch, f, op.c, c);
                FO_EACH(a[i] != 0.0 ? b[i] : c[i])
                break;
            }
            case FO_OP_FMA: {
                double c[V];
                operand<NR, V>(ch, f, op.c, c);
                FO_EACH(fma(a[i], b[i], c[i]))
                break;
            }
            default: FO_EACH(0.0) break;
        }
#undef FO_EACH
        reg_write<NR, V>(f, op.dst, r);
    }
}

// One scalar evaluation of the chain by a whole warp.  The register file is
// spread over the lanes: lane k holds register k (`mine`), operands are fetched
// with a shuffle from the lane named by the operand byte, and the lane named by
// `dst` keeps the result.  No register is indexed at run time and no lane
// diverges; the cost is a few shuffles per step.  All 32 lanes must call it with
// the same chain; the result is returned in every lane.
__device__ __forceinline__ double warp_operand(const DevChain &ch, double mine, int opnd)
{
    if (opnd & 0x80) return ch.consts[opnd & 0x7f];
    return __shfl_sync(0xffffffffu, mine, opnd & 31);
}

__device__ __forceinline__ double warp_chain(const DevChain &ch, double mine, int lane)
{
    const int n = ch.n_ops;
    for (int s = 0; s < n; ++s) {
        const DevOp op = ch.ops[s];
        const double a = warp_operand(ch, mine, op.a);
        double b = 0.0, c = 0.0, r;
        if (op.opcode >= FO_OP_ADD) b = warp_operand(ch, mine, op.b);
        if (op.opcode >= FO_OP_SEL) c = warp_operand(ch, mine, op.c);
        switch (op.opcode) {
            case FO_OP_MOV: r = a; break;
            case FO_OP_NEG: r = -a; break;
            case FO_OP_ABS: r = fabs(a); break;
            case FO_OP_SQRT: r = slow_sqrt(a); break;
            case FO_OP_EXP: r = slow_exp(a); break;
            case FO_OP_LOG: r = slow_log(a); break;
            case FO_OP_SQ: r = a * a; break;
            case FO_OP_ADD: r = a + b; break;
            case FO_OP_SUB: r = a - b; break;
            case FO_OP_MUL: r = a * b; break;
            case FO_OP_DIV: r = slow_div(a, b); break;
            case FO_OP_MIN: r = fmin(a, b); break;
            case FO_OP_MAX: r = fmax(a, b); break;
            case FO_OP_POW: r = slow_pow(a, b); break;
            case FO_OP_EQ: r = a == b ? 1.0 : 0.0; break;
            case FO_OP_NE: r = a != b ? 1.0 : 0.0; break;
            case FO_OP_LT: r = a < b ? 1.0 : 0.0; break;
            case FO_OP_LE: r = a <= b ? 1.0 : 0.0; break;
            case FO_OP_GT: r = a > b ? 1.0 : 0.0; break;
            case FO_OP_GE: r = a >= b ? 1.0 : 0.0; break;
            case FO_OP_SEL: r = a != 0.0 ? b : c; break;
            case FO_OP_FMA: r = fma(a, b, c); break;
            default: r = 0.0; break;
        }
        if (lane == op.dst) mine = r;
    }
    return warp_operand(ch, mine, ch.out[0]);
}

}  // namespace fo
