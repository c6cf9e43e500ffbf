// Two ways to evaluate an operator chain inside a kernel, behind one interface:
//
//   EvalInterp<NR>  the general register-machine interpreter of chain.cuh;
//   EvalSpec<ID>    the same arithmetic, in the same order, written out at
//                   compile time for a few chains that the paper's fusion
//                   examples keep producing (Fig. 1; Section 5.2).
//
// The host recognises a specialised chain by comparing the translated program
// with the specialisation's reference program (spec_host.cu); any other chain
// runs through the interpreter.  Both give bit-identical results.
#pragma once

#include "cell_flat.cuh"
#include "chain.cuh"

namespace fo {

enum SpecId {
    kSpecNone = 0,
    kSpecMul2,      // a * side0                         sum(X * Y)
    kSpecMul3,      // (a * side0) * side1               sum(X * Y * Z), Fig. 1(a)
    kSpecSq,        // a * a                             sum(X^2)
    kSpecMagg2,     // (a * side0, a * side1)            Section 5.2 multi-aggregate
    kSpecMagg3,     // (a * side0, a * side1, a * a)     Fig. 1(c)-style
    kSpecScaledAdd, // side0 + (a * c) * side1           the cell-wise operator of Section 2.2 (I + 1e-6 * U * r)
    kSpecCount
};

// Host: specialisation matching a translated Cell / MAgg chain, or kSpecNone.
int match_cell_spec(const DevChain &ch);
// Host: for kSpecScaledAdd, the entry of ch.consts that holds c (the kernels read it from consts[0]).
int scaled_add_const(const DevChain &ch);


template <int NR>
struct EvalInterp {
    static constexpr bool kInterp = true;
    static constexpr int kOutMax = FO_MAX_OUT;
    __device__ __forceinline__ static bool uses_side(const DevChain &ch, int k)
    {
        return 1 + k < NR && ((ch.side_used >> k) & 1u);
    }
    template <int V, int NOUT>
    __device__ __forceinline__ static void run(const DevChain &ch, const double (&in)[kIn][V],
                                               double (&o)[NOUT][V])
    {
        RegFile<NR, V> f;
#pragma unroll
        for (int k = 0; k < kIn; ++k) {
            if (k < NR) {
#pragma unroll
                for (int i = 0; i < V; ++i) f.r[k < NR ? k : 0][i] = in[k][i];
            }
        }
        run_chain<NR, V>(ch, f);
#pragma unroll
        for (int k = 0; k < NOUT; ++k) {
            if (k < ch.n_out) {
                operand<NR, V>(ch, f, ch.out[k], o[k]);
            } else {
#pragma unroll
                for (int i = 0; i < V; ++i) o[k][i] = 0.0;
            }
        }
    }
};

template <int ID>
struct SpecFn;

template <>
struct SpecFn<kSpecMul2> {
    static constexpr unsigned kSideMask = 1u;
    static constexpr int kOut = 1;
    __device__ __forceinline__ static void eval(const double *in, const double *, double *o) { o[0] = in[0] * in[1]; }
};
template <>
struct SpecFn<kSpecMul3> {
    static constexpr unsigned kSideMask = 3u;
    static constexpr int kOut = 1;
    __device__ __forceinline__ static void eval(const double *in, const double *, double *o)
    {
        o[0] = (in[0] * in[1]) * in[2];
    }
};
template <>
struct SpecFn<kSpecSq> {
    static constexpr unsigned kSideMask = 0u;
    static constexpr int kOut = 1;
    __device__ __forceinline__ static void eval(const double *in, const double *, double *o) { o[0] = in[0] * in[0]; }
};
template <>
struct SpecFn<kSpecScaledAdd> {
    static constexpr unsigned kSideMask = 3u;
    static constexpr int kOut = 1;
    __device__ __forceinline__ static void eval(const double *in, const double *c, double *o)
    {
        o[0] = in[1] + (in[0] * c[0]) * in[2];
    }
};
template <>
struct SpecFn<kSpecMagg2> {
    static constexpr unsigned kSideMask = 3u;
    static constexpr int kOut = 2;
    __device__ __forceinline__ static void eval(const double *in, const double *, double *o)
    {
        o[0] = in[0] * in[1];
        o[1] = in[0] * in[2];
    }
};
template <>
struct SpecFn<kSpecMagg3> {
    static constexpr unsigned kSideMask = 3u;
    static constexpr int kOut = 3;
    __device__ __forceinline__ static void eval(const double *in, const double *, double *o)
    {
        o[0] = in[0] * in[1];
        o[1] = in[0] * in[2];
        o[2] = in[0] * in[0];
    }
};

template <int ID>
using EvalSpec = EvalFn<SpecFn<ID>>;

}  // namespace fo
