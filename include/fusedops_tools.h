/*
 * fusedops_tools.h - test and measurement hooks of the fused-operator library.
 *
 * Nothing here is needed to execute a fused operator; the product interface is
 * fusedops.h.  These calls let tests pin the library's internal choices (which
 * evaluation of a chain runs, what a run-time specialised kernel compiles to)
 * and let the benchmark measure the machine rates its rooflines divide by.
 */
#ifndef FUSEDOPS_TOOLS_H
#define FUSEDOPS_TOOLS_H

#include "fusedops.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Chains that match one of the library's compile-time specialisations (the
 * products and multi-aggregates of Fig. 1(a), (c)) normally run as straight-line
 * code; every other chain runs through the general interpreter.  Both give the
 * same bits.  on != 0 sends every Cell / MAgg chain through the interpreter
 * (process-wide; for tests and measurements).  Returns the previous setting. */
int fo_set_force_interpreter(int on);

/* Measurement knobs (process-wide).  The library picks kernel shapes and
 * schedules from the inputs; a knob overrides one such choice so that tests can
 * reach every compiled kernel and measurements can compare them.  Results stay
 * within the documented tolerance whatever the knobs say; only speed, and the
 * order of partial sums, change.  value == NULL clears a knob.  Returns FO_OK,
 * FO_ERR_UNSUPPORTED for an unknown name, FO_ERR_SHAPE for a value of 48 or
 * more characters.  Names:
 *   cell.ctas_per_sm  1..8   CTAs per SM of the streaming Cell / MAgg kernel
 *   row.narrow        0      dense rows of at most 32 columns through the warp-per-row kernel
 *   b1.mma            0 | 1  fused_row_b1: multiply-add kernel / tensor-core kernel
 *   b1.shape, b1.mma_shape   compiled shapes of those two kernels ("p,r,kl" / "w,kb")
 *   b1.narrow         0      fused_row_b1 without the thread-per-row kernel
 *   outer.kernel      "bulk" | "pipe" | "direct" | "dense"   schedule of fused_outer (per stored cell with
 *                     factor rows staged by bulk copies / by 16-byte copies / with plain gathers,
 *                     or tile by tile for densely stored inputs); by default the library chooses
 *                     from layout, rank and stored share
 *   cell.stamps       1      the streaming Cell / MAgg kernel records phase times (fo_cell_stamps) */
int fo_tune(const char *name, const char *value);

/* Phase times of the streaming Cell / MAgg kernel (full_agg), for measurements of small
 * inputs where launch, first-load latency and the last stage are a large share.  With
 * the knob cell.stamps set to 1 the kernel records, in nanoseconds of the GPU's global
 * timer, ns[0] the earliest CTA start, ns[1] the latest end of a CTA's scan, ns[2] the
 * latest publication of a partial sum, ns[3] the moment the result was written, in the
 * control words of the workspace.  This call synchronises `stream`, returns the four
 * stamps of the last such call and clears them. */
int fo_cell_stamps(void *ws, void *stream, unsigned long long *ns);

/* Generates and compiles (for sm_100a, without loading or launching: no GPU
 * needed) a run-time specialised kernel of a Cell chain; FO_OK, a chain error,
 * FO_ERR_UNSUPPORTED without NVRTC; the compiler log is copied to `log`.
 * `store` picks the skeleton: 0 flat stream (aggregating), 1 flat stream (no_agg),
 * 2 / 3 / 4 row-wise kernel (row_agg / no_agg / full_agg), 5 column kernel, 6 / 7 / 8
 * CSR main input with 2 / 8 / 32 lanes per row. */
int fo_jit_compile_check(const fo_chain *chain, int n_sides, int n_scalars, int store,
                         char *log, size_t log_bytes);
/* The same for a chain of the Outer template.  `kernel`: 0 / 1 the per-cell kernel with
 * plain gathers (full_agg at rank <= 112, left_mm at rank <= 256), 2 / 3 the kernel that
 * stages factor rows with 16-byte copies (full_agg, right_mm), 4 / 5 the tiled kernel (full_agg,
 * no_agg), 6 / 7 the kernel that stages factor rows with bulk copies (full_agg, no_agg). */
int fo_jit_compile_check_outer(const fo_chain *chain, int n_sides, int n_scalars, int kernel,
                               char *log, size_t log_bytes);
/* The same for a chain of the Row template.  `kernel`: 0 / 1 / 2 the dense kernel (1000-column
 * shape col_t_agg, 8192-column shape no_agg unstaged, 64-column shape row_agg), 3 the
 * thread-per-row kernel, 4 the CSR column-scatter kernel, 5 the CSR register kernel. */
int fo_jit_compile_check_row(const fo_chain *chain, int n_sides, int n_scalars, int kernel,
                             char *log, size_t log_bytes);

/* The k-th result of a chain written out as an expression over the inputs,
 * after validation and translation for a template (`use`: 0 Cell / MAgg,
 * 1 Row, 2 Outer), e.g. "mul(ne(r0,k0),mul(sub(r0,r1),sub(r0,r1)))" for the
 * weighted squared loss of Eq. 1.  rN: input register N (Cell: r0 = a, r1.. =
 * sides; Row: r0 = d, r1.. = sides; Outer: r0 = a, r1 = d); kN: entry N of the
 * constant table (scalars first, then immediates); sq(x) is written mul(x,x).
 * Chains with the same text do the same arithmetic in the same order; the
 * library picks its built-in straight-line evaluations by this text.  Host
 * only, no GPU needed.  Returns FO_OK, a chain error, or FO_ERR_SHAPE when the
 * text does not fit in `cap` bytes. */
int fo_chain_describe(const fo_chain *chain, int use, int n_sides,
                      const double *scalars, int n_scalars, int k,
                      char *text, size_t cap);

/* ---------------------------------------------------------------- probes
 * Machine-rate probes (no counterpart in the paper).  The Outer template
 * (Fig. 1(d)) gathers one row of V per stored cell and does `rank` multiply-adds
 * on it, so its roofline has two terms besides HBM bandwidth: the rate at which
 * whole rows can be gathered at random from a matrix resident in L2, and the
 * fp64 multiply-add issue rate.  These calls run a kernel that does only that;
 * the caller times them with events on `stream`.
 *   fo_probe_out_len()    doubles both probes write to `out` (device; one per
 *                         launched thread, so that the work cannot be dropped).
 *   fo_probe_l2_gather()  reads rows idx[0..n) (device int32, each in [0, V.rows))
 *                         of the dense matrix V, 8 lanes per row, 16-byte loads:
 *                         n * V.cols * 8 bytes move.  V.cols and V.ld even, V.data
 *                         16-byte aligned, else FO_ERR_UNSUPPORTED.
 *   fo_probe_bulk_gather() the same rows through the bulk-copy engine: 8 warps per SM, each
 *                         with two slots of 16 rows in flight in shared memory, one bulk
 *                         copy per row (a differently shaped measurement of the same
 *                         rate: nothing of its access pattern is shared with
 *                         fo_probe_l2_gather or the Outer kernels).  Same conditions on V;
 *                         the doubles of a row pair must fit 220 KB / 256 per row.  `out`
 *                         needs fo_probe_out_len() doubles here too (the kernel writes
 *                         fewer and keeps one word behind them as the flag of its bounded
 *                         waits: non-zero if one ran out).
 *   fo_probe_fp64_fma()   every one of the fo_probe_out_len() threads runs
 *                         8 * iters dependent-chain-of-8 multiply-adds from
 *                         registers: 16 * iters * fo_probe_out_len() flop.
 * Asynchronous; allocate nothing; errors as for the other calls. */
size_t fo_probe_out_len(void);
int fo_probe_l2_gather(const fo_dense *V, const int *idx, long long n, double *out, void *stream);
int fo_probe_bulk_gather(const fo_dense *V, const int *idx, long long n, double *out, void *stream);
int fo_probe_fp64_fma(long long iters, double *out, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* FUSEDOPS_TOOLS_H */
