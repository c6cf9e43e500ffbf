/*
 * fusedops.h - C ABI of the fused-operator library (CUDA, sm_100a).
 *
 * The library executes the four fused-operator template types of
 * "On Optimizing Operator Fusion Plans for Large-Scale Machine Learning in
 * SystemML" (Section 2.2, Table 1: Row, Cell, MAgg, Outer) on one GPU, over
 * dense row-major and CSR float64 matrices.  A fused operator is described by
 *   - a template call (fused_cell / fused_magg / fused_row / fused_outer),
 *   - the template variant (an aggregation type of Table 1), and
 *   - an explicit scalar operator chain (fo_chain): the straight-line program
 *     the paper's generated `genexec` method holds (Section 2.2, listings).
 * The data access, the parallel schedule and the aggregation live in the
 * library's kernels, as they live in the paper's hand-coded template skeletons
 * (Section 2.2, "Runtime Integration").
 *
 * Conventions for every call
 *   - Matrix data, index arrays, `out` and `ws` are DEVICE pointers owned by the
 *     caller.  fo_chain, fo_op, fo_side, fo_mat structs and the `scalars` array
 *     are HOST memory; they are copied at launch and may be freed on return.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream).  No call allocates, frees or synchronises, with one
 *     documented exception: the first use of a chain that the library
 *     specialises at run time (see fo_set_jit) compiles and loads a kernel inside
 *     the fused_* call unless the chain was prepared (fo_jit_prepare,
 *     fo_jit_prepare_call) or the mode forbids it.  fused_cell_static never does.
 *   - Inputs are never written.  `out` is fully overwritten.
 *   - `ws` is scratch of at least fused_*_workspace_bytes() bytes, 256-byte
 *     aligned, prepared once with fo_workspace_init(); every call leaves it
 *     ready for the next.  Two calls that overlap on the GPU must not share it.
 *   - Return value: FO_OK or a negative fo_status.  Nothing throws, aborts or
 *     traps.  On an error return nothing was launched.
 *   - All values are IEEE float64.  CSR: rowptr has rows+1 int32 offsets with
 *     rowptr[0] == 0 and rowptr[rows] == nnz, colidx int32 strictly ascending
 *     inside a row, explicit zeros allowed.  Dense: row-major, element (i, j) at
 *     data[i * ld + j], ld >= cols.
 *   - Sums are deterministic: for given shapes the order of every floating-point
 *     addition is fixed, so repeated calls return identical bits (exception:
 *     the variants that scatter through atomics: FO_ROW_COL_T_AGG / FO_ROW_COL_AGG and
 *     FO_ROW_COL_AGG_B1_T over a CSR main input, FO_CELL_COL_AGG over a CSR main input,
 *     FO_OUTER_LEFT_MM; each is documented at its call).
 */
#ifndef FUSEDOPS_H
#define FUSEDOPS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ------------------------------------------------------------------ status */
typedef enum fo_status {
    FO_OK = 0,
    FO_ERR_NULL = -1,           /* a required pointer is NULL */
    FO_ERR_SHAPE = -2,          /* dimensions of inputs do not fit together */
    FO_ERR_CHAIN = -3,          /* bad opcode / operand, use before definition, too long */
    FO_ERR_UNSUPPORTED = -4,    /* variant or size outside what the kernels cover */
    FO_ERR_WORKSPACE = -5,      /* ws NULL, misaligned or too small */
    FO_ERR_CUDA = -6,           /* the CUDA runtime refused the launch */
    FO_ERR_DEVICE_TIMEOUT = -7, /* a bounded device-side wait ran out (see fo_query_device_status) */
    FO_ERR_STATIC_LIMIT = -8    /* fused_cell_static: the call needs more than the built-in scratch */
} fo_status;

/* ---------------------------------------------------------------- matrices */
typedef struct fo_dense {
    int64_t rows, cols, ld;
    const double *data;         /* device */
} fo_dense;

typedef struct fo_csr {
    int64_t rows, cols, nnz;    /* nnz < 2^31 */
    const int32_t *rowptr;      /* device, rows + 1 */
    const int32_t *colidx;      /* device, nnz */
    const double *vals;         /* device, nnz */
} fo_csr;

enum { FO_DENSE = 0, FO_CSR = 1 };
typedef struct fo_mat {
    int32_t kind;               /* FO_DENSE or FO_CSR; the other member is ignored */
    int32_t reserved;
    fo_dense dense;
    fo_csr csr;
} fo_mat;

/*
 * Side input (the paper's SideInput b[k], Section 2.2 cell-wise listing).
 *   FO_AT_CELL: same shape as the main input, value read at (rix, cix);
 *   FO_AT_ROW : column vector (rows x 1, element i at data[i * ld]), read at (rix);
 *   FO_AT_COL : row vector (1 x cols), read at (cix).
 * Side inputs are dense, with one exception (the sparse side inputs of Table 1's
 * Y+-, read through getValue() in Section 5.2 "Cell Operations"): if `sparse` is
 * not NULL the side is that CSR matrix - same shape as the main input,
 * FO_AT_CELL, `m` ignored - and reads 0.0 wherever it stores no cell.  Sparse
 * sides are accepted by fused_cell and fused_magg over a CSR main input (a
 * sparse driver with sparse sides); every other call returns
 * FO_ERR_UNSUPPORTED for them.
 */
enum { FO_AT_CELL = 0, FO_AT_ROW = 1, FO_AT_COL = 2 };
typedef struct fo_side {
    fo_dense m;
    int32_t access;
    int32_t reserved;
    const fo_csr *sparse;       /* host pointer or NULL; see below */
} fo_side;

/* ------------------------------------------------------------ operator chain */
#define FO_MAX_OPS      32      /* steps per chain */
#define FO_MAX_TMPS      8      /* temporaries t0..t7 */
#define FO_MAX_SIDES     4
#define FO_MAX_SCALARS   8
#define FO_MAX_OUT       8      /* results of one chain (MAgg: number of aggregates) */

/* Operand bytes. */
#define FO_TMP(k)     ((uint8_t)(0x00 | (k)))   /* temporary k, must have been written */
#define FO_SIDE(k)    ((uint8_t)(0x40 | (k)))   /* k-th side input at this cell / row */
#define FO_SCALAR(k)  ((uint8_t)(0x80 | (k)))   /* scalars[k] */
#define FO_MAIN       ((uint8_t)0xC0)           /* a: main-input value (Cell, MAgg, Outer) */
#define FO_DOT        ((uint8_t)0xC1)           /* d: Row: X_i . v;  Outer: U_i . V_j */
#define FO_IMM        ((uint8_t)0xC2)           /* this step's `imm` constant */

typedef enum fo_opcode {
    FO_OP_MOV = 0,   /* dst = a */
    FO_OP_NEG, FO_OP_ABS, FO_OP_SQRT, FO_OP_EXP, FO_OP_LOG,
    FO_OP_SQ,        /* dst = a * a */
    FO_OP_ADD, FO_OP_SUB, FO_OP_MUL, FO_OP_DIV, FO_OP_MIN, FO_OP_MAX, FO_OP_POW,
    FO_OP_EQ, FO_OP_NE, FO_OP_LT, FO_OP_LE, FO_OP_GT, FO_OP_GE,   /* 1.0 or 0.0 */
    FO_OP_SEL,       /* dst = (a != 0) ? b : c */
    FO_OP_FMA,       /* dst = a * b + c (one rounding) */
    FO_OP_COUNT_
} fo_opcode;

typedef struct fo_op {
    uint8_t opcode;             /* fo_opcode */
    uint8_t dst;                /* temporary index 0..FO_MAX_TMPS-1 */
    uint8_t a, b, c;            /* operand bytes; unused ones are ignored */
    uint8_t reserved[3];
    double imm;                 /* value of FO_IMM operands of this step */
} fo_op;

typedef struct fo_chain {
    int32_t n_ops;              /* 0..FO_MAX_OPS */
    int32_t n_out;              /* 1..FO_MAX_OUT (1 except for fused_magg) */
    const fo_op *ops;           /* host */
    uint8_t out[FO_MAX_OUT];    /* operand bytes of the results */
} fo_chain;

/* ------------------------------------------------------ template variants */
/* Cell (Table 1: no_agg, row_agg, col_agg, full_agg) */
enum { FO_CELL_NO_AGG = 0, FO_CELL_ROW_AGG = 1, FO_CELL_COL_AGG = 2, FO_CELL_FULL_AGG = 3 };
/* Row (Table 1).  fused_row implements all of no_agg, row_agg, col_agg, full_agg
 * and col_t_agg (col_agg, 1 x n, and col_t_agg, n x 1, are the same n values in
 * memory).  The *_B1 variants (row intermediates that are k-vectors,
 * from a product with a side matrix) belong to fused_row_b1. */
enum { FO_ROW_NO_AGG = 0, FO_ROW_ROW_AGG = 1, FO_ROW_COL_AGG = 2, FO_ROW_FULL_AGG = 3,
       FO_ROW_COL_T_AGG = 4, FO_ROW_NO_AGG_B1 = 5, FO_ROW_COL_AGG_B1_T = 6 };
/* Outer (Table 1: left_mm, right_mm, no_agg, full_agg) */
enum { FO_OUTER_LEFT_MM = 0, FO_OUTER_RIGHT_MM = 1, FO_OUTER_NO_AGG = 2, FO_OUTER_FULL_AGG = 3 };

/* -------------------------------------------------------------- workspace */
/* Bytes of scratch a call with these arguments needs (0 on invalid arguments).
 * Pure host arithmetic: usable without a GPU. */
size_t fused_cell_workspace_bytes(const fo_mat *X, int agg);
size_t fused_magg_workspace_bytes(const fo_mat *X, int n_out);
size_t fused_row_workspace_bytes(const fo_mat *X, int agg);
size_t fused_outer_workspace_bytes(const fo_csr *X, int rank, int agg);
size_t fused_row_b1_workspace_bytes(const fo_mat *X, int k, int agg);

/* Clears the control words at the head of a workspace (asynchronous on `stream`).
 * Needed once after allocation, and again after a call returned
 * FO_ERR_DEVICE_TIMEOUT through fo_query_device_status. */
int fo_workspace_init(void *ws, size_t ws_bytes, void *stream);

/* Synchronises `stream`, then reads the workspace's device-side status word:
 * *status = FO_OK or FO_ERR_DEVICE_TIMEOUT.  Returns FO_OK unless the query
 * itself failed. */
int fo_query_device_status(const void *ws, void *stream, int *status);

const char *fo_status_string(int status);

/* Last CUDA runtime error code seen by a call that returned FO_ERR_CUDA
 * (thread-local), 0 if none. */
int fo_last_cuda_error(void);

/* Run-time specialisation (the paper's template expansion to source, compilation
 * and plan cache, Section 2.1 "Codegen Architecture").  A chain that has no
 * built-in straight-line form - in any call: fused_cell / fused_magg over dense or
 * CSR inputs, fused_row, fused_outer - is written out as straight-line code inside
 * the kernel the call would otherwise interpret it in, compiled for the current
 * GPU with NVRTC (a few hundred ms to a second) and cached under kernel and
 * translated program, per CUDA context, for the life of the process; calls with the
 * same chain - whatever the values of its scalars and immediates - reuse it.  (The
 * pre / post chains of fused_row_b1 are interpreted.)
 * Results are bit-identical to the interpreter's.  NVRTC and the driver library
 * are loaded on demand; if they are missing or a compilation fails the
 * interpreter runs instead, so results never depend on them.
 *   fo_set_jit(mode)  FO_JIT_OFF: never specialise.  FO_JIT_FIRST_USE (default):
 *                     the fused_* calls compile a chain the first time they
 *                     see it - that one call compiles, loads a module (which
 *                     allocates) and may synchronise; do it outside stream capture.
 *                     FO_JIT_PREPARED: the calls only look kernels up; a chain that
 *                     was not prepared runs through the interpreter, and no call
 *                     ever compiles, loads or allocates.  Returns the old mode.
 *   fo_jit_prepare()  compiles, loads and caches the flat-stream kernel of a chain now,
 *                     for the current device (n_sides / n_scalars as in the later
 *                     calls; store != 0: the no_agg form, else the aggregating form).
 *                     FO_OK (also when it was cached already), a chain error,
 *                     FO_ERR_UNSUPPORTED without NVRTC / the driver library,
 *                     FO_ERR_CHAIN if the compilation or the load failed.
 *   fo_jit_prepare_call()  the same for exactly the kernel a later fused_cell (magg = 0)
 *                     or fused_magg (magg != 0) call with these arguments would run:
 *                     X and the sides are looked at for shapes, leading dimensions
 *                     and alignment only (no device access).  FO_OK also when the
 *                     chain has a built-in form; FO_ERR_UNSUPPORTED for a CSR X (its
 *                     kernel is compiled at first use, or never in FO_JIT_PREPARED).
 *   fo_jit_stats()    kernels compiled, specialised launches, failed compilations so
 *                     far; returns 1 if NVRTC and the driver library are usable. */
enum { FO_JIT_OFF = 0, FO_JIT_FIRST_USE = 1, FO_JIT_PREPARED = 2 };
int fo_set_jit(int mode);
int fo_jit_prepare(const fo_chain *chain, int n_sides, int n_scalars, int store);
int fo_jit_prepare_call(const fo_chain *chain, const fo_mat *X, const fo_side *sides, int n_sides,
                        int n_scalars, int agg, int magg);
int fo_jit_stats(int *compiled, int *launches, int *failures);

/* ------------------------------------------------------------------ Cell
 * Table 1, Cell template; Section 2.2 cell-wise listing.
 * For every cell (i, j) of a dense main input X (for a CSR main input: every
 * STORED cell - the sparse-safe binding) the chain computes one value from
 * a = X_ij, side values and scalars; then
 *   FO_CELL_FULL_AGG: out[0]        = sum over all cells
 *   FO_CELL_ROW_AGG : out[i]        = sum over j          (rows doubles)
 *   FO_CELL_COL_AGG : out[j]        = sum over i          (cols doubles)
 *   FO_CELL_NO_AGG  : dense X: out[i * cols + j] = value  (rows * cols doubles,
 *                     packed); CSR X: out[p] = value of stored cell p (nnz
 *                     doubles, X's pattern).
 * A CSR main input with a chain that is not zero-preserving gives the result
 * of the sparse-safe binding, not of the dense one; the caller decides that
 * (in the paper the compiler marks templates sparse-safe, Section 2.2).
 * Determinism: FO_CELL_COL_AGG over a CSR X adds into `out` with global atomics on
 * a zeroed result, so the order of its additions is not fixed; everything else
 * is bit-reproducible.
 * out_nnz (device, one int64, or NULL): with FO_CELL_NO_AGG the number of written
 * values that are not zero - what a sparse result would store (-0.0 counts as
 * zero, NaN as non-zero).  It costs one more pass over `out`.  Not NULL with
 * another variant: FO_ERR_UNSUPPORTED.  A CSR result keeps X's index arrays
 * (values on X's pattern), so rowptr / colidx of the result are X's own.
 * Errors: FO_ERR_CHAIN if the chain uses FO_DOT; FO_ERR_SHAPE if a side does
 * not match X under its access kind; empty X (no cells) writes zeros.
 * Aggregation is by sum; the paper's templates show sums only, and MIN / MAX
 * aggregation is not built.
 */
int fused_cell(const fo_chain *chain, const fo_mat *X,
               const fo_side *sides, int n_sides,
               const double *scalars, int n_scalars,
               int agg, double *out, long long *out_nnz,
               void *ws, size_t ws_bytes, void *stream);

/* ------------------------------------------------------- Cell, built-in scratch
 * (No counterpart in the paper: a deployment variant of fused_cell.)
 *
 * Some callers cannot obtain device memory at the point where they need a fused
 * operator: code that runs inside a region where another component owns the
 * allocator, callbacks that must not call cudaMalloc or a framework allocator
 * (an allocation may synchronise the device, or is simply forbidden there), and
 * hosts whose memory pool is handed out once at start-up.  For them this entry
 * point takes no workspace: the scratch is a 1 MiB array that lives inside the
 * library image on every GPU that loads it, from load until the process exits.
 *
 * Same arguments (without the non-zero count), results and bits as fused_cell
 * (dense X; all four variants).
 * It calls no cudaMalloc / cudaFree and no allocating library routine.  In
 * particular it never compiles or loads a run-time specialised kernel: a chain
 * that fused_cell or fo_jit_prepare specialised earlier is reused (a lookup),
 * any other chain runs through the built-in straight-line code or the
 * interpreter - same bits, lower speed.
 *   - Limit: the call must need at most fused_cell_static_limit_bytes() (1 MiB)
 *     of scratch, i.e. fused_cell_workspace_bytes(X, agg) <= that.  This always
 *     holds for no_agg, row_agg and full_agg.  col_agg keeps one partial row of
 *     `cols` doubles per row panel (up to about 1200 panels for tall matrices),
 *     so it fits for, e.g., 1000 x 1000 or 1 000 000 x 100 but not for
 *     1 000 000 x 1000.  Beyond the limit: FO_ERR_STATIC_LIMIT, nothing is launched.
 *   - The first call on each device looks up the array's device address (a
 *     one-time runtime query, with that device current).  Make that first call
 *     outside any stream capture.
 *   - Every call on a device shares the one array, which keeps what the last
 *     call left in it.  The kernels leave its control words zeroed for the next
 *     call and overwrite the rest before reading it, so calls in sequence on one
 *     stream need no clearing; calls that may overlap on the GPU (different
 *     streams, different threads) race on it and must be serialised by the caller.
 */
int fused_cell_static(const fo_chain *chain, const fo_mat *X,
                      const fo_side *sides, int n_sides,
                      const double *scalars, int n_scalars,
                      int agg, double *out, void *stream);
size_t fused_cell_static_limit_bytes(void);

/* ------------------------------------------------------------------ MAgg
 * Table 1, MAgg template; Section 5.2 "Multi-Aggregate Operations".
 * chain->n_out full-sum aggregates over shared inputs in ONE scan:
 * out[k] = sum over all cells of the chain's k-th result (n_out doubles, the
 * paper's k x 1 output, in the order of chain->out).
 */
int fused_magg(const fo_chain *chain, const fo_mat *X,
               const fo_side *sides, int n_sides,
               const double *scalars, int n_scalars,
               double *out, void *ws, size_t ws_bytes, void *stream);

/* ------------------------------------------------------------------- Row
 * Table 1, Row template; Fig. 1(b); Section 5.2 "Row Operations".
 * One pass over the rows of X (dense or CSR).  For row i:
 *     d   = X_i . v                    (v: device, X.cols doubles)
 *     t_i = chain(d, sides read at row i, scalars)     (sides must be FO_AT_ROW)
 *   FO_ROW_COL_T_AGG: out += t_i * X_i^T   -> out[j] = sum_i t_i X_ij (cols doubles)
 *   FO_ROW_COL_AGG  : the same n sums, read as a 1 x n row
 *   FO_ROW_ROW_AGG  : out[i] = t_i                                   (rows doubles)
 *   FO_ROW_FULL_AGG : out[0] = sum_i t_i
 *   FO_ROW_NO_AGG   : dense X: out[i * cols + j] = t_i * X_ij  (rows x cols, packed);
 *                     CSR X: out[p] = t_i * vals[p] for stored cell p of row i
 *                     (nnz doubles, X's pattern)
 * With the chain  t = side0 * d  this is  t(X) %*% (w * (X %*% v)).
 * The row-wise operator is this fixed skeleton - a product with a side vector (or,
 * in fused_row_b1, a side matrix), a scalar chain on it, and one of the Table 1
 * aggregations - not a free program over the paper's vector primitives
 * (vectMult, vectMinus, vectSum, vectMultAdd composed at will): that general
 * form is not built.
 * X wider than 8192 columns returns FO_ERR_UNSUPPORTED (the single-pass
 * kernels keep a row, respectively v and the output vector, on chip).
 * Determinism: bit-reproducible except FO_ROW_COL_T_AGG / FO_ROW_COL_AGG over
 * CSR, whose scatter-add into on-chip accumulators is unordered.
 */
int fused_row(const fo_chain *chain, const fo_mat *X, const double *v,
              const fo_side *sides, int n_sides,
              const double *scalars, int n_scalars,
              int agg, double *out, void *ws, size_t ws_bytes, void *stream);

/* ---------------------------------------------- Row, matrix-valued intermediates
 * Table 1, Row template, variants no_agg_B1 / col_agg_B1; Eq. 2 and the row-wise
 * operator listing of Section 2.2 (RowType COL_AGG_B1_T); Section 5.2 "Row
 * Operations" (t(X) %*% (X %*% V)) and "Hybrid Algorithms" (k = 2 .. 32).
 * One pass over the rows of X (rows x n).  B is a dense n x k side
 * matrix, 1 <= k <= FO_B1_MAX_K.  For row i:
 *     D_ic = X_i . B[:, c]                       c = 0 .. k-1  (the listing's vectMatMult)
 *     s_i  = sum_c pre(d = D_ic, sides, scalars)               (vectSum; pre may be NULL)
 *     T_ic = post(d = D_ic, sides, s_i, scalars)
 *   FO_ROW_COL_AGG_B1_T: out[j * k + c] = sum_i X_ij T_ic   (n x k, packed; vectOuterMultAdd)
 *   FO_ROW_NO_AGG_B1   : out[i * k + c] = T_ic              (rows x k, packed)
 * In both chains FO_DOT names D_ic.  Sides: FO_AT_CELL sides are rows x k and
 * are read at (i, c); FO_AT_ROW sides rows x 1, read at (i); FO_AT_COL sides
 * 1 x k, read at (c).  In `post`, FO_ROWSUM(n_sides) names s_i: it takes the
 * side slot right behind the call's own sides, so with `pre` given at most
 * FO_MAX_SIDES - 1 sides can be passed; without `pre` that operand is invalid.
 * With pre = NULL and an empty post chain whose result is FO_DOT this is
 * t(X) %*% (X %*% B); with one FO_AT_CELL side P, pre = P * d and
 * post = P * d - P * s it is Eq. 2.
 * X may be CSR: the same operator over the stored cells (a row without stored
 * cells has D_i = 0 and still passes through the chains).  Limits
 * (FO_ERR_UNSUPPORTED beyond them): CSR X: n * k' <= 9600 with k' = k rounded up
 * to a power of two (>= 2); dense X: k <= 32; the columns
 * a group of warps can hold shrink as k grows (n <= 4096 for k <= 2, 2048 for
 * k <= 4, 1024 for k <= 8, 512 for k <= 16, 256 for k <= 32); for col_agg_B1_T
 * n * k <= 24576 (the CTA's output tile lives in shared memory).
 * Bit-reproducible for given shapes over a dense X; over a CSR X the additions
 * into the shared output tile of col_agg_B1_T are unordered.
 */
#define FO_B1_MAX_K 32
#define FO_ROWSUM(n_sides)  FO_SIDE(n_sides)
int fused_row_b1(const fo_chain *pre, const fo_chain *post, const fo_mat *X, const fo_dense *B,
                 const fo_side *sides, int n_sides,
                 const double *scalars, int n_scalars,
                 int agg, double *out, void *ws, size_t ws_bytes, void *stream);

/* ----------------------------------------------------------------- Outer
 * Table 1, Outer template; Fig. 1(d), Eq. 1 and the outer-product listing of
 * Section 2.2.  For every stored cell (i, j) of the CSR matrix X:
 *     a = X_ij,  d = U_i . V_j  (U: rows x rank, V: cols x rank, dense),
 *     w_ij = chain(a, d, sides read at (i, j), scalars)
 *   FO_OUTER_FULL_AGG: out[0] = sum w_ij
 *   FO_OUTER_NO_AGG  : out[p] = w of stored cell p          (nnz doubles)
 *   FO_OUTER_RIGHT_MM: out[i * rank + c] = sum_j w_ij V_jc  (rows x rank, packed)
 *   FO_OUTER_LEFT_MM : out[j * rank + c] = sum_i w_ij U_ic  (cols x rank, packed)
 * FO_OUTER_LEFT_MM adds into rows of `out` shared by all rows of X: global
 * atomics on a zeroed result, so the order of its additions is not fixed; the
 * other variants are bit-reproducible.
 * U V^T is never formed; cells that are not stored cost nothing.  Stored
 * zeros ARE visited (a chain tests a != 0 itself, as the listing does).
 * Side inputs (Table 1 binds dense side inputs to the Outer template as well): at
 * most 3, dense; FO_AT_CELL sides are rows x cols and read at (i, j), FO_AT_ROW
 * sides rows x 1 read at i, FO_AT_COL sides 1 x cols read at j.  A chain that
 * reads a side runs through the general per-cell kernel (no staging of factor
 * rows, no tiled schedule): correct for every variant, slower than a chain over
 * a and d alone.
 * out_nnz (device, one int64, or NULL): with FO_OUTER_NO_AGG the number of
 * written values that are not zero, as for fused_cell; with another variant
 * FO_ERR_UNSUPPORTED.
 * Schedules: per stored cell (factor rows of V staged in shared memory, by bulk
 * copies or 16-byte asynchronous copies depending on the rank), or -
 * when about one cell in seven or more is stored - tile by tile, forming each
 * 64 x 32 tile of U V^T on the fp64 tensor cores and sampling it at the stored
 * cells (full_agg / no_agg).  The library chooses; results agree within the
 * documented tolerance.
 * rank <= 256.  Errors: FO_ERR_SHAPE if U.rows != X.rows, V.rows != X.cols,
 * U.cols != V.cols or a side does not match X under its access kind.
 */
int fused_outer(const fo_chain *chain, const fo_csr *X,
                const fo_dense *U, const fo_dense *V,
                const fo_side *sides, int n_sides,
                const double *scalars, int n_scalars,
                int agg, double *out, long long *out_nnz,
                void *ws, size_t ws_bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* FUSEDOPS_H */
