// Interface of the run-time specialiser (jit.cu) towards the Cell / MAgg entry points.
#pragma once

#include "cell_csr.cuh"
#include "cell_tiles.cuh"

namespace fo {

constexpr int kJitUnavailable = 1;     // not an error: the caller uses the interpreter instead

bool jit_enabled();
bool jit_first_use();          // the mode in which an entry point may compile a chain it sees for the first time

// Which skeleton a run-time specialised kernel instantiates, and with which template
// arguments (their meaning depends on the kind; see wrapper_text in jit.cu).
enum JitKind { kJitFlat = 0, kJitRows = 1, kJitCols = 2, kJitCsr = 3, kJitOuterDirect = 4, kJitOuterPipe = 5,
               kJitOuterDense = 6, kJitRowDense = 7, kJitRowNarrow = 8, kJitRowCsr = 9, kJitRowCsrReg = 10,
               kJitOuterBulk = 11 };
struct JitSpec {
    int kind, a, b, c, d, e;
};

// Launches the kernel `sp` specialised for `ch`.  With `may_compile` a chain seen for
// the first time is compiled, loaded and cached; otherwise only an already cached
// kernel is used and nothing is compiled, loaded or allocated.  (An entry point passes
// may_compile only in the mode "compile at first use"; an explicit prepare call always.)
// With launch = false the kernel is only made ready.  Returns FO_OK if
// launched (made ready), kJitUnavailable if there is no specialised kernel (not
// cached and compiling not allowed, NVRTC or the driver library missing, switched
// off, or the compilation failed), FO_ERR_CUDA if the launch itself failed.
// `params` points to the kernel's parameter block: CellParams, CsrCellParams for kJitCsr,
// OuterParams for the Outer kernels (the tiled one takes a DenseSplit as `params2`), RowParams for
// the Row kernels; `smem`: dynamic shared memory of the launch; `block`: threads per CTA.
int jit_launch(const JitSpec &sp, const DevChain &ch, const void *params, unsigned grid_x, unsigned grid_y,
               cudaStream_t st, bool may_compile, bool launch, size_t smem = 0, const void *params2 = nullptr,
               unsigned block = kThreads);

// CTAs of the cached kernel `sp` for `ch` that fit on an SM (0 if there is none).
int jit_occupancy(const JitSpec &sp, const DevChain &ch);

}  // namespace fo
