// Interface of the run-time specialiser (jit.cu) towards the Cell / MAgg entry points.
#pragma once

#include "cell_flat.cuh"

namespace fo {

constexpr int kJitUnavailable = 1;     // not an error: the caller uses the interpreter instead

bool jit_enabled();

// Launches the flat streaming kernel specialised for `ch`.  With `may_compile` (and
// the process-wide mode "compile at first use") a chain seen for the first time is
// compiled, loaded and cached; otherwise only an already cached kernel is used and
// nothing is compiled, loaded or allocated.  Returns FO_OK if launched,
// kJitUnavailable if there is no specialised kernel (not cached and compiling not
// allowed, NVRTC or the driver library missing, switched off, or the compilation
// failed), FO_ERR_CUDA if the launch itself failed.
int jit_launch_flat(const DevChain &ch, const CellParams &p, bool store, int grid, cudaStream_t st,
                    bool may_compile);

}  // namespace fo
