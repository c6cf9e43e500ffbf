// Cell / MAgg over a CSR main input (cell_csr.cu), called from the entry points
// in cell.cu.
#pragma once

#include "common.cuh"

namespace fo {

size_t cell_csr_ws_bytes(int agg, int n_out);

int run_cell_csr(const fo_chain *chain, const fo_csr &X, const fo_side *sides, int n_sides,
                 const double *scalars, int n_scalars, int agg, bool magg, double *out, void *ws,
                 size_t ws_bytes, void *stream, bool may_compile);

}  // namespace fo
