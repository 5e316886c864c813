// Tensor-core (tcgen05) engine of the large contractions.
#pragma once

#include "dion_common.cuh"

namespace dion {

// One-time per-process set-up of the tensor-core kernels (shared-memory opt-in).
inline int umma_configure() { return DION_OK; }

// Returns 1 if the product was launched on the tensor cores, 0 if this engine
// does not take the product (the caller then uses the fp32 FMA engine), or a
// negative DION_ERR_* code.
inline int umma_try_launch(const GemmArgs&, int /*precision*/, int /*sm_count*/, cudaStream_t) { return 0; }

}  // namespace dion
