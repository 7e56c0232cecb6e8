// Host-side helpers shared by the translation units of the library (not part of the ABI).
#pragma once

#include <cuda_runtime.h>

namespace espo {

// Remember a failed CUDA call for espo_last_cuda_error() and map it to ESPO_ERR_CUDA.
int record_cuda_error(cudaError_t e);

#define ESPO_CUDA_TRY(expr)                                            \
  do {                                                                 \
    cudaError_t espo_e_ = (expr);                                      \
    if (espo_e_ != cudaSuccess) return ::espo::record_cuda_error(espo_e_); \
  } while (0)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace espo
