// Error reporting shared by all entry points of the library.
#include <cuda_runtime.h>

#include "espo.h"
#include "espo_host.h"

namespace espo {
static thread_local int g_last_cuda_error = 0;
int record_cuda_error(cudaError_t e) {
  g_last_cuda_error = (int)e;
  (void)cudaGetLastError();   // clear the runtime's sticky copy of a launch-configuration error
  return ESPO_ERR_CUDA;
}
}  // namespace espo

extern "C" {

const char* espo_strerror(int code) {
  switch (code) {
    case ESPO_OK: return "ok";
    case ESPO_ERR_NULL: return "a required pointer was NULL";
    case ESPO_ERR_BAD_DTYPE: return "unknown element type code";
    case ESPO_ERR_BAD_SHAPE: return "bad size or stride";
    case ESPO_ERR_ALIGN: return "pointer not aligned as required";
    case ESPO_ERR_CAPACITY: return "more rows or tokens than the state or workspace can hold";
    case ESPO_ERR_CUDA: return "a CUDA runtime call failed (see espo_last_cuda_error)";
    case ESPO_ERR_BAD_PARAM: return "parameter outside its documented range";
    default: return "unknown error code";
  }
}

int espo_last_cuda_error(void) { return espo::g_last_cuda_error; }

}  // extern "C"
