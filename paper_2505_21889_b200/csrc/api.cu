// Status strings and version of the EFIM C ABI.
#include <cuda_runtime.h>
#include "efim.h"

static thread_local int g_last_cuda_error = 0;

extern "C" void efim_note_cuda_error(int code) { g_last_cuda_error = code; }

extern "C" const char* efim_last_cuda_error(void) {
  return g_last_cuda_error ? cudaGetErrorString(static_cast<cudaError_t>(g_last_cuda_error)) : "no error";
}

extern "C" const char* efim_strerror(efim_status s) {
  switch (s) {
    case EFIM_OK: return "ok";
    case EFIM_ERR_INVALID_ARG: return "invalid argument";
    case EFIM_ERR_UNSUPPORTED: return "unsupported shape";
    case EFIM_ERR_OUT_OF_RANGE: return "length out of range";
    case EFIM_ERR_WORKSPACE: return "workspace too small";
    case EFIM_ERR_CUDA: return "CUDA call failed";
    case EFIM_ERR_TIMEOUT: return "device wait timed out";
  }
  return "unknown status";
}

extern "C" int efim_version(void) { return 100; }
