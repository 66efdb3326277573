// Status strings and version of the EFIM C ABI.
#include <atomic>
#include <cuda_runtime.h>
#include "common.cuh"

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

extern "C" int efim_version(void) { return 200; }

namespace efim {
// SM count of the current device (the planners size their grids by it), remembered per
// device; 148 (a B200) when no device can be asked, so that sizing queries still answer.
int sm_count() {
  constexpr int kMaxDevices = 64;
  static std::atomic<int> cached[kMaxDevices];
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return 148;
  }
  if (dev >= 0 && dev < kMaxDevices) {
    const int c = cached[dev].load(std::memory_order_relaxed);
    if (c > 0) return c;
  }
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    return 148;
  }
  if (dev >= 0 && dev < kMaxDevices) cached[dev].store(n, std::memory_order_relaxed);
  return n;
}
}  // namespace efim
