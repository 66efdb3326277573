// efim_selftest_bounded_wait: exercises the give-up branch of the library's bounded device
// wait in isolation.  One warp waits on an mbarrier that nothing will ever complete - no
// copy, no MMA, nothing else in flight - so the wait must run into its limit, record
// EFIM_DEV_TIMEOUT and return; the kernel then ends normally and the context stays usable.
#include "mbar.cuh"

namespace efim {
__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(unsigned long long limit_ns, int32_t* status,
                                                                  unsigned long long* waited_ns) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    mbar_fence_init();
    abort_flag = 0;
  }
  __syncwarp();
  const unsigned long long t0 = global_ns();
  const bool completed = mbar_wait_bounded(smem_u32(&bar), 0, limit_ns, &abort_flag, status);
  // a second wait after the expiry returns at once: the abort flag is up
  mbar_wait_bounded(smem_u32(&bar), 0, limit_ns, &abort_flag, status);
  const unsigned long long t1 = global_ns();
  if (threadIdx.x == 0 && waited_ns) *waited_ns = completed ? 0ull : t1 - t0;
}
}  // namespace efim

extern "C" efim_status efim_selftest_bounded_wait(uint64_t limit_ns, int32_t* d_status, uint64_t* d_waited_ns,
                                                  void* stream) {
  if (!d_status || limit_ns == 0 || limit_ns > 100000000ull) return EFIM_ERR_INVALID_ARG;   // at most 0.1 s
  efim::bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
      limit_ns, d_status, reinterpret_cast<unsigned long long*>(d_waited_ns));
  EFIM_CUDA_TRY(cudaGetLastError());
  return EFIM_OK;
}
