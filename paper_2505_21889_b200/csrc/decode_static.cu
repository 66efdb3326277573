// efim_decode_attn_static: decode attention for callers that cannot allocate.
//
// Some callers have no way to obtain a workspace: code running where cudaMalloc is
// forbidden (a serving loop that has handed all device memory to its KV pool and
// must not allocate again, a plug-in that is only given input/output pointers, a
// real-time thread where an allocation could block on the driver).  For them the
// chunk partials live in one fixed array inside the library instead of a
// caller-provided workspace.  Everything else (kernels, chunking, results) is the
// path efim_decode_attn takes.
#include <atomic>
#include <mutex>
#include "decode_attn.cuh"

namespace {

constexpr size_t kScratchBytes = 8u << 20;     // 8 MiB per GPU, held from library load to exit
static __device__ __align__(256) unsigned char g_decode_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices];             // device address of the array, per device
std::atomic<bool> g_scratch_ready[kMaxDevices];
std::mutex g_scratch_mutex;

// In host code `g_decode_scratch` is only a handle for the symbol; its address on the
// current device has to be asked for once per device.
efim_status scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return EFIM_ERR_CUDA;
  if (!g_scratch_ready[dev].load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ready[dev].load(std::memory_order_relaxed)) {
      void* ptr = nullptr;
      if (cudaGetSymbolAddress(&ptr, g_decode_scratch) != cudaSuccess || ptr == nullptr) return EFIM_ERR_CUDA;
      g_scratch_addr[dev] = ptr;
      g_scratch_ready[dev].store(true, std::memory_order_release);
    }
  }
  *out = g_scratch_addr[dev];
  return EFIM_OK;
}

efim_status scratch_source(void** d_workspace, size_t* workspace_bytes) {
  *workspace_bytes = kScratchBytes;
  return scratch_for_current_device(d_workspace);
}

}  // namespace

extern "C" size_t efim_decode_static_scratch_bytes(void) { return kScratchBytes; }

extern "C" efim_status efim_decode_attn_static(const efim_cache_desc* cache, int32_t batch,
                                               const int32_t* d_ctx_len, int32_t max_ctx_len,
                                               const int32_t* d_block_table, int32_t max_pages_per_seq,
                                               const void* d_q, void* d_out, float* d_lse, float sm_scale,
                                               int32_t* d_status, void* stream) {
  // Same validation, plan and kernels as efim_decode_attn, with the library's array as the
  // workspace: a request that needs more than the array holds comes back as EFIM_ERR_WORKSPACE.
  // Every partial the merge kernel reads is written by this call's split kernel first, so
  // what an earlier call left in the array never has to be cleared.
  return efim::decode_run(cache, batch, d_ctx_len, max_ctx_len, d_block_table, max_pages_per_seq, nullptr, nullptr,
                          nullptr, false, d_q, d_out, d_lse, sm_scale, nullptr, 0, d_status, stream, scratch_source);
}
