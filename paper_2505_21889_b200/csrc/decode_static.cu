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

}  // namespace

extern "C" size_t efim_decode_static_scratch_bytes(void) { return kScratchBytes; }

extern "C" efim_status efim_decode_attn_static(const efim_cache_desc* cache, int32_t batch,
                                               const int32_t* d_ctx_len, int32_t max_ctx_len,
                                               const int32_t* d_block_table, int32_t max_pages_per_seq,
                                               const void* d_q, void* d_out, float* d_lse, float sm_scale,
                                               int32_t* d_status, void* stream) {
  efim_status st = efim::check_cache(cache);
  if (st != EFIM_OK) return st;
  if (batch < 0 || max_pages_per_seq <= 0) return EFIM_ERR_INVALID_ARG;
  if (batch == 0) return EFIM_OK;
  if (!d_ctx_len || !d_block_table || !d_q || !d_out) return EFIM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_q) | reinterpret_cast<uintptr_t>(d_out)) & 15) return EFIM_ERR_INVALID_ARG;
  const long long cap = (long long)max_pages_per_seq * cache->page_size;
  if (max_ctx_len <= 0) max_ctx_len = (int32_t)(cap > 2147483647LL ? 2147483647LL : cap);
  if (max_ctx_len > cap) return EFIM_ERR_OUT_OF_RANGE;
  const efim::DecodePlan pl = efim::plan_decode(batch, cache->num_q_heads, cache->num_kv_heads, cache->head_dim,
                                                max_ctx_len);
  const size_t need = pl.part_o_bytes + pl.part_lse_bytes;
  if (need > kScratchBytes) return EFIM_ERR_WORKSPACE;      // batch x heads x chunks too large for the fixed array
  void* scratch = nullptr;
  st = scratch_for_current_device(&scratch);
  if (st != EFIM_OK) return st;
  efim::DecodeParams p{};
  p.q = static_cast<const uint16_t*>(d_q);
  p.k_pool = static_cast<const uint16_t*>(cache->d_k_pool);
  p.v_pool = static_cast<const uint16_t*>(cache->d_v_pool);
  p.row_len = d_ctx_len;
  p.row_seq = nullptr;
  p.block_table = d_block_table;
  p.out = static_cast<uint16_t*>(d_out);
  p.lse = d_lse;
  // every partial the merge kernel reads is written by this call's split kernel
  // first, so what an earlier call left in the array never has to be cleared
  p.part_lse = static_cast<float*>(scratch);
  p.part_o = reinterpret_cast<float*>(static_cast<char*>(scratch) + pl.part_lse_bytes);
  p.status = d_status;
  p.R = batch;
  p.Hq = cache->num_q_heads;
  p.Hkv = cache->num_kv_heads;
  p.max_pages_per_seq = max_pages_per_seq;
  p.num_pages = cache->num_pages;
  p.chunk_tokens = pl.chunk_tokens;
  p.n_chunks = pl.n_chunks;
  const float scale = sm_scale > 0.f ? sm_scale : 1.0f / sqrtf((float)cache->head_dim);
  p.scale_log2 = scale * 1.4426950408889634f;
  return efim::launch_decode(p, pl, cache->head_dim, static_cast<cudaStream_t>(stream));
}
