// efim_append_prefill_attn: causal attention of the new `inc` tokens over the
// cached `<P>prefix<S>suffix<M>` keys and over each other (EFIM Sec. 1, Sec. 2.2).
//
// Row path: every new token is treated as one query row with its own visible
// length C + i + 1 and handed to the split-KV row kernels.
#include "decode_attn.cuh"

namespace efim {

// row t of the packed batch -> (block-table row, number of visible keys)
__global__ void expand_rows_kernel(const int32_t* __restrict__ q_indptr, const int32_t* __restrict__ cached_len,
                                   int batch, int total, int32_t* __restrict__ row_len,
                                   int32_t* __restrict__ row_seq) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= total) return;
  int lo = 0, hi = batch;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (__ldg(q_indptr + mid) <= t) lo = mid; else hi = mid;
  }
  row_seq[t] = lo;
  row_len[t] = __ldg(cached_len + lo) + (t - __ldg(q_indptr + lo)) + 1;
}

struct PrefillPlan {
  int max_len;
  size_t rows_bytes;      // row_len + row_seq
  DecodePlan dec;
};

static PrefillPlan plan_prefill(const efim_cache_desc* c, const efim_batch_desc* b) {
  PrefillPlan pl{};
  int max_len = 1;
  for (int s = 0; s < b->batch; ++s)
    if (b->h_new_len[s] > 0) max_len = max(max_len, b->h_cached_len[s] + b->h_new_len[s]);
  pl.max_len = max_len;
  pl.rows_bytes = ((size_t)b->total_new_tokens * 2 * sizeof(int32_t) + 255) / 256 * 256;
  pl.dec = plan_decode(b->total_new_tokens, c->num_q_heads, c->num_kv_heads, c->head_dim, max_len);
  return pl;
}

}  // namespace efim

extern "C" size_t efim_prefill_workspace_bytes(const efim_cache_desc* cache, const efim_batch_desc* batch) {
  if (efim::check_cache(cache) != EFIM_OK || efim::check_batch(cache, batch, true) != EFIM_OK) return 0;
  if (batch->batch == 0 || batch->total_new_tokens == 0) return 0;
  const efim::PrefillPlan pl = efim::plan_prefill(cache, batch);
  return pl.rows_bytes + pl.dec.part_lse_bytes + pl.dec.part_o_bytes;
}

extern "C" efim_status efim_append_prefill_attn(const efim_cache_desc* cache, const efim_batch_desc* batch,
                                                const void* d_q, void* d_out, float* d_lse, float sm_scale,
                                                void* d_workspace, size_t workspace_bytes, int32_t* d_status,
                                                void* stream) {
  efim_status st = efim::check_cache(cache);
  if (st != EFIM_OK) return st;
  st = efim::check_batch(cache, batch, true);
  if (st != EFIM_OK) return st;
  if (batch->batch == 0 || batch->total_new_tokens == 0) return EFIM_OK;
  if (!d_q || !d_out) return EFIM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_q) | reinterpret_cast<uintptr_t>(d_out)) & 15) return EFIM_ERR_INVALID_ARG;
  const efim::PrefillPlan pl = efim::plan_prefill(cache, batch);
  const size_t need = pl.rows_bytes + pl.dec.part_lse_bytes + pl.dec.part_o_bytes;
  if (!d_workspace || workspace_bytes < need) return EFIM_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(d_workspace) & 255) return EFIM_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int T = batch->total_new_tokens;
  char* ws = static_cast<char*>(d_workspace);
  int32_t* row_len = reinterpret_cast<int32_t*>(ws);
  int32_t* row_seq = row_len + T;
  efim::expand_rows_kernel<<<(T + 255) / 256, 256, 0, s>>>(batch->d_q_indptr, batch->d_cached_len, batch->batch, T,
                                                          row_len, row_seq);
  EFIM_CUDA_TRY(cudaGetLastError());
  efim::DecodeParams p{};
  p.q = static_cast<const uint16_t*>(d_q);
  p.k_pool = static_cast<const uint16_t*>(cache->d_k_pool);
  p.v_pool = static_cast<const uint16_t*>(cache->d_v_pool);
  p.row_len = row_len;
  p.row_seq = row_seq;
  p.block_table = batch->d_block_table;
  p.out = static_cast<uint16_t*>(d_out);
  p.lse = d_lse;
  p.part_lse = reinterpret_cast<float*>(ws + pl.rows_bytes);
  p.part_o = reinterpret_cast<float*>(ws + pl.rows_bytes + pl.dec.part_lse_bytes);
  p.status = d_status;
  p.R = T;
  p.Hq = cache->num_q_heads;
  p.Hkv = cache->num_kv_heads;
  p.max_pages_per_seq = batch->max_pages_per_seq;
  p.num_pages = cache->num_pages;
  p.chunk_tokens = pl.dec.chunk_tokens;
  p.n_chunks = pl.dec.n_chunks;
  const float scale = sm_scale > 0.f ? sm_scale : 1.0f / sqrtf((float)cache->head_dim);
  p.scale_log2 = scale * 1.4426950408889634f;
  return efim::launch_decode(p, pl.dec, cache->head_dim, s);
}
