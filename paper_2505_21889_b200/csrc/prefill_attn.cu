// efim_append_prefill_attn: causal attention of the new `inc` tokens over the
// cached `<P>prefix<S>suffix<M>` keys and over each other (EFIM Sec. 1, Sec. 2.2).
// Host side: validates, plans the work list from the host length mirrors, copies
// it into the workspace and launches the tensor-core kernel (prefill_tc.cu).
#include <vector>
#include "prefill_tc.cuh"

extern "C" size_t efim_prefill_workspace_bytes(const efim_cache_desc* cache, const efim_batch_desc* batch) {
  if (efim::check_cache(cache) != EFIM_OK || efim::check_batch(cache, batch, true) != EFIM_OK) return 0;
  if (batch->batch == 0 || batch->total_new_tokens == 0) return 0;
  return efim::pf::make_plan(cache, batch, nullptr, nullptr).total();
}

extern "C" int32_t efim_prefill_launch_count(const efim_cache_desc* cache, const efim_batch_desc* batch) {
  if (efim::check_cache(cache) != EFIM_OK || efim::check_batch(cache, batch, true) != EFIM_OK) return 0;
  if (batch->batch == 0 || batch->total_new_tokens == 0) return 0;
  const efim::pf::Plan pl = efim::pf::make_plan(cache, batch, nullptr, nullptr);
  return pl.n_items == 0 ? 0 : (pl.s_max > 1 ? 2 : 1);
}

extern "C" efim_status efim_append_prefill_attn(const efim_cache_desc* cache, const efim_batch_desc* batch,
                                                const void* d_q, void* d_out, float* d_lse, float sm_scale,
                                                void* d_workspace, size_t workspace_bytes, int32_t* d_status,
                                                void* stream) {
  using namespace efim;
  efim_status st = check_cache(cache);
  if (st != EFIM_OK) return st;
  st = check_batch(cache, batch, true);
  if (st != EFIM_OK) return st;
  if (batch->batch == 0 || batch->total_new_tokens == 0) return EFIM_OK;
  if (!d_q || !d_out) return EFIM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_q) | reinterpret_cast<uintptr_t>(d_out)) & 15) return EFIM_ERR_INVALID_ARG;
  const pf::Plan sized = pf::make_plan(cache, batch, nullptr, nullptr);
  if (!d_workspace || workspace_bytes < sized.total()) return EFIM_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(d_workspace) & 255) return EFIM_ERR_INVALID_ARG;
  // work list + per-sequence split sizes, built in one host block and copied once
  std::vector<unsigned char> host(sized.items_bytes + sized.split_bytes);
  pf::WorkItem* items = reinterpret_cast<pf::WorkItem*>(host.data());
  int32_t* split = reinterpret_cast<int32_t*>(host.data() + sized.items_bytes);
  const pf::Plan pl = pf::make_plan(cache, batch, items, split);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(d_workspace);
  EFIM_CUDA_TRY(cudaMemcpyAsync(ws, host.data(), host.size(), cudaMemcpyHostToDevice, s));
  pf::Params p{};
  p.q = static_cast<const uint16_t*>(d_q);
  p.out = static_cast<uint16_t*>(d_out);
  p.lse = d_lse;
  p.cached_len = batch->d_cached_len;
  p.new_len = batch->d_new_len;
  p.q_indptr = batch->d_q_indptr;
  p.block_table = batch->d_block_table;
  p.items = reinterpret_cast<const pf::WorkItem*>(ws);
  p.split_tokens = reinterpret_cast<const int32_t*>(ws + pl.items_bytes);
  p.part_lse = reinterpret_cast<float*>(ws + pl.items_bytes + pl.split_bytes);
  p.part_o = reinterpret_cast<float*>(ws + pl.items_bytes + pl.split_bytes + pl.part_lse_bytes);
  p.status = d_status;
  p.batch = batch->batch;
  p.total_new_tokens = batch->total_new_tokens;
  p.Hq = cache->num_q_heads;
  p.Hkv = cache->num_kv_heads;
  p.G = cache->num_q_heads / cache->num_kv_heads;
  p.max_pages_per_seq = batch->max_pages_per_seq;
  p.num_pages = cache->num_pages;
  p.s_max = pl.s_max;
  const float scale = sm_scale > 0.f ? sm_scale : 1.0f / sqrtf((float)cache->head_dim);
  p.scale_log2 = scale * 1.4426950408889634f;
  return pf::launch(cache, p, pl, s);
}
