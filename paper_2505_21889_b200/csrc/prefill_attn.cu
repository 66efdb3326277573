// efim_append_prefill_attn: causal attention of the new `inc` tokens over the
// cached `<P>prefix<S>suffix<M>` keys and over each other (EFIM Sec. 1, Sec. 2.2).
// Host side: validates, plans the work list from the host length mirrors, copies
// it into the workspace and launches the tensor-core kernel (prefill_tc.cu).
#include <cstring>
#include <vector>
#include "prefill_tc.cuh"
#include "mbar.cuh"

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

namespace {
// Head of a host plan blob; the work list and the per-sequence split sizes follow it.
struct PlanHeader {
  uint32_t magic;
  int32_t batch, total_new_tokens, Hq, Hkv, D, n_items, s_max;
  uint64_t lengths_hash;                 // of the host mirrors the plan was made from
  uint64_t items_bytes, split_bytes, part_lse_bytes, part_o_bytes;
};
constexpr uint32_t PLAN_MAGIC = 0x4d494645u;      // "EFIM"
constexpr size_t PLAN_HEAD_BYTES = 256;

uint64_t lengths_hash(const efim_batch_desc* b) {
  uint64_t h = 1469598103934665603ull;
  for (int s = 0; s < b->batch; ++s) {
    h = (h ^ (uint32_t)b->h_cached_len[s]) * 1099511628211ull;
    h = (h ^ (uint32_t)b->h_new_len[s]) * 1099511628211ull;
  }
  return h;
}
bool batch_has_work(const efim_batch_desc* b) { return b->batch != 0 && b->total_new_tokens != 0; }

// Writes header and lists of a plan whose list sizes are already known (`sized`).
void fill_plan(const efim_cache_desc* cache, const efim_batch_desc* batch, const efim::pf::Plan* sized, void* h_plan) {
  using namespace efim;
  PlanHeader hd{};
  hd.magic = PLAN_MAGIC;
  hd.batch = batch->batch;
  hd.total_new_tokens = batch->total_new_tokens;
  hd.Hq = cache->num_q_heads;
  hd.Hkv = cache->num_kv_heads;
  hd.D = cache->head_dim;
  hd.lengths_hash = lengths_hash(batch);
  if (sized) {
    unsigned char* body = static_cast<unsigned char*>(h_plan) + PLAN_HEAD_BYTES;
    memset(body, 0, sized->items_bytes + sized->split_bytes);
    const pf::Plan pl = pf::make_plan(cache, batch, reinterpret_cast<pf::WorkItem*>(body),
                                      reinterpret_cast<int32_t*>(body + sized->items_bytes));
    hd.n_items = pl.n_items;
    hd.s_max = pl.s_max;
    hd.items_bytes = pl.items_bytes;
    hd.split_bytes = pl.split_bytes;
    hd.part_lse_bytes = pl.part_lse_bytes;
    hd.part_o_bytes = pl.part_o_bytes;
  }
  memset(h_plan, 0, PLAN_HEAD_BYTES);
  memcpy(h_plan, &hd, sizeof(hd));
}
}  // namespace

extern "C" size_t efim_prefill_plan_bytes(const efim_cache_desc* cache, const efim_batch_desc* batch) {
  if (efim::check_cache(cache) != EFIM_OK || efim::check_batch(cache, batch, true) != EFIM_OK) return 0;
  if (!batch_has_work(batch)) return PLAN_HEAD_BYTES;
  const efim::pf::Plan pl = efim::pf::make_plan(cache, batch, nullptr, nullptr);
  return PLAN_HEAD_BYTES + pl.items_bytes + pl.split_bytes;
}

extern "C" efim_status efim_prefill_plan(const efim_cache_desc* cache, const efim_batch_desc* batch, void* h_plan,
                                         size_t plan_bytes) {
  using namespace efim;
  efim_status st = check_cache(cache);
  if (st != EFIM_OK) return st;
  st = check_batch(cache, batch, true);
  if (st != EFIM_OK) return st;
  if (!h_plan || plan_bytes < PLAN_HEAD_BYTES) return EFIM_ERR_INVALID_ARG;
  if (!batch_has_work(batch)) {
    fill_plan(cache, batch, nullptr, h_plan);
    return EFIM_OK;
  }
  const pf::Plan sized = pf::make_plan(cache, batch, nullptr, nullptr);
  if (plan_bytes < PLAN_HEAD_BYTES + sized.items_bytes + sized.split_bytes) return EFIM_ERR_WORKSPACE;
  fill_plan(cache, batch, &sized, h_plan);
  return EFIM_OK;
}

namespace {
// Runs a plan.  `rope` with a table: the query rows are rotated as the kernel loads them.
efim_status run_planned(const efim_cache_desc* cache, const efim_batch_desc* batch, const efim_rope_desc* rope,
                        const void* h_plan, size_t plan_bytes, int32_t lists_resident, const void* d_q, void* d_out,
                        float* d_lse, float sm_scale, void* d_workspace, size_t workspace_bytes, int32_t* d_status,
                        void* stream) {
  using namespace efim;
  efim_status st = check_cache(cache);
  if (st != EFIM_OK) return st;
  st = check_batch(cache, batch, true);
  if (st != EFIM_OK) return st;
  if (!h_plan || plan_bytes < PLAN_HEAD_BYTES) return EFIM_ERR_INVALID_ARG;
  PlanHeader hd;
  memcpy(&hd, h_plan, sizeof(hd));
  // the plan must be the one made for this cache shape and these lengths
  if (hd.magic != PLAN_MAGIC || hd.batch != batch->batch || hd.total_new_tokens != batch->total_new_tokens ||
      hd.Hq != cache->num_q_heads || hd.Hkv != cache->num_kv_heads || hd.D != cache->head_dim ||
      hd.lengths_hash != lengths_hash(batch) || plan_bytes < PLAN_HEAD_BYTES + hd.items_bytes + hd.split_bytes)
    return EFIM_ERR_INVALID_ARG;
  if (!batch_has_work(batch) || hd.n_items == 0) return EFIM_OK;
  if (!d_q || !d_out) return EFIM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_q) | reinterpret_cast<uintptr_t>(d_out)) & 15) return EFIM_ERR_INVALID_ARG;
  pf::Plan pl{};
  pl.n_items = hd.n_items;
  pl.s_max = hd.s_max;
  pl.items_bytes = hd.items_bytes;
  pl.split_bytes = hd.split_bytes;
  pl.part_lse_bytes = hd.part_lse_bytes;
  pl.part_o_bytes = hd.part_o_bytes;
  if (!d_workspace || workspace_bytes < pl.total()) return EFIM_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(d_workspace) & 255) return EFIM_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(d_workspace);
  // work list + per-sequence split sizes go to the head of the workspace in one copy
  // (unless an earlier call with this plan and workspace has left them there)
  if (!lists_resident)
    EFIM_CUDA_TRY(cudaMemcpyAsync(ws, static_cast<const unsigned char*>(h_plan) + PLAN_HEAD_BYTES,
                                  pl.items_bytes + pl.split_bytes, cudaMemcpyHostToDevice, s));
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
  p.wait_ns = WAIT_LIMIT_NS;
  if (rope && rope->d_cos_sin) {
    if (rope->max_position <= 0 || (reinterpret_cast<uintptr_t>(rope->d_cos_sin) & 15)) return EFIM_ERR_INVALID_ARG;
    p.cos_sin = rope->d_cos_sin;
    p.max_position = rope->max_position;
    p.interleaved = rope->interleaved;
  }
  return pf::launch(cache, p, pl, s);
}

// Plans into a temporary blob, then runs it.
efim_status plan_and_run(const efim_cache_desc* cache, const efim_batch_desc* batch, const efim_rope_desc* rope,
                         const void* d_q, void* d_out, float* d_lse, float sm_scale, void* d_workspace,
                         size_t workspace_bytes, int32_t* d_status, void* stream) {
  using namespace efim;
  efim_status st = check_cache(cache);
  if (st != EFIM_OK) return st;
  st = check_batch(cache, batch, true);
  if (st != EFIM_OK) return st;
  if (!batch_has_work(batch)) return EFIM_OK;
  const pf::Plan sized = pf::make_plan(cache, batch, nullptr, nullptr);
  std::vector<unsigned char> blob(PLAN_HEAD_BYTES + sized.items_bytes + sized.split_bytes);
  fill_plan(cache, batch, &sized, blob.data());
  return run_planned(cache, batch, rope, blob.data(), blob.size(), 0, d_q, d_out, d_lse, sm_scale, d_workspace,
                     workspace_bytes, d_status, stream);
}
}  // namespace

extern "C" efim_status efim_append_prefill_attn_planned(const efim_cache_desc* cache, const efim_batch_desc* batch,
                                                        const void* h_plan, size_t plan_bytes,
                                                        int32_t lists_resident, const void* d_q, void* d_out,
                                                        float* d_lse, float sm_scale, void* d_workspace,
                                                        size_t workspace_bytes, int32_t* d_status, void* stream) {
  return run_planned(cache, batch, nullptr, h_plan, plan_bytes, lists_resident, d_q, d_out, d_lse, sm_scale,
                     d_workspace, workspace_bytes, d_status, stream);
}

// Plan and run in one call.
extern "C" efim_status efim_append_prefill_attn(const efim_cache_desc* cache, const efim_batch_desc* batch,
                                                const void* d_q, void* d_out, float* d_lse, float sm_scale,
                                                void* d_workspace, size_t workspace_bytes, int32_t* d_status,
                                                void* stream) {
  return plan_and_run(cache, batch, nullptr, d_q, d_out, d_lse, sm_scale, d_workspace, workspace_bytes, d_status,
                      stream);
}

// Steps 1 and 2 of a turn: the new tokens' k/v go into the pages (k rotated), then the new
// queries, rotated as they are loaded, attend over everything before them.
extern "C" efim_status efim_append_prefill_step(const efim_cache_desc* cache, const efim_batch_desc* batch,
                                                const efim_rope_desc* rope, const void* d_q, const void* d_k_new,
                                                const void* d_v_new, void* d_out, float* d_lse, float sm_scale,
                                                const void* h_plan, size_t plan_bytes, int32_t lists_resident,
                                                void* d_workspace, size_t workspace_bytes, int32_t* d_status,
                                                void* stream) {
  if ((d_k_new == nullptr) != (d_v_new == nullptr)) return EFIM_ERR_INVALID_ARG;
  if (d_k_new) {
    const efim_status st = efim_kv_append(cache, batch, rope, nullptr, d_k_new, d_v_new, d_status, stream);
    if (st != EFIM_OK) return st;
  }
  if (h_plan)
    return run_planned(cache, batch, rope, h_plan, plan_bytes, lists_resident, d_q, d_out, d_lse, sm_scale,
                       d_workspace, workspace_bytes, d_status, stream);
  return plan_and_run(cache, batch, rope, d_q, d_out, d_lse, sm_scale, d_workspace, workspace_bytes, d_status, stream);
}
