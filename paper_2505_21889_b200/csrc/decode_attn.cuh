// Internal interface of the split-KV row-attention kernels (shared by the
// decode entry point and the small-row path of append-prefill).
#pragma once
#include "common.cuh"

namespace efim {

struct DecodeParams {
  const uint16_t* q;          // [R][Hq][D] bf16
  const uint16_t* k_pool;     // [pages][Hkv][16][D]
  const uint16_t* v_pool;
  const int32_t* row_len;     // [R] keys visible to row r: [0, row_len[r])
  const int32_t* row_seq;     // [R] block-table row of r, or null for identity
  const int32_t* block_table; // [*][max_pages_per_seq]
  uint16_t* out;              // [R][Hq][D] bf16
  float* lse;                 // [R][Hq] natural log, or null
  float* part_o;              // [R][Hq][n_chunks][D]   (n_chunks > 1)
  float* part_lse;            // [R][Hq][n_chunks]      base-2 log
  int32_t* status;
  int R, Hq, Hkv, max_pages_per_seq, num_pages, chunk_tokens, n_chunks;
  int key_cap;                // keys the launch can cover: min(n_chunks * chunk_tokens, table capacity);
                              // a longer device length is clamped to it and reported
  unsigned long long wait_ns; // limit of every device-side wait
  float scale_log2;           // sm_scale * log2(e)
  // fused decode step: the row's last key (position row_len[r] - 1) is this step's new token.
  // Its k/v are rotated, put into the page slot and used from shared memory in the same
  // kernel; q comes in unrotated.  All null / 0 for a plain decode.
  const uint16_t* k_new;      // [R][Hkv][D]
  const uint16_t* v_new;
  uint16_t* k_pool_w;         // the pools again, writable
  uint16_t* v_pool_w;
  const float* cos_sin;       // [max_position][D] or null (no rotation)
  int fused, interleaved, max_position;
};

struct DecodePlan {
  int group_tile;             // q heads of one kv head handled per CTA (<= 7)
  int gsplit;                 // CTAs per kv head
  int chunk_tokens;           // keys per chunk (multiple of 64)
  int n_chunks;
  size_t part_o_bytes, part_lse_bytes;
};

DecodePlan plan_decode(int rows, int Hq, int Hkv, int D, int max_len);
efim_status launch_decode(const DecodeParams& p, const DecodePlan& pl, int D, cudaStream_t s);

// Validation, planning and launch behind efim_decode_attn, efim_decode_step (fused = true:
// rope / d_k_new / d_v_new are used) and efim_decode_attn_static.  The latter passes a
// `ws_source`: asked, once the arguments have passed validation and only if the plan needs
// partials, for the workspace to use (the library's fixed array) in place of the caller's.
typedef efim_status (*WorkspaceSource)(void** d_workspace, size_t* workspace_bytes);
efim_status decode_run(const efim_cache_desc* cache, int32_t batch, const int32_t* d_ctx_len, int32_t max_ctx_len,
                       const int32_t* d_block_table, int32_t max_pages_per_seq, const efim_rope_desc* rope,
                       const void* d_k_new, const void* d_v_new, bool fused, const void* d_q, void* d_out,
                       float* d_lse, float sm_scale, void* d_workspace, size_t workspace_bytes, int32_t* d_status,
                       void* stream, WorkspaceSource ws_source = nullptr);

}  // namespace efim
