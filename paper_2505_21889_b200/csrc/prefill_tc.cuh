// Internal interface of the tensor-core append-prefill kernel.
#pragma once
#include <cuda.h>
#include "common.cuh"

namespace efim {
namespace pf {

constexpr int BM = 128;        // query rows per tile (one TMEM lane each)
constexpr int BN = 128;        // keys per KV tile (8 pages)
constexpr int NQ = 2;          // query tiles per CTA sharing one K/V stream
constexpr int NSTAGE = 5;      // K/V ring entries (one K or V tile of 128 keys each)
constexpr int NSTAGE_MAX = 6;  // ring entries when there is a single query tile (the other tile's space is used)
constexpr int THREADS = 384;   // 2 softmax warpgroups + 1 service warpgroup (2 TMA warps, 2 MMA warps)
// Register split (setmaxnreg): the block launches with 168 registers per thread
// (65536 / 384, rounded to 8) = 64512 in total; 2 x 128 x 216 + 128 x 72 = 64512 uses them all
// (the sum must not exceed the launch total: an increase beyond it would wait forever).  With
// 64 registers the service warps spilled a few words inside the MMA-issuing loop.
constexpr int REGS_SOFTMAX = 216;
constexpr int REGS_SERVICE = 72;

// One CTA's work: packed rows [row0, row0 + 256) of (seq, kv head) against KV tiles
// [tile_begin, tile_end).  Packed row R = token * G + head-in-group.  The sequence's
// lengths and first query row ride along (the planner has them from the host mirrors),
// so that a CTA's first dependent chain is "item -> block table / query rows" instead of
// "item -> lengths -> block table / query rows".
struct WorkItem {
  int32_t seq;
  int16_t kvh;
  int16_t chunk;               // >= 0: write a partial for this KV chunk; -1: final output
  int32_t row0, tile_begin, tile_end;
  int32_t cached, new_len;     // cached_len[seq], new_len[seq]
  int32_t tok0;                // q_indptr[seq]
};
static_assert(sizeof(WorkItem) == 32, "work items are read as two 16-byte vectors");

struct Params {
  const uint16_t* q;           // [T][Hq][D]
  uint16_t* out;               // [T][Hq][D]
  float* lse;                  // [T][Hq] or null
  const int32_t* cached_len;
  const int32_t* new_len;
  const int32_t* q_indptr;
  const int32_t* block_table;
  const WorkItem* items;
  const int32_t* split_tokens; // [batch] keys per KV chunk of a split sequence, 0 = not split
  float* part_o;               // [T][Hq][s_max][D]
  float* part_lse;             // [T][Hq][s_max]  base-2
  int32_t* status;
  int batch, total_new_tokens;
  int Hq, Hkv, G, max_pages_per_seq, num_pages, s_max;
  float scale_log2;
  unsigned long long wait_ns;  // limit of every device-side wait
  // rotation of the query rows as they are loaded (null: q is already rotated)
  const float* cos_sin;        // [max_position][D]
  int max_position, interleaved;
};

struct Plan {
  int n_items;
  int s_max;                   // largest KV split count (1 = no partials, no merge)
  size_t items_bytes, split_bytes, part_lse_bytes, part_o_bytes;
  size_t total() const { return items_bytes + split_bytes + part_lse_bytes + part_o_bytes; }
};

// Host: size the plan (items == nullptr) or fill `items`/`split_tokens` too.
Plan make_plan(const efim_cache_desc* c, const efim_batch_desc* b, WorkItem* items, int32_t* split_tokens);

efim_status launch(const efim_cache_desc* c, const Params& p, const Plan& pl, cudaStream_t s);

}  // namespace pf
}  // namespace efim
