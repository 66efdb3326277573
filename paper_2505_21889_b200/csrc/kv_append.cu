// efim_kv_append: rotary embedding of the new tokens' q/k fused with the scatter
// of k/v into the paged cache (EFIM Sec. 1: only the `inc` tokens are new and
// they follow `<P>prefix<S>suffix<M>`, so token i of sequence s has position
// cached_len[s] + i).  Pure streaming: every byte is read once and written once.
#include "common.cuh"
#include <math.h>

namespace efim {

struct KvAppendParams {
  uint16_t* q;              // [T][Hq][D] in/out, may be null
  const uint16_t* k_new;    // [T][Hkv][D]
  const uint16_t* v_new;
  uint16_t* k_pool;         // [pages][Hkv][P][D]
  uint16_t* v_pool;
  const int32_t* cached_len;
  const int32_t* q_indptr;
  const int32_t* block_table;
  const float* cos_sin;     // [max_position][D] or null
  int32_t* status;
  int batch, max_pages_per_seq, total_new_tokens;
  int num_pages, Hq, Hkv, max_position, interleaved;
};

// WPT warps per new token, 256 threads per CTA.  A lane keeps one position along the head
// dimension (vector j, and for the rotate-half pairing its partner j + D/16), so its
// cos/sin values are loaded once, and walks the heads - q heads (rotated in place), then
// k heads (rotated into the page slot) - two at a time so that several 16-byte loads are
// in flight per lane; v is copied straight into the page slot.  Many tokens: one warp per
// token keeps every SM full of independent streams.  Few tokens (a decode step): eight
// warps per token, because then the time is one token's latency.
constexpr int KV_APPEND_THREADS = 256;

template <int D, int WPT>
__global__ void __launch_bounds__(KV_APPEND_THREADS) kv_append_kernel(const KvAppendParams p) {
  constexpr int VEC = D / 8;            // 16-byte vectors per head row
  constexpr int HALF = VEC / 2;
  constexpr int LANES = 32 * WPT;       // lanes working on one token
  const int lane = threadIdx.x % LANES;
  const int t = blockIdx.x * (KV_APPEND_THREADS / LANES) + threadIdx.x / LANES;
  if (t >= p.total_new_tokens) return;
  // sequence of this token: last s with q_indptr[s] <= t.  Up to 32 sequences are probed by the
  // warp's lanes at once (one round trip instead of a chain of five); more by bisection.
  int s;
  if (p.batch <= 32) {
    const int wl = threadIdx.x & 31;
    const bool le = wl < p.batch && __ldg(p.q_indptr + wl) <= t;
    s = 31 - __clz((int)(__ballot_sync(0xffffffffu, le) | 1u));
  } else {
    int lo = 0, hi = p.batch;
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (__ldg(p.q_indptr + mid) <= t) lo = mid; else hi = mid;
    }
    s = lo;
  }
  const int pos = __ldg(p.cached_len + s) + (t - __ldg(p.q_indptr + s));
  const int page_idx = pos >> 4;
  int err = 0;
  int page = -1;
  if (pos < 0 || page_idx >= p.max_pages_per_seq || (p.cos_sin && pos >= p.max_position)) {
    err = EFIM_DEV_BAD_POSITION;
  } else {
    page = __ldg(p.block_table + (size_t)s * p.max_pages_per_seq + page_idx);
    if (page < 0 || page >= p.num_pages) err = EFIM_DEV_BAD_PAGE;
  }
  if (err) {
    if (lane == 0 && p.status) atomicOr(p.status, err);
    return;
  }
  const int slot = pos & 15;
  const size_t pool_tok = ((size_t)page * p.Hkv) * 16 * D + (size_t)slot * D;   // + h * 16 * D
  const uint4* kin = reinterpret_cast<const uint4*>(p.k_new + (size_t)t * p.Hkv * D);
  const uint4* vin = reinterpret_cast<const uint4*>(p.v_new + (size_t)t * p.Hkv * D);
  uint4* qio = p.q ? reinterpret_cast<uint4*>(p.q + (size_t)t * p.Hq * D) : nullptr;
  const int nq = p.q ? p.Hq : 0;
  // straight copy of a [Hkv][D] row into the page slot, four vectors in flight per lane
  auto copy_row = [&](const uint4* src, uint16_t* pool) {
    const int n = p.Hkv * VEC;
    for (int u0 = lane; u0 < n; u0 += 4 * LANES) {
      uint4 v[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (u0 + LANES * i < n) v[i] = ldg_stream(src + u0 + LANES * i);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int u = u0 + LANES * i;
        if (u < n) *reinterpret_cast<uint4*>(pool + pool_tok + (size_t)(u / VEC) * 16 * D + (u % VEC) * 8) = v[i];
      }
    }
  };
  copy_row(vin, p.v_pool);
  if (!p.cos_sin) {
    copy_row(kin, p.k_pool);
    return;
  }
  const float* cs = p.cos_sin + (size_t)pos * D;     // cos[0..D/2) then sin[0..D/2)
  const int nh = nq + p.Hkv;
  // where vector `vec` of head h is read from / written to
  auto src_of = [&](int h, int vec) { return h < nq ? qio + h * VEC + vec : kin + (h - nq) * VEC + vec; };
  auto dst_of = [&](int h, int vec) {
    return h < nq ? qio + h * VEC + vec
                  : reinterpret_cast<uint4*>(p.k_pool + pool_tok + (size_t)(h - nq) * 16 * D + vec * 8);
  };
  if (!p.interleaved) {
    constexpr int HP = LANES / HALF;                 // heads the token's lanes cover at once
    const int j = lane % HALF, h0 = lane / HALF;
    float c[8], sn[8];
    *reinterpret_cast<float4*>(c) = __ldg(reinterpret_cast<const float4*>(cs + j * 8));
    *reinterpret_cast<float4*>(c + 4) = __ldg(reinterpret_cast<const float4*>(cs + j * 8 + 4));
    *reinterpret_cast<float4*>(sn) = __ldg(reinterpret_cast<const float4*>(cs + D / 2 + j * 8));
    *reinterpret_cast<float4*>(sn + 4) = __ldg(reinterpret_cast<const float4*>(cs + D / 2 + j * 8 + 4));
    for (int h = h0; h < nh; h += 2 * HP) {
      const int h2 = h + HP;
      uint4 a = *src_of(h, j), b = *src_of(h, j + HALF), a2, b2;
      if (h2 < nh) { a2 = *src_of(h2, j); b2 = *src_of(h2, j + HALF); }
      rotate8(a, b, c, sn);
      *dst_of(h, j) = a;
      *dst_of(h, j + HALF) = b;
      if (h2 < nh) {
        rotate8(a2, b2, c, sn);
        *dst_of(h2, j) = a2;
        *dst_of(h2, j + HALF) = b2;
      }
    }
  } else {
    constexpr int HP = LANES / VEC;
    const int j = lane % VEC, h0 = lane / VEC;
    float c[4], sn[4];
    *reinterpret_cast<float4*>(c) = __ldg(reinterpret_cast<const float4*>(cs + j * 4));
    *reinterpret_cast<float4*>(sn) = __ldg(reinterpret_cast<const float4*>(cs + D / 2 + j * 4));
    for (int h = h0; h < nh; h += 2 * HP) {
      const int h2 = h + HP;
      uint4 a = *src_of(h, j), a2;
      if (h2 < nh) a2 = *src_of(h2, j);
      rotate4_interleaved(a, c, sn);
      *dst_of(h, j) = a;
      if (h2 < nh) {
        rotate4_interleaved(a2, c, sn);
        *dst_of(h2, j) = a2;
      }
    }
  }
}
}  // namespace efim

extern "C" efim_status efim_rope_table_build(double base, int32_t head_dim, int32_t max_position, float* h_out) {
  if (!h_out || head_dim <= 0 || (head_dim & 1) || max_position <= 0 || !(base > 0.0)) return EFIM_ERR_INVALID_ARG;
  const int half = head_dim / 2;
  for (int f = 0; f < half; ++f) {
    const double theta = pow(base, -2.0 * (double)f / (double)head_dim);
    for (int p = 0; p < max_position; ++p) {
      const double ang = (double)p * theta;
      h_out[(size_t)p * head_dim + f] = (float)cos(ang);
      h_out[(size_t)p * head_dim + half + f] = (float)sin(ang);
    }
  }
  return EFIM_OK;
}

extern "C" efim_status efim_kv_append(const efim_cache_desc* cache, const efim_batch_desc* batch,
                                      const efim_rope_desc* rope, void* d_q, const void* d_k_new,
                                      const void* d_v_new, int32_t* d_status, void* stream) {
  efim_status st = efim::check_cache(cache);
  if (st != EFIM_OK) return st;
  st = efim::check_batch(cache, batch, false);
  if (st != EFIM_OK) return st;
  if (batch->batch == 0 || batch->total_new_tokens == 0) return EFIM_OK;
  if (!d_k_new || !d_v_new) return EFIM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_k_new) | reinterpret_cast<uintptr_t>(d_v_new) |
       reinterpret_cast<uintptr_t>(d_q)) & 15) return EFIM_ERR_INVALID_ARG;
  efim::KvAppendParams p{};
  p.q = static_cast<uint16_t*>(d_q);
  p.k_new = static_cast<const uint16_t*>(d_k_new);
  p.v_new = static_cast<const uint16_t*>(d_v_new);
  p.k_pool = static_cast<uint16_t*>(cache->d_k_pool);
  p.v_pool = static_cast<uint16_t*>(cache->d_v_pool);
  p.cached_len = batch->d_cached_len;
  p.q_indptr = batch->d_q_indptr;
  p.block_table = batch->d_block_table;
  p.cos_sin = nullptr;
  if (rope && rope->d_cos_sin) {
    if (rope->max_position <= 0 || (reinterpret_cast<uintptr_t>(rope->d_cos_sin) & 15)) return EFIM_ERR_INVALID_ARG;
    p.cos_sin = rope->d_cos_sin;
    p.max_position = rope->max_position;
    p.interleaved = rope->interleaved;
  }
  p.status = d_status;
  p.batch = batch->batch;
  p.max_pages_per_seq = batch->max_pages_per_seq;
  p.total_new_tokens = batch->total_new_tokens;
  p.num_pages = cache->num_pages;
  p.Hq = cache->num_q_heads;
  p.Hkv = cache->num_kv_heads;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // warps per token: 1 when there are enough tokens to fill the GPU with independent warps, up to 8 for a handful
  const int T = batch->total_new_tokens;
  const int wpt = T >= 16384 ? 1 : T >= 4096 ? 2 : T >= 1024 ? 4 : 8;
  const unsigned grid = (unsigned)(((long long)T * wpt * 32 + efim::KV_APPEND_THREADS - 1) / efim::KV_APPEND_THREADS);
#define EFIM_KV_APPEND_LAUNCH(D_, W_) efim::kv_append_kernel<D_, W_><<<grid, efim::KV_APPEND_THREADS, 0, s>>>(p)
  if (cache->head_dim == 128) {
    if (wpt == 1) EFIM_KV_APPEND_LAUNCH(128, 1);
    else if (wpt == 2) EFIM_KV_APPEND_LAUNCH(128, 2);
    else if (wpt == 4) EFIM_KV_APPEND_LAUNCH(128, 4);
    else EFIM_KV_APPEND_LAUNCH(128, 8);
  } else {
    if (wpt == 1) EFIM_KV_APPEND_LAUNCH(64, 1);
    else if (wpt == 2) EFIM_KV_APPEND_LAUNCH(64, 2);
    else if (wpt == 4) EFIM_KV_APPEND_LAUNCH(64, 4);
    else EFIM_KV_APPEND_LAUNCH(64, 8);
  }
#undef EFIM_KV_APPEND_LAUNCH
  EFIM_CUDA_TRY(cudaGetLastError());
  return EFIM_OK;
}
