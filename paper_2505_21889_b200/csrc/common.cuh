// Shared host/device helpers for the EFIM kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "efim.h"

// the CUDA error behind the calling thread's last EFIM_ERR_CUDA (api.cu)
extern "C" void efim_note_cuda_error(int code);

#define EFIM_CUDA_TRY(expr)                          \
  do {                                               \
    cudaError_t e__ = (expr);                        \
    if (e__ != cudaSuccess) {                        \
      efim_note_cuda_error((int)e__);                \
      return EFIM_ERR_CUDA;                          \
    }                                                \
  } while (0)

namespace efim {

// SM count of the current device, cached per device (api.cu)
int sm_count();

// Validation shared by every entry point: shapes the kernels are built for.
inline efim_status check_cache(const efim_cache_desc* c) {
  if (!c || !c->d_k_pool || !c->d_v_pool) return EFIM_ERR_INVALID_ARG;
  if (c->num_pages <= 0 || c->num_q_heads <= 0 || c->num_kv_heads <= 0) return EFIM_ERR_INVALID_ARG;
  if (c->num_q_heads % c->num_kv_heads != 0) return EFIM_ERR_INVALID_ARG;
  if (c->num_kv_heads > 32767) return EFIM_ERR_UNSUPPORTED;
  // a (page, kv head) pair is one 32-bit coordinate of the prefill kernel's page copies
  if ((long long)c->num_pages * c->num_kv_heads > 0x7fffffffLL) return EFIM_ERR_UNSUPPORTED;
  if (c->page_size != 16) return EFIM_ERR_UNSUPPORTED;
  if (c->head_dim != 64 && c->head_dim != 128) return EFIM_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(c->d_k_pool) & 127) || (reinterpret_cast<uintptr_t>(c->d_v_pool) & 127))
    return EFIM_ERR_INVALID_ARG;
  return EFIM_OK;
}

inline efim_status check_batch(const efim_cache_desc* c, const efim_batch_desc* b, bool need_host) {
  if (!b) return EFIM_ERR_INVALID_ARG;
  if (b->batch < 0 || b->total_new_tokens < 0 || b->max_pages_per_seq <= 0) return EFIM_ERR_INVALID_ARG;
  if (b->batch == 0) return EFIM_OK;
  if (!b->d_cached_len || !b->d_new_len || !b->d_q_indptr || !b->d_block_table) return EFIM_ERR_INVALID_ARG;
  if (need_host) {
    if (!b->h_cached_len || !b->h_new_len) return EFIM_ERR_INVALID_ARG;
    long long total = 0;
    const long long cap = (long long)b->max_pages_per_seq * c->page_size;
    for (int s = 0; s < b->batch; ++s) {
      if (b->h_cached_len[s] < 0 || b->h_new_len[s] < 0) return EFIM_ERR_INVALID_ARG;
      if ((long long)b->h_cached_len[s] + b->h_new_len[s] > cap) return EFIM_ERR_OUT_OF_RANGE;
      total += b->h_new_len[s];
    }
    if (total != b->total_new_tokens) return EFIM_ERR_INVALID_ARG;
  }
  return EFIM_OK;
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// two floats -> packed bf16x2 (round to nearest even); lo lands in the low half
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// packed pairs of fp32 (one 64-bit register): two FMAs / multiplies per instruction
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t fmul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// ---- rotary embedding, as every kernel of the library applies it: fp32 FMA from the bf16
// inputs and the fp32 cos/sin table, one rounding to bf16.  (The same instruction sequence
// everywhere, so a q or k rotated by one kernel equals the one rotated by another bit for bit.)
// Rotate 8 (a, b) pairs held in two 16-byte vectors: a' = a c - b s, b' = b c + a s.
__device__ __forceinline__ void rotate8(uint4& va, uint4& vb, const float* c, const float* s) {
  uint32_t* a = reinterpret_cast<uint32_t*>(&va);
  uint32_t* b = reinterpret_cast<uint32_t*>(&vb);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float a0 = bf16lo(a[i]), a1 = bf16hi(a[i]);
    float b0 = bf16lo(b[i]), b1 = bf16hi(b[i]);
    float ra0 = fmaf(a0, c[2 * i], -(b0 * s[2 * i]));
    float ra1 = fmaf(a1, c[2 * i + 1], -(b1 * s[2 * i + 1]));
    float rb0 = fmaf(b0, c[2 * i], a0 * s[2 * i]);
    float rb1 = fmaf(b1, c[2 * i + 1], a1 * s[2 * i + 1]);
    a[i] = pack_bf16x2(ra0, ra1);
    b[i] = pack_bf16x2(rb0, rb1);
  }
}

// Interleaved pairing: one 16-byte vector holds 4 pairs (2f, 2f+1).
__device__ __forceinline__ void rotate4_interleaved(uint4& v, const float* c, const float* s) {
  uint32_t* w = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float a = bf16lo(w[i]), b = bf16hi(w[i]);
    float ra = fmaf(a, c[i], -(b * s[i]));
    float rb = fmaf(b, c[i], a * s[i]);
    w[i] = pack_bf16x2(ra, rb);
  }
}

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

}  // namespace efim
