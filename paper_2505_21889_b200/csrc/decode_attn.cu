// efim_decode_attn: split-KV paged decode attention with a log-sum-exp merge
// (decode of the generated middle, EFIM Sec. 2.2 / Fig. 4).  Bandwidth-bound:
// every K/V byte of the visible context is read once with 128-bit loads, the dot
// products run on fp32 FMAs, the reductions on warp shuffles; no tensor cores.
//
// One CTA = (query row, kv head [x group tile], key chunk).  Each of its 4 warps
// walks whole pages (16 tokens) round-robin, staged into shared memory by bulk
// copies (one per K page and V page).  Inside a warp D/8 lanes share one token
// row (16 bytes each), so 32/(D/8) tokens are read per 128-bit shared-memory load.
#include "decode_attn.cuh"
#include "mbar.cuh"
#include <algorithm>

namespace efim {

// Sum x[0..N) across the `LPT` lanes of a token group, leaving N/LPT sums per lane.
// Round with lane-bit `off`: lanes with the bit clear keep the lower half of the
// values and receive the partner's lower half; the others the upper half.  After
// all rounds lane j holds the values whose index has, from the top bit down, the
// bits of j; the remaining low index bits enumerate the values it keeps.
template <int N, int LPT>
__device__ __forceinline__ void transposed_reduce(float* x, int j) {
  int n = N;
#pragma unroll
  for (int off = LPT / 2; off >= 1; off >>= 1) {
    const int half = n / 2;
    const bool up = (j & off) != 0;
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
      if (i < half) {
        const float send = up ? x[i] : x[i + half];
        const float keep = up ? x[i + half] : x[i];
        x[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
      }
    }
    n = half;
  }
}

// ---- shared-memory staging of whole pages -------------------------------------------
// One (page, kv head) tile is 16*D*2 contiguous bytes in a pool, so a single bulk copy
// brings it into shared memory.  Every warp owns a ring of DEC_STAGES stages (K page +
// V page), keeps DEC_STAGES pages in flight without holding them in registers, and
// consumes them in order; an mbarrier per stage counts the copied bytes.  Two stages make
// the ring 64 KB per CTA at D = 128, so three CTAs (12 warps) share an SM: the kernel is
// short of warps to issue from, not of bytes in flight (with three stages and two CTAs
// per SM it ran at 84 % of the measured copy bandwidth, with two and three at 99 %).
// Group tiles of more than 4 query heads need the registers of a third CTA for their q and o
// rows: they run two CTAs to an SM and take a third stage instead.
__host__ __device__ constexpr int dec_stages(int group_tile) { return group_tile > 4 ? 3 : 2; }
__host__ __device__ constexpr int dec_ctas_per_sm(int group_tile) { return group_tile > 4 ? 2 : 3; }

__device__ __forceinline__ void dec_bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

// Rotation of one 16-byte vector (8 bf16) of a head row, exactly as efim_kv_append does it
// (fp32 FMA, one rounding to bf16).  Rotate-half pairing: `mine` is vector j of the row,
// `other` vector j ^ (D/16); the first half of the row gets a c - b s, the second b c + a s.
// Interleaved pairing: the pairs (2f, 2f+1) sit inside the vector and `other` is not used.
__device__ __forceinline__ uint4 dec_rotate_vec(uint4 mine, uint4 other, const float* cs, int D, int j, int interleaved) {
  uint32_t* m = reinterpret_cast<uint32_t*>(&mine);
  const uint32_t* o = reinterpret_cast<const uint32_t*>(&other);
  if (!interleaved) {
    const int half = D / 16;
    const bool first = j < half;
    const float* c = cs + (j % half) * 8;
    const float* sn = c + D / 2;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float m0 = bf16lo(m[i]), m1 = bf16hi(m[i]), o0 = bf16lo(o[i]), o1 = bf16hi(o[i]);
      const float c0 = __ldg(c + 2 * i), c1 = __ldg(c + 2 * i + 1), s0 = __ldg(sn + 2 * i), s1 = __ldg(sn + 2 * i + 1);
      const float r0 = first ? fmaf(m0, c0, -(o0 * s0)) : fmaf(m0, c0, o0 * s0);
      const float r1 = first ? fmaf(m1, c1, -(o1 * s1)) : fmaf(m1, c1, o1 * s1);
      m[i] = pack_bf16x2(r0, r1);
    }
  } else {
    const float* c = cs + j * 4;
    const float* sn = c + D / 2;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float a = bf16lo(m[i]), b = bf16hi(m[i]);
      const float ci = __ldg(c + i), si = __ldg(sn + i);
      m[i] = pack_bf16x2(fmaf(a, ci, -(b * si)), fmaf(b, ci, a * si));
    }
  }
  return mine;
}

// GT query heads of one kv head per CTA.  Up to 4 heads are scored in one pass over a staged
// page; 5 to 7 in two passes of 4 (the second padded with zero queries) over the same page in
// shared memory - the K/V bytes come from HBM once.
template <int D, int GT, bool FUSED>
__global__ void __launch_bounds__(128, dec_ctas_per_sm(GT)) decode_splitkv_kernel(const DecodeParams p) {
  constexpr int DEC_STAGES = dec_stages(GT);
  constexpr int LPT = D / 8;            // lanes sharing one token row
  constexpr int TPS = 32 / LPT;         // tokens per warp-wide 16-byte read
  constexpr int STEPS = 16 / TPS;       // reads per page
  constexpr int PH = GT > 4 ? 2 : 1;    // passes over a page's keys
  constexpr int HPP = GT > 4 ? 4 : ((GT + 1) & ~1);   // heads per pass (padded to even)
  constexpr int GP = PH * HPP;          // heads with padding
  constexpr int NV = STEPS * HPP;       // partial dot products per lane per pass
  constexpr int NF = HPP / 2;           // finished scores per lane per pass
  constexpr int PAGE_BYTES = 16 * D * 2;
  static_assert(NV / LPT == NF, "reduction leaves HPP/2 values per lane");

  extern __shared__ __align__(128) uint8_t dec_ring[];   // [4 warps][DEC_STAGES][K page | V page]
  __shared__ __align__(8) uint64_t s_bar[4][DEC_STAGES];
  __shared__ float s_p[4][16][GP];      // per warp: probabilities of the current page
  __shared__ float s_m[4][GP], s_l[4][GP];
  __shared__ float s_o[4][GT][D];

  const int r = blockIdx.x;
  const int G = p.Hq / p.Hkv;
  const int gsplit = (G + GT - 1) / GT;
  const int kvh = blockIdx.y / gsplit;
  const int g0 = (blockIdx.y % gsplit) * GT;
  const int ng = min(GT, G - g0);
  const int c = blockIdx.z;
  // The first block-table entries of every warp are fetched before the row's length is known
  // (any entry of the row may be read; those past the length are dropped below), so that the
  // two loads share one round trip: a short step's time is mostly this ramp.
  const int seq = p.row_seq ? __ldg(p.row_seq + r) : r;
  const int32_t* bt = p.block_table + (size_t)seq * p.max_pages_per_seq;
  const int first_pg = ((c * p.chunk_tokens) >> 4) + (threadIdx.x >> 5);
  const int my_pg = first_pg + 4 * (threadIdx.x & 31);
  const int pid_early = my_pg < p.max_pages_per_seq ? __ldg(bt + my_pg) : -1;
  int len = __ldg(p.row_len + r);
  // longer than the launch was planned for (max_ctx_len) or than the block table can address:
  // clamp and report.  A fused step then has no valid position for its new token and runs as a
  // plain decode over the clamped range.
  bool append = FUSED;
  if (len > p.key_cap) {
    len = p.key_cap;
    append = false;
    if (threadIdx.x == 0 && p.status) atomicOr(p.status, EFIM_DEV_BAD_POSITION);
  }
  const int begin = c * p.chunk_tokens;
  const int head0 = kvh * G + g0;
  const int tid = threadIdx.x;
  // fused step: the new token sits at position len - 1; its rotation needs a table row
  const float* cs_row = nullptr;
  bool skip_row = false;
  if (FUSED && append && len > 0 && p.cos_sin) {
    if (len - 1 >= p.max_position) {
      // no table row for the new token's position: report it and skip the row (nothing is
      // appended; the output is zero, lse -inf)
      if (tid == 0 && p.status) atomicOr(p.status, EFIM_DEV_BAD_POSITION);
      skip_row = true;
    } else {
      cs_row = p.cos_sin + (size_t)(len - 1) * D;
    }
  }
  if (begin >= len || skip_row) {
    // nothing to attend in this chunk.  A row without any key (or a skipped one) still gets a
    // defined result: directly, or as an empty partial for every chunk the merge will read.
    if (p.n_chunks == 1) {
      if (len <= 0 || skip_row) {
        for (int i = tid; i < ng * D; i += 128) p.out[((size_t)r * p.Hq + head0) * D + i] = 0;
        if (p.lse && tid < ng) p.lse[(size_t)r * p.Hq + head0 + tid] = -INFINITY;
      }
    } else if (skip_row && begin < len) {
      for (int i = tid; i < ng * D; i += 128) {
        const size_t row_head = (size_t)r * p.Hq + head0 + i / D;
        p.part_o[(row_head * p.n_chunks + c) * D + i % D] = 0.f;
        if (i % D == 0) p.part_lse[row_head * p.n_chunks + c] = -INFINITY;
      }
    }
    return;
  }
  const int end = min(len, begin + p.chunk_tokens);
  const int lane = tid & 31, warp = tid >> 5;
  const int j = lane % LPT, tg = lane / LPT;

  // ---- this warp's pages: first_pg, first_pg + 4, ... ; start their copies before anything else
  const int last_pg = (end - 1) >> 4;
  const int n_pages = first_pg <= last_pg ? (last_pg - first_pg) / 4 + 1 : 0;
  uint8_t* ring = dec_ring + warp * (DEC_STAGES * 2 * PAGE_BYTES);
  if (lane == 0) {
    for (int sg = 0; sg < DEC_STAGES; ++sg)
      mbar_init(smem_u32(&s_bar[warp][sg]), 1);
    mbar_fence_init();
  }
  __syncwarp();
  // page ids of the next 32 pages of this warp, one per lane (refilled every 32 pages)
  int pid_cache = (lane < n_pages) ? pid_early : -1;
  auto issue = [&](int i) {             // start the copies of this warp's i-th page into stage i % DEC_STAGES
    const int pid = __shfl_sync(0xffffffffu, pid_cache, i & 31);
    const bool ok = pid >= 0 && pid < p.num_pages;
    if (lane == 0) {
      const uint32_t bar = smem_u32(&s_bar[warp][i % DEC_STAGES]);
      if (ok) {
        const uint32_t dst = smem_u32(ring + (i % DEC_STAGES) * 2 * PAGE_BYTES);
        const size_t off = ((size_t)pid * p.Hkv + kvh) * 16 * D;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(2 * PAGE_BYTES) : "memory");
        dec_bulk_load(dst, p.k_pool + off, PAGE_BYTES, bar);
        dec_bulk_load(dst + PAGE_BYTES, p.v_pool + off, PAGE_BYTES, bar);
      } else {
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");   // nothing to copy
        if (p.status) atomicOr(p.status, EFIM_DEV_BAD_PAGE);
      }
    }
    return ok;
  };
  uint32_t ok_bits = 0;                 // which of the in-flight pages are valid (bit = stage)
#pragma unroll
  for (int i = 0; i < DEC_STAGES; ++i)
    if (i < n_pages && issue(i)) ok_bits |= 1u << i;

  // q and o as packed fp32 pairs (dims 2e, 2e+1): the inner products and the P V
  // update run on two-wide FMAs
  uint64_t q2[GP][4];
#pragma unroll
  for (int g = 0; g < GP; ++g) {
    if (g < ng) {
      const uint4* qrow = reinterpret_cast<const uint4*>(p.q + ((size_t)r * p.Hq + head0 + g) * D);
      uint4 w = __ldg(qrow + j);
      if (FUSED && cs_row) w = dec_rotate_vec(w, __ldg(qrow + (j ^ (LPT / 2))), cs_row, D, j, p.interleaved);
      const uint32_t* u = reinterpret_cast<const uint32_t*>(&w);
#pragma unroll
      for (int e = 0; e < 4; ++e) q2[g][e] = pack2(bf16lo(u[e]) * p.scale_log2, bf16hi(u[e]) * p.scale_log2);
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) q2[g][e] = 0ull;
    }
  }
  uint64_t o2[GT][4];
#pragma unroll
  for (int g = 0; g < GT; ++g)
#pragma unroll
    for (int e = 0; e < 4; ++e) o2[g][e] = 0ull;
  float m_run[GP], l_part[PH][NF];
#pragma unroll
  for (int g = 0; g < GP; ++g) m_run[g] = -INFINITY;
#pragma unroll
  for (int ph = 0; ph < PH; ++ph)
#pragma unroll
    for (int i = 0; i < NF; ++i) l_part[ph][i] = 0.f;

  const int odd = j & 1;
  const int st_mine = j >> 1;                   // step whose scores this lane ends up with
  int gave_up_at = -1;                          // page index at which a stage wait expired

  for (int i = 0; i < n_pages; ++i) {
    const int pg = first_pg + 4 * i;
    const int sg = i % DEC_STAGES;
    const bool page_ok = (ok_bits >> sg) & 1u;
    // ---- wait for the stage (bounded; on expiry flag and stop walking)
    {
      const bool ok = mbar_wait_bounded(smem_u32(&s_bar[warp][sg]), (i / DEC_STAGES) & 1, p.wait_ns, nullptr,
                                        lane == 0 ? p.status : nullptr);
      if (__any_sync(0xffffffffu, !ok)) {
        gave_up_at = i;
        break;
      }
    }
    if (FUSED && append && page_ok && pg == ((len - 1) >> 4)) {
      // The page of the new token: whatever the copy brought for its slot is replaced, in
      // shared memory, by the token's rotated k and its v; the CTA of the kv head's first
      // group tile also puts them into the pools.  (Other CTAs that read this page patch
      // their own copy the same way, so nobody depends on when the pool is written.)
      if (tg == 0) {
        const int slot = (len - 1) & 15;
        const uint4* krow = reinterpret_cast<const uint4*>(p.k_new + ((size_t)r * p.Hkv + kvh) * D);
        const uint4* vrow = reinterpret_cast<const uint4*>(p.v_new + ((size_t)r * p.Hkv + kvh) * D);
        uint4 kv = __ldg(krow + j);
        if (cs_row) kv = dec_rotate_vec(kv, __ldg(krow + (j ^ (LPT / 2))), cs_row, D, j, p.interleaved);
        const uint4 vv = __ldg(vrow + j);
        uint8_t* kpage = ring + sg * 2 * PAGE_BYTES;
        *reinterpret_cast<uint4*>(kpage + (slot * D + j * 8) * 2) = kv;
        *reinterpret_cast<uint4*>(kpage + PAGE_BYTES + (slot * D + j * 8) * 2) = vv;
        if (g0 == 0) {
          const int pid = __ldg(bt + pg);
          const size_t off = (((size_t)pid * p.Hkv + kvh) * 16 + slot) * D + j * 8;
          *reinterpret_cast<uint4*>(p.k_pool_w + off) = kv;
          *reinterpret_cast<uint4*>(p.v_pool_w + off) = vv;
        }
      }
      __syncwarp();
    }
    if (page_ok) {
      const uint8_t* kst = ring + sg * 2 * PAGE_BYTES + (tg * D + j * 8) * 2;
      const uint8_t* vst = kst + PAGE_BYTES;
      // ---- scores: partial dot products over this lane's 8 dims, then the cross-lane sum;
      // HPP heads per pass
      const int tok_in_page = st_mine * TPS + tg;       // the token whose scores this lane ends up with
      const bool visible = (pg << 4) + tok_in_page < end;
      float alpha[GP];
#pragma unroll
      for (int ph = 0; ph < PH; ++ph) {
        float x[NV];
#pragma unroll
        for (int st = 0; st < STEPS; ++st) {
          const uint4 kv = *reinterpret_cast<const uint4*>(kst + st * TPS * D * 2);
          const uint32_t* u = reinterpret_cast<const uint32_t*>(&kv);
          uint64_t k2[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) k2[e] = pack2(bf16lo(u[e]), bf16hi(u[e]));
#pragma unroll
          for (int g = 0; g < HPP; ++g) {
            float acc = 0.f;
            if (ph * HPP + g < GT) {
              uint64_t a2 = 0ull;
#pragma unroll
              for (int e = 0; e < 4; ++e) a2 = ffma2(q2[ph * HPP + g][e], k2[e], a2);
              float lo, hi;
              unpack2(a2, lo, hi);
              acc = lo + hi;
            }
            x[st * HPP + g] = acc;
          }
        }
        transposed_reduce<NV, LPT>(x, j);
        // lane j now holds, for token (st_mine*TPS + tg) of the page, heads ph*HPP + odd*NF + i
        float sc[NF], mx[NF];
#pragma unroll
        for (int a = 0; a < NF; ++a) { sc[a] = visible ? x[a] : -INFINITY; mx[a] = sc[a]; }
#pragma unroll
        for (int off = 2; off < 32; off <<= 1)
#pragma unroll
          for (int a = 0; a < NF; ++a) mx[a] = fmaxf(mx[a], __shfl_xor_sync(0xffffffffu, mx[a], off));
        float mine[NF], alpha_mine[NF];
#pragma unroll
        for (int a = 0; a < NF; ++a) {
          const int h_lo = ph * HPP + a, h_hi = ph * HPP + NF + a;
          const float other = __shfl_xor_sync(0xffffffffu, mx[a], 1);
          const float m_lo = odd ? other : mx[a];       // head h_lo
          const float m_hi = odd ? mx[a] : other;       // head h_hi
          const float n_lo = fmaxf(m_run[h_lo], m_lo), n_hi = fmaxf(m_run[h_hi], m_hi);
          alpha[h_lo] = exp2f(m_run[h_lo] - n_lo);
          alpha[h_hi] = exp2f(m_run[h_hi] - n_hi);
          m_run[h_lo] = n_lo;
          m_run[h_hi] = n_hi;
          mine[a] = odd ? n_hi : n_lo;
          alpha_mine[a] = odd ? alpha[h_hi] : alpha[h_lo];
        }
#pragma unroll
        for (int a = 0; a < NF; ++a) {
          const float pr = exp2f(sc[a] - mine[a]);      // masked: exp2(-inf) = 0
          l_part[ph][a] = fmaf(l_part[ph][a], alpha_mine[a], pr);
          s_p[warp][tok_in_page][ph * HPP + odd * NF + a] = pr;
        }
      }
      __syncwarp();
      // ---- values
#pragma unroll
      for (int g = 0; g < GT; ++g) {
        const uint64_t al2 = pack2(alpha[g], alpha[g]);
#pragma unroll
        for (int e = 0; e < 4; ++e) o2[g][e] = fmul2(o2[g][e], al2);
      }
#pragma unroll
      for (int st = 0; st < STEPS; ++st) {
        const int tp = st * TPS + tg;
        if ((pg << 4) + tp < end) {                   // never touch slots past the context
          const uint4 vv = *reinterpret_cast<const uint4*>(vst + st * TPS * D * 2);
          const uint32_t* u = reinterpret_cast<const uint32_t*>(&vv);
          uint64_t v2[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) v2[e] = pack2(bf16lo(u[e]), bf16hi(u[e]));
#pragma unroll
          for (int g = 0; g < GT; ++g) {
            const float pr = s_p[warp][tp][g];
            const uint64_t pr2 = pack2(pr, pr);
#pragma unroll
            for (int e = 0; e < 4; ++e) o2[g][e] = ffma2(pr2, v2[e], o2[g][e]);
          }
        }
      }
    }
    __syncwarp();                                     // everyone is done with the stage and with s_p
    // ---- refill the stage with the page DEC_STAGES ahead
    const int nxt = i + DEC_STAGES;
    if (nxt < n_pages) {
      if ((nxt & 31) == 0) pid_cache = (nxt + lane < n_pages) ? __ldg(bt + first_pg + 4 * (nxt + lane)) : -1;
      ok_bits &= ~(1u << sg);
      if (issue(nxt)) ok_bits |= 1u << sg;
    }
  }

  if (gave_up_at >= 0) {
    // copies issued for the stages still in flight must land before the CTA's shared memory
    // can be handed to another CTA
    for (int k = gave_up_at; k < min(gave_up_at + DEC_STAGES, n_pages); ++k)
      mbar_drain(smem_u32(&s_bar[warp][k % DEC_STAGES]), (k / DEC_STAGES) & 1);
  }
  float o[GT][8];
#pragma unroll
  for (int g = 0; g < GT; ++g)
#pragma unroll
    for (int e = 0; e < 4; ++e) unpack2(o2[g][e], o[g][2 * e], o[g][2 * e + 1]);
  // ---- fold the token groups of the warp, then the 4 warps
#pragma unroll
  for (int off = LPT; off < 32; off <<= 1)
#pragma unroll
    for (int g = 0; g < GT; ++g)
#pragma unroll
      for (int e = 0; e < 8; ++e) o[g][e] += __shfl_xor_sync(0xffffffffu, o[g][e], off);
#pragma unroll
  for (int off = 2; off < 32; off <<= 1)
#pragma unroll
    for (int ph = 0; ph < PH; ++ph)
#pragma unroll
      for (int i = 0; i < NF; ++i) l_part[ph][i] += __shfl_xor_sync(0xffffffffu, l_part[ph][i], off);
  if (lane < 2) {
#pragma unroll
    for (int ph = 0; ph < PH; ++ph)
#pragma unroll
      for (int i = 0; i < NF; ++i) s_l[warp][ph * HPP + lane * NF + i] = l_part[ph][i];
  }
  if (lane == 0) {
#pragma unroll
    for (int g = 0; g < GP; ++g) s_m[warp][g] = m_run[g];
  }
  if (tg == 0) {
#pragma unroll
    for (int g = 0; g < GT; ++g)
#pragma unroll
      for (int e = 0; e < 8; ++e) s_o[warp][g][j * 8 + e] = o[g][e];
  }
  __syncthreads();
  for (int idx = tid; idx < ng * D; idx += 128) {
    const int g = idx / D, d = idx % D;
    float M = fmaxf(fmaxf(s_m[0][g], s_m[1][g]), fmaxf(s_m[2][g], s_m[3][g]));   // warp 0 always has a page
    float L = 0.f, O = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float sc = exp2f(s_m[w][g] - M);
      L = fmaf(s_l[w][g], sc, L);
      O = fmaf(s_o[w][g][d], sc, O);
    }
    const float val = (L > 0.f) ? O / L : 0.f;    // all pages of the chunk rejected: defined output
    const size_t row_head = (size_t)r * p.Hq + head0 + g;
    if (p.n_chunks == 1) {
      p.out[row_head * D + d] = __bfloat16_as_ushort(__float2bfloat16_rn(val));
      if (p.lse && d == 0) p.lse[row_head] = (M + log2f(L)) * 0.6931471805599453f;
    } else {
      p.part_o[(row_head * p.n_chunks + c) * D + d] = val;
      if (d == 0) p.part_lse[row_head * p.n_chunks + c] = M + log2f(L);
    }
  }
}

// Merge the chunk partials of one (row, head): lse = log2 sum 2^lse_c,
// o = sum 2^(lse_c - lse) o_c.  One warp per (row, head), lanes over head_dim.
template <int D>
__global__ void __launch_bounds__(128) decode_merge_kernel(const DecodeParams p) {
  constexpr int EPL = D / 32;
  const int lane = threadIdx.x & 31;
  const size_t row_head = (size_t)blockIdx.x * 4 + (threadIdx.x >> 5);
  if (row_head >= (size_t)p.R * p.Hq) return;
  const int r = (int)(row_head / p.Hq);
  const int len = min(__ldg(p.row_len + r), p.key_cap);
  uint16_t* out = p.out + row_head * D + lane * EPL;
  if (len <= 0) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) out[e] = 0;
    if (p.lse && lane == 0) p.lse[row_head] = -INFINITY;
    return;
  }
  const int nc = min((len + p.chunk_tokens - 1) / p.chunk_tokens, p.n_chunks);
  const float* pl = p.part_lse + row_head * p.n_chunks;
  const float* po = p.part_o + row_head * p.n_chunks * D + lane * EPL;
  // the lanes fetch the chunks' lse values side by side; the partial rows are then loaded four
  // at a time and folded in chunk order (a chain of dependent loads cost more than the split
  // kernel's tail on short steps)
  float M = -INFINITY;
  for (int c0 = 0; c0 < nc; c0 += 32)
    if (c0 + lane < nc) M = fmaxf(M, __ldg(pl + c0 + lane));
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, d));
  if (M == -INFINITY) {                            // every chunk came back empty (a skipped row)
#pragma unroll
    for (int e = 0; e < EPL; ++e) out[e] = 0;
    if (p.lse && lane == 0) p.lse[row_head] = -INFINITY;
    return;
  }
  float L = 0.f, acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  for (int c0 = 0; c0 < nc; c0 += 4) {
    float w[4];
    __align__(16) float v[4][EPL];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (c0 + i < nc) {
        w[i] = __ldg(pl + c0 + i);
        if constexpr (EPL == 4) {
          *reinterpret_cast<float4*>(v[i]) = __ldg(reinterpret_cast<const float4*>(po + (size_t)(c0 + i) * D));
        } else {
          *reinterpret_cast<float2*>(v[i]) = __ldg(reinterpret_cast<const float2*>(po + (size_t)(c0 + i) * D));
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (c0 + i < nc) {
        const float wi = exp2f(w[i] - M);
        L += wi;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] = fmaf(wi, v[i][e], acc[e]);
      }
    }
  }
  const float inv = 1.f / L;
#pragma unroll
  for (int e = 0; e < EPL; ++e) out[e] = __bfloat16_as_ushort(__float2bfloat16_rn(acc[e] * inv));
  if (p.lse && lane == 0) p.lse[row_head] = (M + log2f(L)) * 0.6931471805599453f;
}

DecodePlan plan_decode(int rows, int Hq, int Hkv, int D, int max_len) {
  DecodePlan pl;
  const int G = Hq / Hkv;
  // Groups of up to 7 query heads share one CTA's walk over the K/V pages (5 to 7 in two
  // passes over the page in shared memory: 3.1-3.7 TB/s of K/V against 3.0 when the pages
  // were fetched twice).  From 8 heads on the fp32 FMAs, not the bytes, are the bound (8 heads
  // in one CTA measured 1.9 TB/s against 3.2 as two CTAs of 4), so larger groups are cut into
  // tiles of 4, or of 3 where that divides the group and 4 does not.
  if (G <= 7) {
    pl.group_tile = G;
  } else {
    pl.group_tile = (G % 4 != 0 && G % 3 == 0) ? 3 : 4;
  }
  pl.gsplit = (G + pl.group_tile - 1) / pl.group_tile;
  if (max_len < 1) max_len = 1;
  // Aim for ~32 CTAs per SM over the launch so that ragged lengths even out, but keep a
  // chunk between 768 and 2048 tokens (384 KB .. 1 MB of K+V at head_dim 128): a CTA pays
  // a few microseconds before its pages stream, and shorter chunks were measured slower
  // (16 rows x 8 kv heads x 2.5k keys: 48.9 us per step with 256-key chunks, 43 with 768).
  // Only when that leaves fewer than two CTAs per SM do the chunks shrink, down to 256.
  const long long n_sm = sm_count();
  const long long ctas_per_chunkless = (long long)rows * Hkv * pl.gsplit;
  long long want_chunks = (n_sm * 32 + ctas_per_chunkless - 1) / ctas_per_chunkless;
  if (want_chunks < 1) want_chunks = 1;
  long long chunk = (max_len + want_chunks - 1) / want_chunks;
  if (chunk < 768) chunk = 768;
  if (chunk > 2048) chunk = 2048;
  if (ctas_per_chunkless * ((max_len + chunk - 1) / chunk) < n_sm * 2) {
    const long long need_chunks = (n_sm * 2 + ctas_per_chunkless - 1) / ctas_per_chunkless;
    chunk = std::max<long long>(256, (max_len + need_chunks - 1) / need_chunks);
    if (chunk > 2048) chunk = 2048;
  }
  chunk = (chunk + 63) / 64 * 64;
  pl.chunk_tokens = (int)chunk;
  pl.n_chunks = (max_len + pl.chunk_tokens - 1) / pl.chunk_tokens;
  pl.part_o_bytes = pl.n_chunks > 1 ? (size_t)rows * Hq * pl.n_chunks * D * sizeof(float) : 0;
  pl.part_lse_bytes = pl.n_chunks > 1 ? ((size_t)rows * Hq * pl.n_chunks * sizeof(float) + 255) / 256 * 256 : 0;
  return pl;
}

template <int D, int GT, bool FUSED>
static efim_status launch_split_f(const DecodeParams& p, dim3 grid, cudaStream_t s) {
  constexpr int ring_bytes = 4 * dec_stages(GT) * 2 * 16 * D * 2;  // 4 warps x stages x (K page + V page)
  EFIM_CUDA_TRY(cudaFuncSetAttribute(decode_splitkv_kernel<D, GT, FUSED>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, ring_bytes));
  decode_splitkv_kernel<D, GT, FUSED><<<grid, 128, ring_bytes, s>>>(p);
  return EFIM_OK;
}
template <int D, int GT>
static efim_status launch_split(const DecodeParams& p, dim3 grid, cudaStream_t s) {
  return p.fused ? launch_split_f<D, GT, true>(p, grid, s) : launch_split_f<D, GT, false>(p, grid, s);
}

template <int D>
static efim_status launch_decode_d(const DecodeParams& p, const DecodePlan& pl, cudaStream_t s) {
  dim3 grid(p.R, p.Hkv * pl.gsplit, pl.n_chunks);
  efim_status st;
  switch (pl.group_tile) {
    case 1: st = launch_split<D, 1>(p, grid, s); break;
    case 2: st = launch_split<D, 2>(p, grid, s); break;
    case 3: st = launch_split<D, 3>(p, grid, s); break;
    case 4: st = launch_split<D, 4>(p, grid, s); break;
    case 5: st = launch_split<D, 5>(p, grid, s); break;
    case 6: st = launch_split<D, 6>(p, grid, s); break;
    default: st = launch_split<D, 7>(p, grid, s); break;
  }
  if (st != EFIM_OK) return st;
  EFIM_CUDA_TRY(cudaGetLastError());
  if (pl.n_chunks > 1) {
    const unsigned blocks = (unsigned)(((size_t)p.R * p.Hq + 3) / 4);
    decode_merge_kernel<D><<<blocks, 128, 0, s>>>(p);
    EFIM_CUDA_TRY(cudaGetLastError());
  }
  return EFIM_OK;
}

efim_status launch_decode(const DecodeParams& p, const DecodePlan& pl, int D, cudaStream_t s) {
  if (p.R == 0) return EFIM_OK;
  if (p.R > 2147483647 / 4 || p.Hkv * pl.gsplit > 65535 || pl.n_chunks > 65535) return EFIM_ERR_UNSUPPORTED;
  return D == 128 ? launch_decode_d<128>(p, pl, s) : launch_decode_d<64>(p, pl, s);
}

}  // namespace efim

extern "C" size_t efim_decode_workspace_bytes(const efim_cache_desc* cache, int32_t batch, int32_t max_ctx_len) {
  if (efim::check_cache(cache) != EFIM_OK || batch <= 0) return 0;
  const efim::DecodePlan pl = efim::plan_decode(batch, cache->num_q_heads, cache->num_kv_heads, cache->head_dim,
                                                max_ctx_len);
  return pl.part_o_bytes + pl.part_lse_bytes;
}

extern "C" int32_t efim_decode_launch_count(const efim_cache_desc* cache, int32_t batch, int32_t max_ctx_len) {
  if (efim::check_cache(cache) != EFIM_OK || batch <= 0) return 0;
  const efim::DecodePlan pl = efim::plan_decode(batch, cache->num_q_heads, cache->num_kv_heads, cache->head_dim,
                                                max_ctx_len);
  return pl.n_chunks > 1 ? 2 : 1;
}

efim_status efim::decode_run(const efim_cache_desc* cache, int32_t batch, const int32_t* d_ctx_len,
                             int32_t max_ctx_len, const int32_t* d_block_table, int32_t max_pages_per_seq,
                             const efim_rope_desc* rope, const void* d_k_new, const void* d_v_new, bool fused,
                             const void* d_q, void* d_out, float* d_lse, float sm_scale, void* d_workspace,
                             size_t workspace_bytes, int32_t* d_status, void* stream, WorkspaceSource ws_source) {
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
  if (need > 0) {
    if (ws_source) {
      st = ws_source(&d_workspace, &workspace_bytes);
      if (st != EFIM_OK) return st;
    }
    if (!d_workspace || workspace_bytes < need) return EFIM_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(d_workspace) & 255) return EFIM_ERR_INVALID_ARG;
  }
  efim::DecodeParams p{};
  p.q = static_cast<const uint16_t*>(d_q);
  p.k_pool = static_cast<const uint16_t*>(cache->d_k_pool);
  p.v_pool = static_cast<const uint16_t*>(cache->d_v_pool);
  p.row_len = d_ctx_len;
  p.row_seq = nullptr;
  p.block_table = d_block_table;
  p.out = static_cast<uint16_t*>(d_out);
  p.lse = d_lse;
  p.part_lse = static_cast<float*>(d_workspace);
  p.part_o = need ? reinterpret_cast<float*>(static_cast<char*>(d_workspace) + pl.part_lse_bytes) : nullptr;
  p.status = d_status;
  p.R = batch;
  p.Hq = cache->num_q_heads;
  p.Hkv = cache->num_kv_heads;
  p.max_pages_per_seq = max_pages_per_seq;
  p.num_pages = cache->num_pages;
  p.chunk_tokens = pl.chunk_tokens;
  p.n_chunks = pl.n_chunks;
  p.key_cap = (int)std::min<long long>((long long)pl.n_chunks * pl.chunk_tokens, cap);
  p.wait_ns = efim::WAIT_LIMIT_NS;
  const float scale = sm_scale > 0.f ? sm_scale : 1.0f / sqrtf((float)cache->head_dim);
  p.scale_log2 = scale * 1.4426950408889634f;
  if (fused) {
    if (!d_k_new || !d_v_new) return EFIM_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(d_k_new) | reinterpret_cast<uintptr_t>(d_v_new)) & 15) return EFIM_ERR_INVALID_ARG;
    p.fused = 1;
    p.k_new = static_cast<const uint16_t*>(d_k_new);
    p.v_new = static_cast<const uint16_t*>(d_v_new);
    p.k_pool_w = static_cast<uint16_t*>(cache->d_k_pool);
    p.v_pool_w = static_cast<uint16_t*>(cache->d_v_pool);
    if (rope && rope->d_cos_sin) {
      if (rope->max_position <= 0 || (reinterpret_cast<uintptr_t>(rope->d_cos_sin) & 15)) return EFIM_ERR_INVALID_ARG;
      p.cos_sin = rope->d_cos_sin;
      p.max_position = rope->max_position;
      p.interleaved = rope->interleaved;
    }
  }
  return efim::launch_decode(p, pl, cache->head_dim, static_cast<cudaStream_t>(stream));
}

extern "C" efim_status efim_decode_attn(const efim_cache_desc* cache, int32_t batch, const int32_t* d_ctx_len,
                                        int32_t max_ctx_len, const int32_t* d_block_table,
                                        int32_t max_pages_per_seq, const void* d_q, void* d_out, float* d_lse,
                                        float sm_scale, void* d_workspace, size_t workspace_bytes,
                                        int32_t* d_status, void* stream) {
  return efim::decode_run(cache, batch, d_ctx_len, max_ctx_len, d_block_table, max_pages_per_seq, nullptr, nullptr,
                      nullptr, false, d_q, d_out, d_lse, sm_scale, d_workspace, workspace_bytes, d_status, stream);
}

extern "C" efim_status efim_decode_step(const efim_cache_desc* cache, int32_t batch, const int32_t* d_ctx_len,
                                        int32_t max_ctx_len, const int32_t* d_block_table,
                                        int32_t max_pages_per_seq, const efim_rope_desc* rope, const void* d_q,
                                        const void* d_k_new, const void* d_v_new, void* d_out, float* d_lse,
                                        float sm_scale, void* d_workspace, size_t workspace_bytes,
                                        int32_t* d_status, void* stream) {
  return efim::decode_run(cache, batch, d_ctx_len, max_ctx_len, d_block_table, max_pages_per_seq, rope, d_k_new,
                      d_v_new, true, d_q, d_out, d_lse, sm_scale, d_workspace, workspace_bytes, d_status, stream);
}
