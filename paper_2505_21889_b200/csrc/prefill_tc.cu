// Tensor-core append-prefill attention for sm_100a (EFIM Sec. 1, Sec. 2.2: the new
// `inc` queries attend causally over the cached `<P>prefix<S>suffix<M>` keys and
// over each other).
//
// One CTA owns up to 256 packed query rows (row = token * G + head-in-group) of one
// (sequence, kv head) as two 128-row tiles, and streams the visible K/V range in
// tiles of 128 keys (8 pages):
//   warps 8,11 TMA producers (K tiles / V tiles): walk the block table, one tiled bulk-tensor
//             copy per page (16 slots x all dims of the kv head) into a 5- or 6-entry
//             shared-memory ring (128B swizzle)
//   warp 10   issues the tcgen05.mma for S_t = Q_t K^T into TMEM
//   warp 9    issues the tcgen05.mma for O_t += P_t V (P read from TMEM)
//   warps 0-7 two softmax groups, one per query tile, one TMEM lane (row) per thread:
//             S from TMEM, mask, running max with lazy rescale, exp2, P (bf16) back to
//             TMEM over S, final normalisation and store
// Hand-offs are mbarriers; every wait is bounded and on expiry sets
// EFIM_DEV_TIMEOUT and lets all roles run out their (fixed) loop counts.
#include "prefill_tc.cuh"
#include "mbar.cuh"
#include <vector>
#include <algorithm>
#include <functional>
#include <atomic>

namespace efim {
namespace pf {

// ------------------------------------------------------------------ PTX wrappers
// Bounded wait (limit p.wait_ns): on expiry the CTA-wide abort flag goes up, after which
// every wait returns at once, and the timeout is recorded in the status word.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          unsigned long long limit_ns) {
  mbar_wait_bounded(bar, parity, limit_ns, abort_flag, status);
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// same with the A operand (P, bf16) read from tensor memory
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n" ::"r"(d_tmem),
      "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// One (page, kv head) of a pool: coordinates (dim % 64, slot % 8, dim / 64, slot / 8, page * Hkv + head);
// the first four are always 0 here (the box covers them whole).
__device__ __forceinline__ void tma_load_page(uint32_t dst, const CUtensorMap* map, uint32_t bar, int page_head) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %3, %3, %3, %4}], "
      "[%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(0), "r"(page_head)
      : "memory");
}

#define EFIM_TMEM_LD32(taddr, r)                                                                                  \
  asm volatile(                                                                                                   \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,"  \
      "%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"                                         \
      : "=r"((r)[0]), "=r"((r)[1]), "=r"((r)[2]), "=r"((r)[3]), "=r"((r)[4]), "=r"((r)[5]), "=r"((r)[6]),        \
        "=r"((r)[7]), "=r"((r)[8]), "=r"((r)[9]), "=r"((r)[10]), "=r"((r)[11]), "=r"((r)[12]), "=r"((r)[13]),    \
        "=r"((r)[14]), "=r"((r)[15]), "=r"((r)[16]), "=r"((r)[17]), "=r"((r)[18]), "=r"((r)[19]), "=r"((r)[20]), \
        "=r"((r)[21]), "=r"((r)[22]), "=r"((r)[23]), "=r"((r)[24]), "=r"((r)[25]), "=r"((r)[26]), "=r"((r)[27]), \
        "=r"((r)[28]), "=r"((r)[29]), "=r"((r)[30]), "=r"((r)[31])                                               \
      : "r"(taddr))

#define EFIM_TMEM_ST32(taddr, r)                                                                                  \
  asm volatile(                                                                                                   \
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17," \
      "%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),                              \
      "r"((r)[0]), "r"((r)[1]), "r"((r)[2]), "r"((r)[3]), "r"((r)[4]), "r"((r)[5]), "r"((r)[6]), "r"((r)[7]),    \
      "r"((r)[8]), "r"((r)[9]), "r"((r)[10]), "r"((r)[11]), "r"((r)[12]), "r"((r)[13]), "r"((r)[14]),            \
      "r"((r)[15]), "r"((r)[16]), "r"((r)[17]), "r"((r)[18]), "r"((r)[19]), "r"((r)[20]), "r"((r)[21]),          \
      "r"((r)[22]), "r"((r)[23]), "r"((r)[24]), "r"((r)[25]), "r"((r)[26]), "r"((r)[27]), "r"((r)[28]),          \
      "r"((r)[29]), "r"((r)[30]), "r"((r)[31])                                                                   \
      : "memory")

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// two-wide fp32 arithmetic (one issue slot for two lanes of work)
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor
// version 1.  Offsets are in bytes and stored without their 4 low bits.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  const uint32_t lo = ((addr >> 4) & 0x3FFFu) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
  const uint32_t hi = ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
  return (static_cast<uint64_t>(hi) << 32) | lo;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = n, A K-major, B K- or MN-major.
__host__ __device__ constexpr uint32_t instr_desc(int n, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(b_mn_major) << 16) |
         (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(BM >> 4) << 24);
}

// Shared-memory plan.  A query tile is [64-element half][128 rows][128 bytes]; a K or V tile
// is [8-key group][64-element half][8 keys][128 bytes], which is what one copy per page
// writes (a page is two key groups).  In both, 16-byte chunk c of row r is stored at chunk
// position c ^ (r & 7) (the 128B swizzle the tensor-map copies and the MMA descriptors use).
template <int D>
struct Smem {
  static constexpr int HALVES = D / 64;
  static constexpr int HALF_BYTES = 128 * 128;                  // 16 KB
  static constexpr int Q_BYTES = HALVES * HALF_BYTES;
  static constexpr int KV_BYTES = HALVES * HALF_BYTES;
  static constexpr int GROUP_BYTES = HALVES * 1024;             // 8 keys of a K/V tile, all dims
  static constexpr int PAGE_BYTES = 2 * GROUP_BYTES;            // one page = one copy
  static constexpr int Q_OFF = 0;
  static constexpr int KV_OFF = Q_OFF + NQ * Q_BYTES;
  static constexpr int BAR_OFF = KV_OFF + NSTAGE * KV_BYTES;
  static constexpr int TOTAL = BAR_OFF + 256 + 1024;            // + alignment slack
  // epilogue exchange between the two softmax groups (re-uses the K/V ring)
  static constexpr int XROW = D + 4;                            // floats per row, padded
  static_assert(BM * XROW * 4 <= NSTAGE * KV_BYTES, "exchange buffer must fit in the ring");
};
// barrier slots (8 bytes each) inside the BAR_OFF block
// (P has two barriers per stream: keys 0-63 and 64-127 of a tile are handed over separately)
enum {
  BAR_Q = 0, BAR_S = 2, BAR_P = 4, BAR_O = 8, BAR_PVI = 10, BAR_FULL = 12, BAR_EMPTY = 12 + NSTAGE_MAX,
  BAR_COUNT = 12 + 2 * NSTAGE_MAX
};

// Epilogue of the 32-row shape: the eight (max, sum, O) states of query row `lane`, left in
// shared memory as [state][row][XROW], are merged; this thread finishes D/8 dims of the row
// (slice `sidx`) and stores them (final output, or a chunk's partial).  Out of line: it runs
// once per CTA and its registers should not count against the loops of the caller.
template <int D>
__device__ __noinline__ void tiny_merge_store(uint16_t* out, float* lse, float* part_o, float* part_lse, int s_max,
                                              const float* xb, int lane, int sidx, bool valid, int chunk,
                                              size_t row_off, size_t th) {
  using L = Smem<D>;
  constexpr int DS = D / 8;
  float M = -INFINITY;
#pragma unroll
  for (int q = 0; q < 8; ++q) M = fmaxf(M, xb[(size_t)(q * 32 + lane) * L::XROW + D]);
  float Lt = 0.f, acc[DS];
#pragma unroll
  for (int d = 0; d < DS; ++d) acc[d] = 0.f;
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const float* row = xb + (size_t)(q * 32 + lane) * L::XROW;
    const float lq = row[D + 1];
    const float wq = lq > 0.f ? ex2(row[D] - M) : 0.f;
    Lt = fmaf(lq, wq, Lt);
#pragma unroll
    for (int d = 0; d < DS; d += 4) {
      const float4 x = *reinterpret_cast<const float4*>(row + sidx * DS + d);
      acc[d] = fmaf(x.x, wq, acc[d]);
      acc[d + 1] = fmaf(x.y, wq, acc[d + 1]);
      acc[d + 2] = fmaf(x.z, wq, acc[d + 2]);
      acc[d + 3] = fmaf(x.w, wq, acc[d + 3]);
    }
  }
  const float inv = Lt > 0.f ? 1.f / Lt : 0.f;
  const float lse2 = Lt > 0.f ? M + log2f(Lt) : -INFINITY;
  if (!valid) return;
  if (chunk < 0) {
    uint4* dst = reinterpret_cast<uint4*>(out + row_off + sidx * DS);
#pragma unroll
    for (int d = 0; d < DS; d += 8)
      dst[d / 8] = make_uint4(pack_bf16x2(acc[d] * inv, acc[d + 1] * inv), pack_bf16x2(acc[d + 2] * inv, acc[d + 3] * inv),
                              pack_bf16x2(acc[d + 4] * inv, acc[d + 5] * inv), pack_bf16x2(acc[d + 6] * inv, acc[d + 7] * inv));
    if (sidx == 0 && lse) lse[th] = lse2 * 0.6931471805599453f;
  } else {
    float4* dst = reinterpret_cast<float4*>(part_o + (th * s_max + chunk) * D + sidx * DS);
#pragma unroll
    for (int d = 0; d < DS; d += 4)
      dst[d / 4] = make_float4(acc[d] * inv, acc[d + 1] * inv, acc[d + 2] * inv, acc[d + 3] * inv);
    if (sidx == 0) part_lse[th * s_max + chunk] = lse2;
  }
}

// O row of every lane of the warp *= alpha (the rare rescale of the 32-row shape; kept out
// of line so that its 32 registers do not count against the loop that calls it).
template <int D>
__device__ __noinline__ void rescale_o_row(uint32_t o_addr, float alpha) {
#pragma unroll
  for (int c0 = 0; c0 < D; c0 += 32) {
    uint32_t o[32];
    EFIM_TMEM_LD32(o_addr + c0, o);
    tmem_wait_ld();
#pragma unroll
    for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
    EFIM_TMEM_ST32(o_addr + c0, o);
  }
}

// One query row -> its row of a shared-memory query tile (swizzled), zero for a row past the
// sequence; with a rotary table the row is rotated by its position on the way (the
// arithmetic of efim_kv_append).  `qrow` = tile base + 128 * tile row, `r` = tile row.
template <int D>
__device__ __forceinline__ void q_row_to_smem(const Params& p, uint8_t* qrow, int r, bool valid, int pos,
                                              size_t row_off) {
  using L = Smem<D>;
  const uint4* src = reinterpret_cast<const uint4*>(p.q + row_off);
  auto put = [&](int c, uint4 v) {
    *reinterpret_cast<uint4*>(qrow + (c >> 3) * L::HALF_BYTES + (((c & 7) ^ (r & 7)) << 4)) = v;
  };
  if (p.cos_sin == nullptr || !valid) {
#pragma unroll
    for (int c = 0; c < D / 8; ++c) {
      uint4 v = make_uint4(0, 0, 0, 0);
      if (valid) v = __ldg(src + c);
      put(c, v);
    }
  } else if (pos >= p.max_position) {
    if (p.status) atomicOr(p.status, EFIM_DEV_BAD_POSITION);
#pragma unroll
    for (int c = 0; c < D / 8; ++c) put(c, make_uint4(0, 0, 0, 0));
  } else {
    const float* cs = p.cos_sin + (size_t)pos * D;
    if (!p.interleaved) {
#pragma unroll
      for (int c = 0; c < D / 16; ++c) {
        uint4 a = __ldg(src + c), b = __ldg(src + c + D / 16);
        float cf[8], sf[8];
        *reinterpret_cast<float4*>(cf) = __ldg(reinterpret_cast<const float4*>(cs + c * 8));
        *reinterpret_cast<float4*>(cf + 4) = __ldg(reinterpret_cast<const float4*>(cs + c * 8 + 4));
        *reinterpret_cast<float4*>(sf) = __ldg(reinterpret_cast<const float4*>(cs + D / 2 + c * 8));
        *reinterpret_cast<float4*>(sf + 4) = __ldg(reinterpret_cast<const float4*>(cs + D / 2 + c * 8 + 4));
        rotate8(a, b, cf, sf);
        put(c, a);
        put(c + D / 16, b);
      }
    } else {
#pragma unroll
      for (int c = 0; c < D / 8; ++c) {
        uint4 a = __ldg(src + c);
        float cf[4], sf[4];
        *reinterpret_cast<float4*>(cf) = __ldg(reinterpret_cast<const float4*>(cs + c * 4));
        *reinterpret_cast<float4*>(sf) = __ldg(reinterpret_cast<const float4*>(cs + D / 2 + c * 4));
        rotate4_interleaved(a, cf, sf);
        put(c, a);
      }
    }
  }
}

// Two softmax groups ("streams") run per CTA.  With more than 128 rows, stream t
// owns query tile t and both walk every KV tile.  With 128 rows or fewer there is
// one query tile; stream 0 takes the even KV tiles and stream 1 the odd ones, each
// with its own running (max, sum, O), and the two states are merged at the end -
// the tensor core then still works on one stream while the other does its softmax.
//
// MODE 0: one query tile (33..128 rows); 1: two query tiles; 2: at most 32 rows (one-token rows of
// a mixed batch, short `inc`s): the one query tile holds the rows four times, once per 32-lane
// quarter, and the softmax warp of quarter w takes keys 32w..32w+31 of every tile with a
// running (max, sum, O) of its own - a quarter of the exponentials per thread and tile, so the
// two alternating streams turn a tile round in about half the time; the eight states of a row
// (2 streams x 4 quarters) are merged at the end through shared memory.
template <int D, int MODE>
__device__ __forceinline__ void prefill_tc_body(const Params& p, const CUtensorMap& map_k, const CUtensorMap& map_v,
                                                const WorkItem& it) {
  using L = Smem<D>;
  constexpr int HALVES = L::HALVES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bars = smem_base + L::BAR_OFF;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + L::BAR_OFF + BAR_COUNT * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + L::BAR_OFF + BAR_COUNT * 8 + 8);
  auto bar = [&](int i) { return bars + 8u * i; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.G;
  const int C = it.cached, N = it.new_len, tok0 = it.tok0;
  const int rows_total = N * G;
  const int rows_here = min(NQ * BM, rows_total - it.row0);
  constexpr bool dual = MODE == 1;                           // two query tiles (rows_here > BM)
  constexpr bool tiny = MODE == 2;                           // at most 32 rows, held four times
  const int i_last = (it.row0 + rows_here - 1) / G;          // last token of this CTA
  const int kv_cap = C + i_last + 1;                         // keys any row here may see
  const int nt = it.tile_end - it.tile_begin;
  const int cnt0 = dual ? nt : (nt + 1) >> 1;                // KV tiles of stream 0 / 1
  const int cnt1 = dual ? nt : nt >> 1;
  // K/V ring.  With one query tile the second tile's shared memory joins the ring
  // (6 entries instead of 5), and the loads are ordered the way the two streams consume
  // them - K0 K1 V0 K2 V1 K3 ... - so that no entry sits loaded but unused for a whole
  // period: such CTAs stream their K/V alone and live on the bytes they keep in flight.
  constexpr int nst = dual ? NSTAGE : NSTAGE_MAX;
  constexpr uint32_t ring_off = dual ? L::KV_OFF : L::KV_OFF - L::KV_BYTES;
  auto ld_k = [&](int n) { return dual ? 2 * n : (n == 0 ? 0 : 2 * n - 1); };          // ring load index of K(n)
  auto ld_v = [&](int n) { return dual ? 2 * n + 1 : min(2 * n + 2, 2 * nt - 1); };    // ... of V(n)

  if (tid == 0) {
    for (int t = 0; t < NQ; ++t) {
      mbar_init(bar(BAR_Q + t), BM);
      mbar_init(bar(BAR_S + t), 1);
      mbar_init(bar(BAR_P + 2 * t), BM);
      mbar_init(bar(BAR_P + 2 * t + 1), BM);
      mbar_init(bar(BAR_O + t), 1);
      mbar_init(bar(BAR_PVI + t), 1);
    }
    for (int s = 0; s < NSTAGE_MAX; ++s) {
      mbar_init(bar(BAR_FULL + s), 1);
      mbar_init(bar(BAR_EMPTY + s), 1);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(const_cast<uint32_t*>(tmem_slot))),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_S = tmem;                // S of stream t at columns [t*128, t*128+128); P (bf16) re-uses its first 64
  const uint32_t tmem_O = tmem + NQ * BN;      // O of stream t at columns [256 + t*D, ...)

  // Register split: every warp of a warpgroup runs the same setmaxnreg; the service
  // group releases first what the two softmax groups then take.
  if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_SERVICE));
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_SOFTMAX));
  }

  if (warp < 8 && tiny) {
    // ============================================================ softmax groups, 32-row shape
    const int st = warp >> 2, w = warp & 3;                 // stream, 32-lane quarter
    const int my_cnt = st == 0 ? cnt0 : cnt1;
    const int r = w * 32 + lane;                            // tile row == TMEM lane; the query row is `lane`
    const int R = it.row0 + lane;
    const bool valid = R < rows_total;
    const int i_tok = valid ? R / G : 0;
    const int g = valid ? R - i_tok * G : 0;
    const int vis = valid ? C + i_tok + 1 : kv_cap;
    const size_t row_off = ((size_t)(tok0 + i_tok) * p.Hq + (size_t)it.kvh * G + g) * D;
    if (st == 0) {
      q_row_to_smem<D>(p, smem_gen + L::Q_OFF + r * 128, r, valid, C + i_tok, row_off);
      fence_async_smem();
      mbar_arrive(bar(BAR_Q + 0));
    }
    const uint32_t lane_addr = (uint32_t)(w * 32) << 16;
    const uint32_t s_addr = tmem_S + lane_addr + st * BN;
    const uint32_t o_addr = tmem_O + lane_addr + st * D;
    float m_ref = -INFINITY, l_sum = 0.f;
    for (int k = 0; k < my_cnt; ++k) {
      mbar_wait(bar(BAR_S + st), k & 1, abort_flag, p.status, p.wait_ns);
      tc_fence_after();
      uint32_t s[32];
      EFIM_TMEM_LD32(s_addr + 32 * w, s);
      tmem_wait_ld();
      // P = bf16 pairs in columns 0..63 of this stream's S; this quarter's keys are columns
      // 16w..16w+15 of it, the rest of the row is zero.  The 32-column half without values goes first.
      uint32_t z[32];
#pragma unroll
      for (int c = 0; c < 32; ++c) z[c] = 0u;
      EFIM_TMEM_ST32(s_addr + (w < 2 ? 32 : 0), z);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar(BAR_P + 2 * st + (w < 2 ? 1 : 0)));
      const int kv0 = (it.tile_begin + 2 * k + st) * BN + 32 * w;
      if (__any_sync(0xffffffffu, kv0 + 32 > vis)) {
#pragma unroll
        for (int c = 0; c < 32; ++c)
          if (kv0 + c >= vis) s[c] = 0xff800000u;           // -inf
      }
      float mx4[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) mx4[a] = __uint_as_float(s[a]);
#pragma unroll
      for (int c = 4; c < 32; c += 4)
#pragma unroll
        for (int a = 0; a < 4; ++a) mx4[a] = fmaxf(mx4[a], __uint_as_float(s[c + a]));
      const float m_new = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
      // lazy rescale, as in the other shapes (O is quiet: S(k) ready means PV(k-1) has landed)
      const bool grow = m_new > m_ref + 8.f;
      if (k == 0) {
        m_ref = m_new;
      } else if (__any_sync(0xffffffffu, grow)) {
        const float alpha = grow ? ex2(m_ref - m_new) : 1.f;
        if (grow) m_ref = m_new;
        l_sum *= alpha;
        rescale_o_row<D>(o_addr, alpha);
      }
      const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
      float ls[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t v[16];
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const float p0 = ex2(fmaf(__uint_as_float(s[2 * e]), p.scale_log2, neg_m));
        const float p1 = ex2(fmaf(__uint_as_float(s[2 * e + 1]), p.scale_log2, neg_m));
        ls[e & 3] += p0 + p1;
        v[e] = pack_bf16x2(p0, p1);
      }
      uint32_t wv[32];
      if (w & 1) {
#pragma unroll
        for (int e = 0; e < 16; ++e) { wv[e] = 0u; wv[16 + e] = v[e]; }
      } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) { wv[e] = v[e]; wv[16 + e] = 0u; }
      }
      EFIM_TMEM_ST32(s_addr + (w < 2 ? 0 : 32), wv);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar(BAR_P + 2 * st + (w < 2 ? 0 : 1)));
      l_sum += (ls[0] + ls[1]) + (ls[2] + ls[3]);
    }
    // ---- epilogue: all MMAs of both streams done (the ring is quiet), then the eight states of
    // every row meet in the ring's shared memory
    mbar_wait(bar(BAR_O + 0), 0, abort_flag, p.status, p.wait_ns);
    if (cnt1 > 0) mbar_wait(bar(BAR_O + 1), 0, abort_flag, p.status, p.wait_ns);
    tc_fence_after();
    static_assert(8 * 32 * L::XROW * 4 <= NSTAGE_MAX * L::KV_BYTES, "the eight states must fit in the ring");
    float* xb = reinterpret_cast<float*>(smem_gen + ring_off);          // [8 states][32 rows][XROW]
    const int sidx = st * 4 + w;
    float* mine = xb + (size_t)(sidx * 32 + lane) * L::XROW;
    const bool have = my_cnt > 0 && l_sum > 0.f;
    if (lane < 32) {
      mine[D] = have ? m_ref : -INFINITY;
      mine[D + 1] = have ? l_sum : 0.f;
    }
#pragma unroll
    for (int c0 = 0; c0 < D; c0 += 32) {
      uint32_t o[32];
      if (my_cnt > 0) {                                                 // warp-uniform: the load is warp-wide
        EFIM_TMEM_LD32(o_addr + c0, o);
        tmem_wait_ld();
      }
#pragma unroll
      for (int c = 0; c < 32; c += 4)
        *reinterpret_cast<uint4*>(mine + c0 + c) =
            have ? make_uint4(o[c], o[c + 1], o[c + 2], o[c + 3]) : make_uint4(0, 0, 0, 0);
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    tiny_merge_store<D>(p.out, p.lse, p.part_o, p.part_lse, p.s_max, xb, lane, sidx, valid, it.chunk, row_off,
                        (size_t)(tok0 + i_tok) * p.Hq + (size_t)it.kvh * G + g);
    tc_fence_before();
  } else if (warp < 8) {
    // ============================================================ softmax groups
    const int st = warp >> 2;                               // stream
    const int my_cnt = st == 0 ? cnt0 : cnt1;
    const int qt = dual ? st : 0;                           // query tile of this stream
    const int r = (warp & 3) * 32 + lane;                   // tile row == TMEM lane
    const int R = it.row0 + qt * BM + r;                    // packed row of the (seq, kv head)
    const bool valid = R < rows_total;
    const int i_tok = valid ? R / G : 0;
    const int g = valid ? R - i_tok * G : 0;
    // keys this row sees; rows past the sequence are computed like the piece's last row and
    // dropped (with 0 here they would take the masking path on every tile and slow their group)
    const int vis = valid ? C + i_tok + 1 : kv_cap;
    const size_t row_off = ((size_t)(tok0 + i_tok) * p.Hq + (size_t)it.kvh * G + g) * D;
    if (dual || st == 0) {
      // ---- Q row -> shared memory (swizzled), zero for rows past the sequence.  With a
      // rotary table the row is rotated by its position C + i on the way (the arithmetic of
      // efim_kv_append, so the result equals a q that call rewrote in place).
      const uint4* src = reinterpret_cast<const uint4*>(p.q + row_off);
      uint8_t* qrow = smem_gen + L::Q_OFF + qt * L::Q_BYTES + r * 128;
      auto put = [&](int c, uint4 v) {
        *reinterpret_cast<uint4*>(qrow + (c >> 3) * L::HALF_BYTES + (((c & 7) ^ (r & 7)) << 4)) = v;
      };
      if (p.cos_sin == nullptr || !valid) {
#pragma unroll
        for (int c = 0; c < D / 8; ++c) {
          uint4 v = make_uint4(0, 0, 0, 0);
          if (valid) v = __ldg(src + c);
          put(c, v);
        }
      } else if (C + i_tok >= p.max_position) {
        // no table row for this position: report it, attend with a zero query (finite output)
        if (p.status) atomicOr(p.status, EFIM_DEV_BAD_POSITION);
#pragma unroll
        for (int c = 0; c < D / 8; ++c) put(c, make_uint4(0, 0, 0, 0));
      } else {
        const float* cs = p.cos_sin + (size_t)(C + i_tok) * D;       // cos[0..D/2) then sin[0..D/2)
        if (!p.interleaved) {
#pragma unroll
          for (int c = 0; c < D / 16; ++c) {
            uint4 a = __ldg(src + c), b = __ldg(src + c + D / 16);
            float cf[8], sf[8];
            *reinterpret_cast<float4*>(cf) = __ldg(reinterpret_cast<const float4*>(cs + c * 8));
            *reinterpret_cast<float4*>(cf + 4) = __ldg(reinterpret_cast<const float4*>(cs + c * 8 + 4));
            *reinterpret_cast<float4*>(sf) = __ldg(reinterpret_cast<const float4*>(cs + D / 2 + c * 8));
            *reinterpret_cast<float4*>(sf + 4) = __ldg(reinterpret_cast<const float4*>(cs + D / 2 + c * 8 + 4));
            rotate8(a, b, cf, sf);
            put(c, a);
            put(c + D / 16, b);
          }
        } else {
#pragma unroll
          for (int c = 0; c < D / 8; ++c) {
            uint4 a = __ldg(src + c);
            float cf[4], sf[4];
            *reinterpret_cast<float4*>(cf) = __ldg(reinterpret_cast<const float4*>(cs + c * 4));
            *reinterpret_cast<float4*>(sf) = __ldg(reinterpret_cast<const float4*>(cs + D / 2 + c * 4));
            rotate4_interleaved(a, cf, sf);
            put(c, a);
          }
        }
      }
      fence_async_smem();
      mbar_arrive(bar(BAR_Q + qt));
    }
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t s_addr = tmem_S + lane_addr + st * BN;
    const uint32_t o_addr = tmem_O + lane_addr + st * D;
    float m_ref = -INFINITY, l_sum = 0.f;
    for (int k = 0; k < my_cnt; ++k) {
      mbar_wait(bar(BAR_S + st), k & 1, abort_flag, p.status, p.wait_ns);
      tc_fence_after();
      uint32_t s[BN];
      EFIM_TMEM_LD32(s_addr + 0, s + 0);
      EFIM_TMEM_LD32(s_addr + 32, s + 32);
      EFIM_TMEM_LD32(s_addr + 64, s + 64);
      EFIM_TMEM_LD32(s_addr + 96, s + 96);
      tmem_wait_ld();
      const int kv0 = (it.tile_begin + (dual ? k : 2 * k + st)) * BN;
      if (__any_sync(0xffffffffu, kv0 + BN > vis)) {
#pragma unroll
        for (int c = 0; c < BN; ++c)
          if (kv0 + c >= vis) s[c] = 0xff800000u;           // -inf
      }
      float mx8[8];
#pragma unroll
      for (int a = 0; a < 8; ++a) mx8[a] = __uint_as_float(s[a]);
#pragma unroll
      for (int c = 8; c < BN; c += 8)
#pragma unroll
        for (int a = 0; a < 8; ++a) mx8[a] = fmaxf(mx8[a], __uint_as_float(s[c + a]));
      const float mx = fmaxf(fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3])),
                             fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));
      const float m_new = mx * p.scale_log2;
      // lazy rescale: keep the old reference maximum until it is off by more than 2^8.
      // O is quiet here: QK(k) was issued after PV(k-1) (barrier PVI) and the tensor pipe
      // completes in order, so S(k) being ready means PV(k-1) has landed.
      const bool grow = m_new > m_ref + 8.f;
      if (k == 0) {
        m_ref = m_new;
      } else if (__any_sync(0xffffffffu, grow)) {
        const float alpha = grow ? ex2(m_ref - m_new) : 1.f;
        if (grow) m_ref = m_new;
        l_sum *= alpha;
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 32) {
          uint32_t o[32];
          EFIM_TMEM_LD32(o_addr + c0, o);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
          EFIM_TMEM_ST32(o_addr + c0, o);
        }
      }
      const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
      // The scale-and-shift before the exponential and the row sum run two-wide with one query
      // tile (measured on two GPUs: cfg2 1-2.5 % faster, cfg3 0-3 %) and one at a time with two
      // tiles, where the two-wide form was 4-7 % slower (cfg4a, cfg4b).
      [[maybe_unused]] const uint64_t sc2 = pack2(p.scale_log2, p.scale_log2), nm2 = pack2(neg_m, neg_m);
      [[maybe_unused]] uint64_t ls2[4] = {0ull, 0ull, 0ull, 0ull};            // four pairs of partial sums
      [[maybe_unused]] float ls[4] = {0.f, 0.f, 0.f, 0.f};
      // P (bf16 pairs) goes back into the first 64 columns of this stream's S, in two
      // halves of 64 keys, so the PV MMAs of the first half are issued under the second
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint32_t w[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          float p0, p1;
          if constexpr (dual) {
            p0 = ex2(fmaf(__uint_as_float(s[h * 64 + 2 * e]), p.scale_log2, neg_m));
            p1 = ex2(fmaf(__uint_as_float(s[h * 64 + 2 * e + 1]), p.scale_log2, neg_m));
            ls[e & 3] += p0 + p1;
          } else {
            float x0, x1;
            unpack2(fma2(pack2(__uint_as_float(s[h * 64 + 2 * e]), __uint_as_float(s[h * 64 + 2 * e + 1])), sc2, nm2),
                    x0, x1);
            p0 = ex2(x0);
            p1 = ex2(x1);
            ls2[e & 3] = add2(ls2[e & 3], pack2(p0, p1));
          }
          w[e] = pack_bf16x2(p0, p1);
        }
        EFIM_TMEM_ST32(s_addr + h * 32, w);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(BAR_P + 2 * st + h));
      }
      if constexpr (dual) {
        l_sum += (ls[0] + ls[1]) + (ls[2] + ls[3]);
      } else {
        float lo, hi;
        unpack2(add2(add2(ls2[0], ls2[1]), add2(ls2[2], ls2[3])), lo, hi);
        l_sum += lo + hi;
      }
    }
    // ---- epilogue
    if (my_cnt > 0) {
      mbar_wait(bar(BAR_O + st), 0, abort_flag, p.status, p.wait_ns);
      if (!dual && cnt1 > 0) mbar_wait(bar(BAR_O + (st ^ 1)), 0, abort_flag, p.status, p.wait_ns);   // ring is quiet
      tc_fence_after();
    }
    float* xbuf = reinterpret_cast<float*>(smem_gen + L::KV_OFF) + r * L::XROW;
    const bool merge = !dual && cnt1 > 0;
    if (merge && st == 1) {
      // stream 1 hands its state to stream 0 through shared memory
      xbuf[D] = m_ref;
      xbuf[D + 1] = l_sum;
#pragma unroll
      for (int c0 = 0; c0 < D; c0 += 32) {
        uint32_t o[32];
        EFIM_TMEM_LD32(o_addr + c0, o);
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < 32; c += 4)
          *reinterpret_cast<uint4*>(xbuf + c0 + c) = make_uint4(o[c], o[c + 1], o[c + 2], o[c + 3]);
      }
    }
    if (merge) asm volatile("bar.sync 1, 256;" ::: "memory");
    if (my_cnt > 0 && (dual || st == 0)) {
      float w0 = 1.f, w1 = 0.f;
      if (merge) {
        const float m1 = xbuf[D], l1 = xbuf[D + 1];
        const float M = fmaxf(m_ref, m1);
        w0 = l_sum > 0.f ? ex2(m_ref - M) : 0.f;
        w1 = l1 > 0.f ? ex2(m1 - M) : 0.f;
        l_sum = l_sum * w0 + l1 * w1;
        m_ref = M;
      }
      const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
      const float lse2 = l_sum > 0.f ? m_ref + log2f(l_sum) : -INFINITY;
      const float a0 = w0 * inv, a1 = w1 * inv;
      const size_t th = (size_t)(tok0 + i_tok) * p.Hq + (size_t)it.kvh * G + g;
#pragma unroll
      for (int c0 = 0; c0 < D; c0 += 32) {
        uint32_t o[32];
        EFIM_TMEM_LD32(o_addr + c0, o);
        tmem_wait_ld();
        float f[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) f[c] = __uint_as_float(o[c]) * a0;
        if (merge) {
#pragma unroll
          for (int c = 0; c < 32; c += 4) {
            const float4 x = *reinterpret_cast<const float4*>(xbuf + c0 + c);
            f[c] = fmaf(x.x, a1, f[c]);
            f[c + 1] = fmaf(x.y, a1, f[c + 1]);
            f[c + 2] = fmaf(x.z, a1, f[c + 2]);
            f[c + 3] = fmaf(x.w, a1, f[c + 3]);
          }
        }
        if (valid) {
          if (it.chunk < 0) {
            uint4* dst = reinterpret_cast<uint4*>(p.out + row_off + c0);
#pragma unroll
            for (int c = 0; c < 4; ++c)
              dst[c] = make_uint4(pack_bf16x2(f[c * 8], f[c * 8 + 1]), pack_bf16x2(f[c * 8 + 2], f[c * 8 + 3]),
                                  pack_bf16x2(f[c * 8 + 4], f[c * 8 + 5]), pack_bf16x2(f[c * 8 + 6], f[c * 8 + 7]));
          } else {
            float4* dst = reinterpret_cast<float4*>(p.part_o + (th * p.s_max + it.chunk) * D + c0);
#pragma unroll
            for (int c = 0; c < 8; ++c) dst[c] = make_float4(f[4 * c], f[4 * c + 1], f[4 * c + 2], f[4 * c + 3]);
          }
        }
      }
      if (valid) {
        if (it.chunk < 0) {
          if (p.lse) p.lse[th] = lse2 * 0.6931471805599453f;
        } else {
          p.part_lse[th * p.s_max + it.chunk] = lse2;
        }
      }
    }
    tc_fence_before();
  } else if (warp == 8 || warp == 11) {
    // ============================================================ TMA producers
    // Every bulk-tensor copy costs its issuing warp ~65 cycles and a 128-key tile takes
    // 8 of them (one box per page: 16 slots x all dims of one kv head).  Warp 8 loads the
    // K tiles and warp 11 the V tiles.
    const int my_which = warp == 8 ? 0 : 1;
    const int32_t* bt = p.block_table + (size_t)it.seq * p.max_pages_per_seq;
    const int page_l = lane;
    const CUtensorMap* my_map = my_which == 0 ? &map_k : &map_v;
    // does this lane fetch a page of tile jj (lanes beyond the tile's visible pages do not)?
    auto wanted = [&](int jj) {
      if (jj >= nt) return false;
      const int tile = it.tile_begin + jj;
      const int keys = min(BN, kv_cap - tile * BN);
      const int npages = keys > 0 ? (keys + 15) >> 4 : 0;
      // (the last test only matters for a plan that does not belong to this block table)
      return page_l < npages && tile * 8 + page_l < p.max_pages_per_seq;
    };
    auto lookup = [&](int jj, bool want) { return want ? __ldg(bt + (it.tile_begin + jj) * 8 + page_l) : -1; };
    // the block-table read is a dependent global load in front of every copy: fetch it two tiles ahead
    bool want_a = wanted(0), want_b = wanted(1);
    int pid_a = lookup(0, want_a), pid_b = lookup(1, want_b);
    for (int jj = 0; jj < nt; ++jj) {
      const int pid = pid_a;
      const bool want = want_a;
      pid_a = pid_b;
      want_a = want_b;
      want_b = wanted(jj + 2);
      pid_b = lookup(jj + 2, want_b);
      const int ld = my_which == 0 ? ld_k(jj) : ld_v(jj);
      const bool ok = want && pid >= 0 && pid < p.num_pages;
      const bool bad = want && !ok;                          // an id outside the pool: reported, never dereferenced
      const uint32_t okmask = __ballot_sync(0xffffffffu, ok);
      const bool any_bad = __any_sync(0xffffffffu, bad);
      const uint32_t bytes = __popc(okmask) * (uint32_t)L::PAGE_BYTES;
      const int slot = ld % nst, use = ld / nst;
      mbar_wait(bar(BAR_EMPTY + slot), (use & 1) ^ 1, abort_flag, p.status, p.wait_ns);
      const uint32_t dst_off = ring_off + slot * L::KV_BYTES + page_l * L::PAGE_BYTES;
      if (any_bad) {
        // the page's 16 keys are replaced by zeros (score 0, value 0), so the tile holds nothing
        // undefined; written with ordinary stores, made visible to the tensor core's reads
        if (bad) {
          if (my_which == 0 && p.status) atomicOr(p.status, EFIM_DEV_BAD_PAGE);
          uint4* z = reinterpret_cast<uint4*>(smem_gen + dst_off);
          for (int i = 0; i < L::PAGE_BYTES / 16; ++i) z[i] = make_uint4(0, 0, 0, 0);
          fence_async_smem();
        }
        __syncwarp();
      }
      if (lane == 0) mbar_expect_tx(bar(BAR_FULL + slot), bytes);
      __syncwarp();
      if (ok) tma_load_page(smem_base + dst_off, my_map, bar(BAR_FULL + slot), pid * p.Hkv + it.kvh);
    }
    // if the CTA gave up, let copies that are still in flight land before shared memory goes away
    if (*abort_flag) {
      for (int jj = max(0, nt - nst); jj < nt; ++jj) {
        const int ld = my_which == 0 ? ld_k(jj) : ld_v(jj);
        const uint32_t b = bar(BAR_FULL + ld % nst), par = (ld / nst) & 1;
        mbar_drain(b, par);
      }
    }
  } else if (warp == 9 || warp == 10) {
    // ============================================================ MMA issuers
    // Issuing an MMA costs its thread about as long as the tensor core needs to run it,
    // so the work is split: warp 9 issues the PV MMAs of both streams, warp 10 the QK
    // MMAs.  QK(k+1) of a stream overwrites the columns P(k) is read from, so warp 10
    // issues it only after warp 9 has issued PV(k) (barrier PVI, tcgen05 fences on both
    // sides); the tensor core runs them in that order.
    const bool pv_role = warp == 9;
    constexpr uint32_t IDESC_QK = instr_desc(BN, 0);
    constexpr uint32_t IDESC_PV = instr_desc(D, 1);
    const uint32_t q_base = smem_base + L::Q_OFF, kv_base = smem_base + ring_off;
    mbar_wait(bar(BAR_Q + 0), 0, abort_flag, p.status, p.wait_ns);
    if (dual) mbar_wait(bar(BAR_Q + 1), 0, abort_flag, p.status, p.wait_ns);
    tc_fence_after();
    // Descriptors: the high word is fixed (SBO = distance between 8-row groups: 1024 in a
    // query tile, GROUP_BYTES in a K/V tile; version 1; 128B swizzle); the low word is
    // (address >> 4) | LBO << 16, so stepping through a tile is one add.
    constexpr uint32_t DESC_HI_Q = (1024u >> 4) | (1u << 14) | (2u << 29);
    constexpr uint32_t DESC_HI_KV = ((uint32_t)L::GROUP_BYTES >> 4) | (1u << 14) | (2u << 29);
    constexpr uint32_t LBO_K = 1u << 16;                                           // K-major: LBO unused
    constexpr uint32_t LBO_V = (1024u >> 4) << 16;                                 // MN-major: next 64 dims
    auto desc_q = [&](uint32_t lo) { return (static_cast<uint64_t>(DESC_HI_Q) << 32) | lo; };
    auto desc = [&](uint32_t lo) { return (static_cast<uint64_t>(DESC_HI_KV) << 32) | lo; };
    const uint32_t kv_lo = kv_base >> 4, q_lo = (q_base >> 4) | LBO_K;
    // O_st (+)= P_st V for half h (keys 64h..64h+63) of KV tile n (ring load 2n+1); P from TMEM
    auto issue_pv_half = [&](int st, int n, int h, uint32_t first) {
      const uint32_t v_lo = (kv_lo + (ld_v(n) % nst) * (L::KV_BYTES >> 4)) | LBO_V;
#pragma unroll
      for (int k = 4 * h; k < 4 * h + 4; ++k)
        umma_bf16_ts(tmem_O + st * D, tmem_S + st * BN + k * 8, desc(v_lo + k * (2 * L::GROUP_BYTES >> 4)), IDESC_PV,
                     (!first || k > 0) ? 1u : 0u);
    };
    auto issue_qk = [&](int st, int n) {
      const uint32_t k_lo = (kv_lo + (ld_k(n) % nst) * (L::KV_BYTES >> 4)) | LBO_K;
      const uint32_t a_lo = q_lo + (dual ? st : 0) * (L::Q_BYTES >> 4);
#pragma unroll
      for (int k = 0; k < D / 16; ++k) {
        const uint32_t off_q = ((k >> 2) * L::HALF_BYTES + (k & 3) * 32) >> 4;
        const uint32_t off_k = ((k >> 2) * 1024 + (k & 3) * 32) >> 4;
        umma_bf16(tmem_S + st * BN, desc_q(a_lo + off_q), desc(k_lo + off_k), IDESC_QK, k > 0 ? 1u : 0u);
      }
    };
    // V rows past the visible range hold stale or foreign data; P is 0 there but
    // 0 * NaN would poison O, so clear them before the tile is used.
    auto clear_v_tail = [&](int n) {
      const int keys = kv_cap - (it.tile_begin + n) * BN;
      if (keys < BN) {
        uint8_t* vb = smem_gen + ring_off + (ld_v(n) % nst) * L::KV_BYTES;
        const int first = max(keys, 0);
        const int chunks = (BN - first) * 8;                // 16-byte chunks to clear per 64-dim half
#pragma unroll
        for (int h = 0; h < HALVES; ++h)
          for (int idx = lane; idx < chunks; idx += 32) {
            const int key = first + (idx >> 3);
            *reinterpret_cast<uint4*>(vb + (key >> 3) * L::GROUP_BYTES + h * 1024 + (key & 7) * 128 + ((idx & 7) << 4)) =
                make_uint4(0, 0, 0, 0);
          }
        fence_async_smem();
        __syncwarp();
      }
    };
    for (int k = 0; k <= cnt0; ++k) {
#pragma unroll
      for (int st = 0; st < 2; ++st) {
        const int my_cnt = st == 0 ? cnt0 : cnt1;
        if (my_cnt == 0 || k > my_cnt) continue;
        const bool last_user = !dual || st == 1;            // last stream to touch this K/V tile
        if (k > 0 && pv_role) {
          const int n = dual ? k - 1 : 2 * (k - 1) + st;
          const int lv = ld_v(n);
          mbar_wait(bar(BAR_FULL + lv % nst), (lv / nst) & 1, abort_flag, p.status, p.wait_ns);
          if (!dual || st == 0) clear_v_tail(n);
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            mbar_wait(bar(BAR_P + 2 * st + h), (k - 1) & 1, abort_flag, p.status, p.wait_ns);
            tc_fence_after();
            if (lane == 0) issue_pv_half(st, n, h, k == 1);
          }
          if (lane == 0) {
            if (last_user) tc_commit(bar(BAR_EMPTY + lv % nst));
            if (k == my_cnt) tc_commit(bar(BAR_O + st));
            tc_fence_before();
            mbar_arrive(bar(BAR_PVI + st));                   // PV(k-1) is issued: S/P columns may be rewritten
          }
          __syncwarp();
        }
        if (k < my_cnt && !pv_role) {
          const int n = dual ? k : 2 * k + st;
          const int lk = ld_k(n);
          mbar_wait(bar(BAR_FULL + lk % nst), (lk / nst) & 1, abort_flag, p.status, p.wait_ns);
          if (k > 0) mbar_wait(bar(BAR_PVI + st), (k - 1) & 1, abort_flag, p.status, p.wait_ns);
          tc_fence_after();
          if (lane == 0) {
            issue_qk(st, n);
            tc_commit(bar(BAR_S + st));
            if (last_user) tc_commit(bar(BAR_EMPTY + lk % nst));
          }
          __syncwarp();
        }
      }
    }
    tc_fence_before();
  }
  __syncthreads();
  if (*abort_flag) {
    // a wait expired: roles ran out of step, copies and MMAs may still be in flight; give
    // them a generous moment to finish before TMEM and shared memory are released
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 9) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

template <int D>
__global__ void __launch_bounds__(THREADS, 1)
prefill_tc_kernel(const Params p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
  WorkItem it;                                                // 32 bytes: two vector loads, no dependent load after them
  {
    const uint4* src = reinterpret_cast<const uint4*>(p.items + blockIdx.x);
    uint4* dst = reinterpret_cast<uint4*>(&it);
    dst[0] = __ldg(src);
    dst[1] = __ldg(src + 1);
  }
  const int rows_here = it.new_len * p.G - it.row0;
  // the three shapes of a CTA are separate instantiations: ring size, load order and the
  // query-tile choice are compile-time constants in the issuing warps' inner loops
  if (rows_here > BM)
    prefill_tc_body<D, 1>(p, map_k, map_v, it);
  else if (rows_here <= 32)
    prefill_tc_body<D, 2>(p, map_k, map_v, it);
  else
    prefill_tc_body<D, 0>(p, map_k, map_v, it);
}

// Merge the KV-chunk partials of split sequences: one warp per (token, head).
template <int D>
__global__ void __launch_bounds__(128) prefill_merge_kernel(const Params p) {
  constexpr int EPL = D / 32;
  const int lane = threadIdx.x & 31;
  const size_t th = (size_t)blockIdx.x * 4 + (threadIdx.x >> 5);
  if (th >= (size_t)p.total_new_tokens * p.Hq) return;
  const int t = (int)(th / p.Hq);
  int lo = 0, hi = p.batch;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (__ldg(p.q_indptr + mid) <= t) lo = mid; else hi = mid;
  }
  const int st = __ldg(p.split_tokens + lo);
  if (st == 0) return;                                      // written directly by the main kernel
  const int vis = __ldg(p.cached_len + lo) + (t - __ldg(p.q_indptr + lo)) + 1;
  const int nc = min(p.s_max, (vis + st - 1) / st);
  const float* pl = p.part_lse + th * p.s_max;
  const float* po = p.part_o + th * p.s_max * D + lane * EPL;
  float M = -INFINITY;
  for (int c = 0; c < nc; ++c) M = fmaxf(M, pl[c]);
  float Lsum = 0.f, acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  for (int c = 0; c < nc; ++c) {
    const float w = exp2f(pl[c] - M);
    Lsum += w;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = fmaf(w, po[(size_t)c * D + e], acc[e]);
  }
  const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
  uint16_t* out = p.out + th * D + lane * EPL;
#pragma unroll
  for (int e = 0; e < EPL; ++e) out[e] = __bfloat16_as_ushort(__float2bfloat16_rn(acc[e] * inv));
  if (p.lse && lane == 0) p.lse[th] = (M + log2f(Lsum)) * 0.6931471805599453f;
}

// ------------------------------------------------------------------ host side
namespace {
// Relative cost of a CTA in tenths of a microsecond, as measured on B200: a 128-key tile
// with two query tiles is bound by the softmax / tensor pipeline, with one by its K/V
// bytes; every CTA pays for its set-up, query load, pipeline fill and epilogue; a split
// adds the partials' round trip and the merge launch.
constexpr long long COST_TILE_DUAL = 21, COST_TILE_SINGLE = 15, COST_CTA = 100, COST_PARTIAL = 8, COST_MERGE = 80;
constexpr long long COST_TILE_SINGLE_TAIL = 9;     // a one-tile CTA's tile when the GPU is no longer full

// Finish time of the launch if the K/V range of every sequence is cut into chunks of
// `chunk_tiles` tiles: the hardware hands CTAs, longest first, to whichever SM is free.
long long estimate_makespan(const efim_cache_desc* c, const efim_batch_desc* b, long long chunk_tiles, int n_sm) {
  const int G = c->num_q_heads / c->num_kv_heads;
  std::vector<long long> cost;
  bool split = false;
  for (int s = 0; s < b->batch; ++s) {
    const long long N = b->h_new_len[s], C = b->h_cached_len[s];
    if (N <= 0) continue;
    const long long rows = N * G;
    const long long kt_max = (C + N + BN - 1) / BN;
    long long S = std::max<long long>(1, std::min<long long>(16, (kt_max + chunk_tiles - 1) / chunk_tiles));
    const long long ct = (kt_max + S - 1) / S;
    S = (kt_max + ct - 1) / ct;
    split |= S > 1;
    for (long long row0 = 0; row0 < rows; row0 += NQ * BM) {
      const long long rows_here = std::min<long long>(rows - row0, NQ * BM);
      const long long kt = (C + (row0 + rows_here - 1) / G + 1 + BN - 1) / BN;
      const long long tc = rows_here > BM ? COST_TILE_DUAL : COST_TILE_SINGLE;
      for (long long tb = 0; tb < kt; tb += ct)
        cost.insert(cost.end(), (size_t)c->num_kv_heads,
                    COST_CTA + std::min(ct, kt - tb) * tc + (S > 1 ? COST_PARTIAL : 0));
    }
  }
  std::sort(cost.begin(), cost.end(), std::greater<long long>());
  std::vector<long long> sm((size_t)n_sm, 0);                // min-heap of SM finish times
  auto later = std::greater<long long>();
  for (long long x : cost) {
    std::pop_heap(sm.begin(), sm.end(), later);
    sm.back() += x;
    std::push_heap(sm.begin(), sm.end(), later);
  }
  return *std::max_element(sm.begin(), sm.end()) + (split ? COST_MERGE : 0);
}
}  // namespace

Plan make_plan(const efim_cache_desc* c, const efim_batch_desc* b, WorkItem* items, int32_t* split_tokens) {
  const int G = c->num_q_heads / c->num_kv_heads;
  const int Hkv = c->num_kv_heads;
  // pass 1: count unsplit items and KV tiles
  long long n_unsplit = 0, tiles_total = 0;
  for (int s = 0; s < b->batch; ++s) {
    const long long N = b->h_new_len[s], C = b->h_cached_len[s];
    if (N <= 0) continue;
    const long long rows = N * G;
    for (long long row0 = 0; row0 < rows; row0 += NQ * BM) {
      const long long i_last = (std::min(rows, row0 + NQ * BM) - 1) / G;
      const long long kt = (C + i_last + 1 + BN - 1) / BN;
      n_unsplit += Hkv;
      tiles_total += kt * Hkv;
    }
  }
  // Few long items cannot fill the SMs, or leave a ragged last wave: try cutting the K/V
  // range of every sequence into chunks that give about 1, 2, 3 or 4 CTAs per SM (each at
  // least 4 tiles long) and keep the cut, or none, with the earliest estimated finish.
  const int n_sm = sm_count();
  long long chunk_tiles = 1LL << 40;
  if (n_unsplit < 4LL * n_sm && tiles_total > 0) {
    long long best = estimate_makespan(c, b, chunk_tiles, n_sm);
    for (int k = 1; k <= 4; ++k) {
      const long long ct = std::max<long long>(4, (tiles_total + (long long)n_sm * k - 1) / ((long long)n_sm * k));
      const long long t = estimate_makespan(c, b, ct, n_sm);
      if (t < best) { best = t; chunk_tiles = ct; }
    }
  }
  Plan pl{};
  int s_max = 1;
  long long n_items = 0, tok0 = 0;
  for (int s = 0; s < b->batch; tok0 += b->h_new_len[s], ++s) {
    const long long N = b->h_new_len[s], C = b->h_cached_len[s];
    if (split_tokens) split_tokens[s] = 0;
    if (N <= 0) continue;
    const long long rows = N * G;
    const long long kt_max = (C + N + BN - 1) / BN;
    long long S = std::min<long long>(16, (kt_max + chunk_tiles - 1) / chunk_tiles);
    if (S < 1) S = 1;
    const long long ct = (kt_max + S - 1) / S;               // tiles per chunk
    S = (kt_max + ct - 1) / ct;
    if (S > 1 && split_tokens) split_tokens[s] = (int32_t)(ct * BN);
    s_max = std::max<int>(s_max, (int)S);
    for (long long row0 = 0; row0 < rows; row0 += NQ * BM) {
      const long long i_last = (std::min(rows, row0 + NQ * BM) - 1) / G;
      const long long kt = (C + i_last + 1 + BN - 1) / BN;
      for (long long ch = 0; ch < S; ++ch) {
        const long long tb = ch * ct, te = std::min(kt, (ch + 1) * ct);
        if (tb >= te) continue;
        for (int h = 0; h < Hkv; ++h) {
          if (items) {
            WorkItem w{};
            w.seq = s; w.kvh = (int16_t)h; w.row0 = (int)row0; w.tile_begin = (int)tb; w.tile_end = (int)te;
            w.chunk = (int16_t)(S > 1 ? (int)ch : -1);
            w.cached = (int32_t)C; w.new_len = (int32_t)N; w.tok0 = (int32_t)tok0;
            items[n_items] = w;
          }
          ++n_items;
        }
      }
    }
  }
  if (items) {
    if (n_items > 8LL * n_sm) {
      // Many waves: CTAs that run together should read the same K/V.  Keep the row tiles
      // of one (sequence, kv head) adjacent (longest first inside the group), so the
      // concurrent working set is a few heads' K/V and stays in L2.
      std::stable_sort(items, items + n_items, [](const WorkItem& a, const WorkItem& b2) {
        if (a.seq != b2.seq) return a.seq < b2.seq;
        if (a.kvh != b2.kvh) return a.kvh < b2.kvh;
        return a.row0 > b2.row0;
      });
    } else {
      // Few waves: costliest first, so the tail of the launch is made of cheap items.  A tile
      // costs a two-tile CTA (bound by its softmax) 2.1 us wherever it runs; a one-tile CTA is
      // bound by its K/V bytes and speeds up once SMs fall idle at the end of the launch (measured:
      // 0.89 us per tile with 8 to 32 such CTAs on the GPU, 1.5 us with 148), so it is weighted
      // 0.9 us here (cfg2: 0.305 ms ordered by tile count, 0.290 by cost at 2.1 : 1.5, 0.281 at
      // 2.1 : 1.2; 2.1 : 0.9 is 3-5 % faster still on three of four other draws of cfg2).
      auto cost = [G](const WorkItem& w) {
        const long long rows_here = std::min<long long>((long long)w.new_len * G - w.row0, NQ * BM);
        return (long long)(w.tile_end - w.tile_begin) * (rows_here > BM ? COST_TILE_DUAL : COST_TILE_SINGLE_TAIL);
      };
      std::stable_sort(items, items + n_items,
                       [&](const WorkItem& a, const WorkItem& b2) { return cost(a) > cost(b2); });
    }
  }
  pl.n_items = (int)n_items;
  pl.s_max = s_max;
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  pl.items_bytes = up((size_t)n_items * sizeof(WorkItem));
  pl.split_bytes = up((size_t)b->batch * sizeof(int32_t));
  const size_t th = (size_t)b->total_new_tokens * c->num_q_heads;
  pl.part_lse_bytes = s_max > 1 ? up(th * s_max * sizeof(float)) : 0;
  pl.part_o_bytes = s_max > 1 ? up(th * s_max * c->head_dim * sizeof(float)) : 0;
  return pl;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// Pool [pages][Hkv][16][D] bf16 as a 5-D tensor (dim % 64, slot % 8, dim / 64, slot / 8,
// page * Hkv + head); one box = the 16 slots x D dims of one (page, head), written to shared
// memory as [slot / 8][dim / 64][slot % 8][64 dims], 128-byte swizzled.
static bool make_pool_map(CUtensorMap* m, void* pool, int pages, int Hkv, int D) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t row = (cuuint64_t)D * 2;
  const cuuint64_t dims[5] = {64, 8, (cuuint64_t)D / 64, 2, (cuuint64_t)pages * Hkv};
  const cuuint64_t strides[4] = {row, 128, 8 * row, 16 * row};
  const cuuint32_t box[5] = {64, 8, (cuuint32_t)D / 64, 2, 1};
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, pool, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A model calls this once per layer with the same few pools over and over: the encoded maps
// of the pools seen last are kept per host thread (a map is a pure function of the key).
struct PoolMapEntry {
  void* pool;
  int pages, Hkv, D;
  CUtensorMap map;
};
static const CUtensorMap* pool_map(void* pool, int pages, int Hkv, int D) {
  constexpr int kEntries = 16;
  thread_local PoolMapEntry cache[kEntries] = {};
  thread_local int next = 0;
  for (int i = 0; i < kEntries; ++i)
    if (cache[i].pool == pool && cache[i].pages == pages && cache[i].Hkv == Hkv && cache[i].D == D)
      return &cache[i].map;
  PoolMapEntry& e = cache[next];
  next = (next + 1) % kEntries;
  e.pool = nullptr;
  if (!make_pool_map(&e.map, pool, pages, Hkv, D)) return nullptr;
  e.pool = pool;
  e.pages = pages;
  e.Hkv = Hkv;
  e.D = D;
  return &e.map;
}

// The kernel's shared-memory size has to be raised once per device.
template <int D>
static efim_status raise_smem_limit() {
  constexpr int kMaxDevices = 64;
  static std::atomic<bool> done[kMaxDevices];
  int dev = 0;
  EFIM_CUDA_TRY(cudaGetDevice(&dev));
  if (dev >= 0 && dev < kMaxDevices && done[dev].load(std::memory_order_acquire)) return EFIM_OK;
  EFIM_CUDA_TRY(cudaFuncSetAttribute(prefill_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     Smem<D>::TOTAL));
  if (dev >= 0 && dev < kMaxDevices) done[dev].store(true, std::memory_order_release);
  return EFIM_OK;
}

template <int D>
static efim_status launch_d(const efim_cache_desc* c, const Params& p, const Plan& pl, cudaStream_t s) {
  const CUtensorMap* pk = pool_map(c->d_k_pool, c->num_pages, c->num_kv_heads, D);
  const CUtensorMap* pv = pool_map(c->d_v_pool, c->num_pages, c->num_kv_heads, D);
  if (!pk || !pv) return EFIM_ERR_CUDA;
  const CUtensorMap mk = *pk, mv = *pv;
  const efim_status st = raise_smem_limit<D>();
  if (st != EFIM_OK) return st;
  prefill_tc_kernel<D><<<pl.n_items, THREADS, Smem<D>::TOTAL, s>>>(p, mk, mv);
  EFIM_CUDA_TRY(cudaGetLastError());
  if (pl.s_max > 1) {
    const unsigned blocks = (unsigned)(((size_t)p.total_new_tokens * p.Hq + 3) / 4);
    prefill_merge_kernel<D><<<blocks, 128, 0, s>>>(p);
    EFIM_CUDA_TRY(cudaGetLastError());
  }
  return EFIM_OK;
}

efim_status launch(const efim_cache_desc* c, const Params& p, const Plan& pl, cudaStream_t s) {
  if (pl.n_items == 0) return EFIM_OK;
  return c->head_dim == 128 ? launch_d<128>(c, p, pl, s) : launch_d<64>(c, p, pl, s);
}

}  // namespace pf
}  // namespace efim
