// KV cache in the 8-bit floating-point format e4m3 with one float scale per (page, kv head): append (quantise)
// and split-KV attention (prefix levels and suffix chunks) over the quantised pools.
//
// Cache layout: k_pool, v_pool [page][kv head][16 tokens][128] bytes (one (page, kv head) slab = 2 KB),
// k_scale, v_scale [page][kv head] float; a code stands for decode(code) * scale.  Queries and outputs stay bf16.
//
// Attention kernel: one warp per (candidate, kv head, part) as in the bf16 suffix kernel - a private ring of
// page stages filled by TMA (one 4 KB box per page: its K slab and its V slab, 128-byte swizzle), fragments by
// ldmatrix, warp-level MMAs, lazily refreshed running maximum - with the codes widened in registers:
//   * e4m3 -> f16 is exact (cvt.rn.f16x2.e4m3x2, two values an instruction), so the products are f16 x f16 with
//     f32 accumulation; the queries are converted bf16 -> f16 once per item (exact inside f16's range);
//   * an ldmatrix "16-bit element" is two codes of neighbouring head-dim positions.  For S = K Q^T the contraction
//     may visit d in any order, so the k-slots of an MMA are dealt as they come (slots 2t, 2t+1, 2t+8, 2t+9 of a
//     16-wide step hold d = 4t .. 4t+3) and the query fragment follows the same order.  For O^T += V^T P^T the
//     transposing ldmatrix delivers, per lane, codes of two tokens x two d positions; one byte permute sorts them
//     into (d, token pair) and (d + 1, token pair), which makes rows r and r + 8 of the MMA's output tile the head-dim
//     positions 2r and 2r + 1: the epilogue stores them as pairs;
//   * the K scale multiplies the scores of its page (with the softmax scale), the V scale the probabilities that
//     go into the second product (the row sum takes the unscaled ones).
// The prefix levels run on the same kernel, every candidate streaming its group's pages (from L2 after the first).
#include <cstdlib>

#include <cuda_fp16.h>

#include "mc_internal.cuh"

namespace mc {
namespace {

constexpr int D = 128;
constexpr int kW = 2;                      // warps (items) per CTA
constexpr int kStages = 4;                 // page stages per warp: two being computed, two in flight (32 KB a CTA, six CTAs
                                           // = twelve warps per SM; measured against 6 and 8 stages with 4 and 3 CTAs:
                                           // cfg4 suffix pass 951 : 968 : 962 us, whole step 1003 : 1018 : 1095 us)
constexpr uint32_t kSlabBytes = kPage * D;           // one (page, kv head) slab of K or of V: 2 KB
constexpr uint32_t kStageBytes = 2 * kSlabBytes;
constexpr long long kDrainCycles = 2000000ll;        // ~1 ms: what a warp that gives up grants its copies in flight

struct __align__(1024) Smem {
  uint8_t ring[kW][kStages][kStageBytes];   // [warp][stage][K slab | V slab], each slab [16 tokens][128 B], swizzled
  uint64_t full[kW][kStages];
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// The same test without suspension: returns at once.
__device__ __forceinline__ bool mbar_test_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false once `limit` cycles have passed (MC_ERR_TIMEOUT is latched).  A limit shorter than the
// time the hardware may keep a thread suspended inside try_wait is honoured by polling without suspension.
__device__ __forceinline__ bool mbar_wait(const Params &p, uint64_t *bar, uint32_t parity, long long limit) {
  const bool polled = limit < 2000000ll;
  if (polled ? mbar_test_wait(bar, parity) : mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (polled ? mbar_test_wait(bar, parity) : mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > limit) {
      latch(p, kDevTimeout);
      return false;
    }
  }
}
// Private suffix pages are read once per step (evict-first); a group's prefix pages are read by every candidate of
// the group and again at the next step (evict-last).
template <int MODE>
__device__ __forceinline__ uint64_t l2_policy() {
  uint64_t pol;
  if (MODE == kSuffix) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(pol));
  else asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;\n" : "=l"(pol));
  return pol;
}
// The K slab and the V slab of one (page, kv head), 4 KB, as one box: lands as [pool][16 tokens][128 bytes] with the
// 128-byte swizzle.  `slab` = page * Hkv + kv head.
__device__ __forceinline__ void tma_load_stage(uint32_t dst, const CUtensorMap *map, int slab, uint64_t *bar,
                                               uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%2, %3, %4, %5}], [%6], %7;\n"
      ::"r"(dst), "l"(map), "r"(0), "r"(0), "r"(slab), "r"(0), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma16816_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t transpose8x8(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
  return y;
}
// four e4m3 codes (bytes 0..3 of x) -> f16 pairs (bytes 0, 1) and (bytes 2, 3); exact
__device__ __forceinline__ void widen4(uint32_t x, uint32_t &lo, uint32_t &hi) {
  asm("{\n\t.reg .b16 l, h;\n\t"
      "mov.b32 {l, h}, %2;\n\t"
      "cvt.rn.f16x2.e4m3x2 %0, l;\n\t"
      "cvt.rn.f16x2.e4m3x2 %1, h;\n\t}\n"
      : "=r"(lo), "=r"(hi) : "r"(x));
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;\n" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
// two bf16 (one 32-bit word, low element first) -> f16 pair; values beyond f16's range saturate to its largest
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w) {
  const float lo = __uint_as_float(w << 16), hi = __uint_as_float(w & 0xffff0000u);
  return pack_f16x2(fminf(fmaxf(lo, -65504.f), 65504.f), fminf(fmaxf(hi, -65504.f), 65504.f));
}

template <int MODE>
__device__ __forceinline__ void
attn_fp8_body(const Params &p, const CUtensorMap &kv_map, uint32_t k_off, uint32_t v_off,
              const __nv_bfloat16 *__restrict__ q, float sl2, float *__restrict__ o_part,
              float *__restrict__ lse_part, long long wait_cycles) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  Smem &sm = *reinterpret_cast<Smem *>(smem_raw);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gid = lane >> 2, tig = lane & 3;
  if ((smem_u32(smem_raw) & 1023u) != 0) {   // the swizzle pattern assumes 1024-byte aligned slabs
    if (threadIdx.x == 0) latch(p, MC_ERR_CUDA);
    return;
  }
  if (lane == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(&sm.full[warp][s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncthreads();
  // (a kernel launched behind this one as its programmatic dependent - the merge, which waits for this grid's
  // completion before it reads anything - may take its place on the SMs once every CTA of this grid has started)
  if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");

  const int nparts_mode = MODE == kPrefix ? p.n_prefix_parts : p.n_parts - p.suffix_part_base;
  const long long n_items = (long long)p.B * p.Hkv * nparts_mode;
  const long long cta = MODE == kSuffix && p.suffix_order ? __ldg(p.suffix_order + blockIdx.x) : blockIdx.x;
  const long long item = cta * kW + warp;
  if (item >= n_items) return;
  int b, h, part;
  if (MODE == kSuffix) {   // kv heads of one page are adjacent in the pool: neighbouring warps stream neighbouring slabs
    h = (int)(item % p.Hkv);
    part = (int)((item / p.Hkv) % nparts_mode);
    b = (int)(item / ((long long)p.Hkv * nparts_mode));
  } else {                 // candidates of a group walk the same pages at the same time
    b = (int)(item % p.B);
    h = (int)((item / p.B) % p.Hkv);
    part = (int)(item / ((long long)p.B * p.Hkv));
  }
  const Span sp = resolve_span<MODE>(p, b, part);
  const int g = p.g;
  const size_t row0 = (size_t)b * p.Hq + (size_t)h * g;
  if (sp.lo >= sp.hi) {
    if (lane < g) lse_part[(row0 + lane) * p.n_parts + sp.part] = -INFINITY;
    return;
  }
  const int n_pages = ((sp.hi + 15) >> 4) - (sp.lo >> 4);    // >= 1
  const int n_ord = (n_pages + 1) & ~1;                      // an odd count is padded with a masked repeat of the last page
  const int32_t *row_pages = sp.pages + (sp.lo >> 4);
  const float *k_scale = p.k_scale, *v_scale = p.v_scale;
  // Page ids, their validity and their two scales are read 32 pages at a time (lane = page ordinal in the block), a
  // block ahead of their use: block k's registers take block k + 2 once block k is consumed - first the ids, four
  // iterations later (the load has returned by then) their validity and the two scales they lead to.  A page with an
  // id outside the pool is loaded from page 0 and masked.
  int ids0 = 0, ids1 = 0;          // blocks with an even / odd index (registers, selected by the block's parity)
  float sk0 = 0.f, sk1 = 0.f, sv0 = 0.f, sv1 = 0.f;
  uint32_t good0 = 0u, good1 = 0u;
  auto load_ids = [&](int blk) {
    const int o = blk * 32 + lane;
    const int id = o < n_pages ? __ldg(row_pages + o) : 0;
    if (blk & 1) ids1 = id; else ids0 = id;
  };
  auto finish_block = [&](int blk) {
    const int o = blk * 32 + lane;
    int id = blk & 1 ? ids1 : ids0;
    const bool ok = o >= n_pages || (unsigned)id < (unsigned)p.num_pages;
    if (!ok) {
      latch(p, kDevBadPage);
      id = 0;
    }
    const uint32_t gm = __ballot_sync(0xffffffffu, ok);
    const size_t slab = (size_t)id * p.Hkv + h;
    const float a = o < n_pages ? __ldg(k_scale + slab) : 0.f, c = o < n_pages ? __ldg(v_scale + slab) : 0.f;
    if (blk & 1) { ids1 = id; good1 = gm; sk1 = a; sv1 = c; } else { ids0 = id; good0 = gm; sk0 = a; sv0 = c; }
  };
  load_ids(0);
  load_ids(1);
  finish_block(0);
  finish_block(1);
  // B operand of the first product: Q^T as f16, column n = head gid; k-step c covers d in [16 c, 16 c + 16) in the
  // order the K fragments deliver it: slots 2t, 2t+1 <- d = 16c + 4t, +1; slots 2t+8, 2t+9 <- d = 16c + 4t + 2, +3
  uint32_t qf[8][2];
  {
    const uint2 *qrow = reinterpret_cast<const uint2 *>(q + ((size_t)b * p.Hq + (size_t)h * g + gid) * D);
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      uint2 w = make_uint2(0u, 0u);
      if (gid < g) w = __ldg(qrow + 4 * c + tig);
      qf[c][0] = bf16x2_to_f16x2(w.x);
      qf[c][1] = bf16x2_to_f16x2(w.y);
    }
  }

  const uint64_t pol = l2_policy<MODE>();
  uint8_t(*ring)[kStageBytes] = sm.ring[warp];
  uint64_t *full = sm.full[warp];
  // Pages o and o + 1 (o even), each issued by the lane that holds its id.  The pad page repeats the last page.
  auto issue_pair = [&](int o) {
    if ((lane & 30) != (o & 30)) return;
    int id = (o >> 5) & 1 ? ids1 : ids0;                                      // o is even: o and o + 1 share a block
    const int id_even = __shfl_sync(0x3u << (lane & 30), id, lane & 30);
    o += lane & 1;
    if (o >= n_pages) id = id_even;                                           // (n_pages is odd then: o - 1 is the last page)
    const int s = o % kStages;
    mbar_expect_tx(&full[s], kStageBytes);
    tma_load_stage(smem_u32(ring[s]), &kv_map, id * p.Hkv + h, &full[s], pol);
  };
#pragma unroll 1
  for (int o = 0; o < kStages && o < n_ord; o += 2) issue_pair(o);

  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // heads 2tig and 2tig+1 (l: this lane's share)
  float acc[8][4];   // acc[c]: d in [16c, 16c + 16); [0],[1]: d = 16c + 2 gid, heads 2tig, 2tig+1; [2],[3]: d = 16c + 2 gid + 1
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;

  // ldmatrix lane addressing inside a slab [16 tokens][128 B]: matrix mat = lane >> 3, row r = lane & 7 of it;
  // both operands take tokens r + 8 (mat & 1) and the 16-byte chunk c0 + (mat >> 1) of the row.
  const int lm = lane >> 3, lr = lane & 7;
  const int tok = lr + 8 * (lm & 1), sub = lm >> 1;
  const uint32_t k_row = k_off + (uint32_t)tok * 128u, v_row = v_off + (uint32_t)tok * 128u;
  const uint32_t swz = (uint32_t)(tok & 7);

  bool alive = true;
#pragma unroll 1
  for (int o = 0; o < n_ord; o += 2) {
    const int s0 = o % kStages, s1 = (o + 1) % kStages;
    alive = mbar_wait(p, &full[s0], (o / kStages) & 1, wait_cycles) &&
            mbar_wait(p, &full[s1], ((o + 1) / kStages) & 1, wait_cycles);
    alive = __all_sync(0xffffffffu, alive);
    if (!alive) break;
    const uint32_t base[2] = {smem_u32(ring[s0]), smem_u32(ring[s1])};
    const bool odd_blk = (o >> 5) & 1;
    const float skb = odd_blk ? sk1 : sk0, svb = odd_blk ? sv1 : sv0;
    const float ks0 = __shfl_sync(0xffffffffu, skb, o & 31), ks1 = __shfl_sync(0xffffffffu, skb, (o + 1) & 31);
    const float vs0 = __shfl_sync(0xffffffffu, svb, o & 31), vs1 = __shfl_sync(0xffffffffu, svb, (o + 1) & 31);
    // ---- scores of both pages: two independent chains per page (even / odd 16-wide step)
    float sc[2][2][4];
#pragma unroll
    for (int pg = 0; pg < 2; ++pg)
#pragma unroll
      for (int e = 0; e < 2; ++e) sc[pg][e][0] = sc[pg][e][1] = sc[pg][e][2] = sc[pg][e][3] = 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {   // chunks 2j and 2j + 1 of both pages
#pragma unroll
      for (int pg = 0; pg < 2; ++pg) {
        uint32_t r0, r1, r2, r3;
        ldsm_x4(base[pg] + k_row + ((((uint32_t)(2 * j + sub)) ^ swz) << 4), r0, r1, r2, r3);
        uint32_t a0, a1, a2, a3;
        widen4(r0, a0, a2);   // tokens 0-7:  slots 2t, 2t+1 | 2t+8, 2t+9
        widen4(r1, a1, a3);   // tokens 8-15
        mma16816_f16(sc[pg][0], a0, a1, a2, a3, qf[2 * j][0], qf[2 * j][1]);
        widen4(r2, a0, a2);
        widen4(r3, a1, a3);
        mma16816_f16(sc[pg][1], a0, a1, a2, a3, qf[2 * j + 1][0], qf[2 * j + 1][1]);
      }
    }
    // ---- masks: tokens at or beyond the part's end, the pad page, pages with a bad id
    const int tok0 = sp.lo + o * kPage;
    const uint32_t gm = odd_blk ? good1 : good0;   // o is even: o and o + 1 lie in the same block of 32
    const int hi0 = (gm >> (o & 31)) & 1u ? sp.hi : 0;
    const int hi1 = (o + 1 < n_pages) && ((gm >> ((o + 1) & 31)) & 1u) ? sp.hi : 0;
    const float c0 = sl2 * ks0, c1 = sl2 * ks1;
    float x[2][2][2];   // [page][row: token gid / gid + 8][head 2tig / 2tig + 1], scaled scores in log2 units
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        x[0][r][e] = tok0 + gid + 8 * r < hi0 ? (sc[0][0][2 * r + e] + sc[0][1][2 * r + e]) * c0 : -INFINITY;
        x[1][r][e] = tok0 + kPage + gid + 8 * r < hi1 ? (sc[1][0][2 * r + e] + sc[1][1][2 * r + e]) * c1 : -INFINITY;
      }
    // ---- running maximum, refreshed only when some score is clearly above it
    float mx0 = fmaxf(fmaxf(x[0][0][0], x[0][1][0]), fmaxf(x[1][0][0], x[1][1][0]));
    float mx1 = fmaxf(fmaxf(x[0][0][1], x[0][1][1]), fmaxf(x[1][0][1], x[1][1][1]));
    if (__any_sync(0xffffffffu, mx0 > m0 + 8.f || mx1 > m1 + 8.f)) {
#pragma unroll
      for (int sh = 4; sh <= 16; sh <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
      }
      const float n0 = fmaxf(m0, mx0), n1 = fmaxf(m1, mx1);
      const float a0 = fast_exp2(m0 - (n0 == -INFINITY ? 0.f : n0)), a1 = fast_exp2(m1 - (n1 == -INFINITY ? 0.f : n1));
      m0 = n0;
      m1 = n1;
      l0 *= a0;
      l1 *= a1;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        acc[i][0] *= a0; acc[i][1] *= a1; acc[i][2] *= a0; acc[i][3] *= a1;
      }
    }
    const float r0m = m0 == -INFINITY ? 0.f : m0, r1m = m1 == -INFINITY ? 0.f : m1;
    uint32_t pb[2][2];   // [page][token half]: (P scaled by the page's V scale)^T as the B operand of the second product
#pragma unroll
    for (int pg = 0; pg < 2; ++pg) {
      const float vs = pg ? vs1 : vs0;
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const float e0 = fast_exp2(x[pg][r][0] - r0m), e1 = fast_exp2(x[pg][r][1] - r1m);
        l0 += e0;
        l1 += e1;
        pb[pg][r] = transpose8x8(pack_f16x2(e0 * vs, e1 * vs));
      }
    }
    // ---- O^T += V^T P^T for both pages
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
      for (int pg = 0; pg < 2; ++pg) {
        uint32_t r0, r1, r2, r3;
        ldsm_x4_trans(base[pg] + v_row + ((((uint32_t)(2 * j + sub)) ^ swz) << 4), r0, r1, r2, r3);
        // a register holds (token 2t: d, d+1 | token 2t+1: d, d+1) with d = 16 c + 2 gid: sort into (d: both
        // tokens | d+1: both tokens), widen, and the halves are rows gid and gid + 8 of the A operand
        uint32_t a0, a1, a2, a3;
        widen4(__byte_perm(r0, 0u, 0x3120), a0, a1);   // tokens 2t, 2t+1
        widen4(__byte_perm(r1, 0u, 0x3120), a2, a3);   // tokens 2t+8, 2t+9
        mma16816_f16(acc[2 * j], a0, a1, a2, a3, pb[pg][0], pb[pg][1]);
        widen4(__byte_perm(r2, 0u, 0x3120), a0, a1);
        widen4(__byte_perm(r3, 0u, 0x3120), a2, a3);
        mma16816_f16(acc[2 * j + 1], a0, a1, a2, a3, pb[pg][0], pb[pg][1]);
      }
    }
    __syncwarp();   // every lane has read both stages before they are refilled
    if (o + kStages < n_ord) issue_pair(o + kStages);
    const int done = o + 2;
    if ((done & 31) == 0) load_ids((done >> 5) + 1);
    if ((done & 31) == 8 && done >= 40) finish_block((done >> 5) + 1);
  }
  if (!alive) {
    const long long t0 = clock64();
    while (clock64() - t0 < kDrainCycles) { }
    return;
  }

#pragma unroll
  for (int sh = 4; sh <= 16; sh <<= 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, sh);
    l1 += __shfl_xor_sync(0xffffffffu, l1, sh);
  }
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int head = 2 * tig + e;
    if (head >= g) continue;
    const float l = e ? l1 : l0, m = e ? m1 : m0;
    const size_t slot = (row0 + head) * p.n_parts + sp.part;
    if (gid == 0) lse_part[slot] = l > 0.f ? (m + log2f(l)) * kLn2 : -INFINITY;
    if (l > 0.f) {
      const float inv = 1.f / l;
      float2 *dst = reinterpret_cast<float2 *>(o_part + slot * D) + gid;   // the 8 lanes of a column write 64 contiguous bytes
#pragma unroll
      for (int i = 0; i < 8; ++i) dst[8 * i] = make_float2(acc[i][e] * inv, acc[i][2 + e] * inv);
    }
  }
}

template <int MODE>
__global__ void __launch_bounds__(kW * 32)
attn_fp8_kernel(Params p, const __grid_constant__ CUtensorMap kv_map, uint32_t k_off, uint32_t v_off,
                const __nv_bfloat16 *__restrict__ q, float sl2, float *__restrict__ o_part,
                float *__restrict__ lse_part, long long wait_cycles) {
  attn_fp8_body<MODE>(p, kv_map, k_off, v_off, q, sl2, o_part, lse_part, wait_cycles);
  // Launched as the programmatic dependent of the tensor-core prefix pass, the suffix grid starts before that one
  // ends; one thread of the grid waits for the prerequisite grid before it exits, so that this grid - and the merge
  // behind it - cannot complete earlier.  Without a prerequisite the instruction returns at once.
  if (MODE == kSuffix && blockIdx.x == gridDim.x - 1 && threadIdx.x == 0)
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
}

// ------------------------------------------------------------------------------------------------
// Expansion of the prefix levels for the tensor-core prefix pass.  That pass wants 16-bit operands in shared
// memory, and the prefix does not change while candidates decode: its pages are widened once into pools of their
// own - K as the exact codes in bf16 (e4m3 fits bf16 exactly; the page's K scale travels beside it and multiplies
// the scores in the softmax, so no rounding touches the scores), V as bf16(code * scale) (one rounding of relative
// size 2^-9 on the values that are averaged).  One CTA per (group, page index) of a level; page (j, i) lands at the
// fixed id base + j * max_pages + i, and the level's table of expanded ids gets that id, or -1 for a page whose
// source id lies outside the pool.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
expand_prefix_kernel(Params p, int base, __nv_bfloat16 *__restrict__ kx, __nv_bfloat16 *__restrict__ vx,
                     float *__restrict__ kx_scale, int32_t *__restrict__ xpages) {
  const int j = blockIdx.x / p.max_pp, i = blockIdx.x % p.max_pp;
  int len = __ldg(p.prefix_len + j);
  len = len < 0 ? 0 : len > p.max_pp * kPage ? p.max_pp * kPage : len;
  if (i * kPage >= len) return;
  const int pid = __ldg(p.prefix_pages + (size_t)j * p.max_pp + i);
  const int cid = base + blockIdx.x;
  if ((unsigned)pid >= (unsigned)p.num_pages) {
    if (threadIdx.x == 0) {
      latch(p, kDevBadPage);
      xpages[blockIdx.x] = -1;
    }
    return;
  }
  if (threadIdx.x == 0) xpages[blockIdx.x] = cid;
  if (threadIdx.x < p.Hkv) kx_scale[(size_t)cid * p.Hkv + threadIdx.x] = __ldg(p.k_scale + (size_t)pid * p.Hkv + threadIdx.x);
  const int n_vec = p.Hkv * kPage * D / 16;   // 16-byte pieces of one page of one pool
  const uint4 *ksrc = reinterpret_cast<const uint4 *>(p.k_pool) + (size_t)pid * n_vec;
  const uint4 *vsrc = reinterpret_cast<const uint4 *>(p.v_pool) + (size_t)pid * n_vec;
  uint4 *kdst = reinterpret_cast<uint4 *>(kx) + (size_t)cid * n_vec * 2;
  uint4 *vdst = reinterpret_cast<uint4 *>(vx) + (size_t)cid * n_vec * 2;
  for (int t = threadIdx.x; t < 2 * n_vec; t += blockDim.x) {
    const bool is_v = t >= n_vec;
    const int c = is_v ? t - n_vec : t;
    const uint4 w = __ldg((is_v ? vsrc : ksrc) + c);
    const float sc = is_v ? __ldg(p.v_scale + (size_t)pid * p.Hkv + c / (kPage * D / 16)) : 1.f;
    const uint32_t in[4] = {w.x, w.y, w.z, w.w};
    uint32_t out[8];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      uint32_t lo, hi;
      widen4(in[k], lo, hi);
      const __half2 a = *reinterpret_cast<__half2 *>(&lo), b = *reinterpret_cast<__half2 *>(&hi);
      const float2 fa = __half22float2(a), fb = __half22float2(b);
      const __nv_bfloat162 ra = __floats2bfloat162_rn(fa.x * sc, fa.y * sc), rb = __floats2bfloat162_rn(fb.x * sc, fb.y * sc);
      out[2 * k] = *reinterpret_cast<const uint32_t *>(&ra);
      out[2 * k + 1] = *reinterpret_cast<const uint32_t *>(&rb);
    }
    uint4 *dst = (is_v ? vdst : kdst) + 2 * c;
    dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
    dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
  }
}

// ------------------------------------------------------------------------------------------------
// append: one block per candidate, one warp per kv head (in turn), a lane holds four neighbouring elements of
// the K row and of the V row.  The token that opens a page (slot 0) fixes the page's scales:
// scale = (2 * max|row|) / 448, or 1 for a row of zeros; later tokens read them.  code = e4m3(x / scale), the
// quotient rounded once in single precision, the conversion to nearest-even with saturation at +-448.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t encode4(float a, float b, float c, float d) {
  uint32_t r;
  asm("{\n\t.reg .b16 l, h;\n\t"
      "cvt.rn.satfinite.e4m3x2.f32 l, %2, %1;\n\t"     // first source operand -> upper byte
      "cvt.rn.satfinite.e4m3x2.f32 h, %4, %3;\n\t"
      "mov.b32 %0, {l, h};\n\t}\n"
      : "=r"(r) : "f"(a), "f"(b), "f"(c), "f"(d));
  return r;
}

__global__ void __launch_bounds__(256) append_fp8_kernel(Params p, const __nv_bfloat16 *__restrict__ k_new,
                                                         const __nv_bfloat16 *__restrict__ v_new, int32_t *suffix_len,
                                                         float *k_scale, float *v_scale) {
  const int b = blockIdx.x;
  const int s = suffix_len[b];
  const int pg = s >> 4;
  int page = -1;
  if (s >= 0 && pg < p.max_sp) page = __ldg(p.suffix_pages + (size_t)b * p.max_sp + pg);
  if ((unsigned)page >= (unsigned)p.num_pages) {  // row full, or a bad table entry: leave the candidate alone
    if (threadIdx.x == 0) latch(p, kDevBadPage);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, slot = s & 15;
  uint8_t *kp = reinterpret_cast<uint8_t *>(const_cast<void *>(p.k_pool));
  uint8_t *vp = reinterpret_cast<uint8_t *>(const_cast<void *>(p.v_pool));
  for (int h = warp; h < p.Hkv; h += 8) {
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      const __nv_bfloat16 *src = (which ? v_new : k_new) + ((size_t)b * p.Hkv + h) * D + 4 * lane;
      const uint2 w = *reinterpret_cast<const uint2 *>(src);
      const float x0 = __uint_as_float(w.x << 16), x1 = __uint_as_float(w.x & 0xffff0000u);
      const float x2 = __uint_as_float(w.y << 16), x3 = __uint_as_float(w.y & 0xffff0000u);
      float *scale_ptr = (which ? v_scale : k_scale) + (size_t)page * p.Hkv + h;
      float scale;
      if (slot == 0) {
        float amax = fmaxf(fmaxf(fabsf(x0), fabsf(x1)), fmaxf(fabsf(x2), fabsf(x3)));
#pragma unroll
        for (int sh = 16; sh >= 1; sh >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, sh));
        scale = amax > 0.f ? __fdiv_rn(amax * 2.f, 448.f) : 1.f;
        if (lane == 0) *scale_ptr = scale;
      } else {
        scale = *scale_ptr;
      }
      const uint32_t codes = encode4(__fdiv_rn(x0, scale), __fdiv_rn(x1, scale), __fdiv_rn(x2, scale), __fdiv_rn(x3, scale));
      uint8_t *dst = (which ? vp : kp) + (((size_t)page * p.Hkv + h) * kPage + slot) * D + 4 * lane;
      *reinterpret_cast<uint32_t *>(dst) = codes;
    }
  }
  __syncthreads();  // every thread has read s and issued its stores before the length moves
  if (threadIdx.x == 0) suffix_len[b] = s + 1;
}

// Several tokens per candidate: block (t, b) quantises token t of candidate b for suffix position s = len + t.  The
// scale of its page is the one the page's opening token fixes: its own row when it opens the page (it also stores
// the scale), the row of the batch's token that does when that token is part of this call, else the stored one.  The
// lengths move in a second launch.
__global__ void __launch_bounds__(256)
append_tokens_fp8_kernel(Params p, const __nv_bfloat16 *__restrict__ k_new, const __nv_bfloat16 *__restrict__ v_new,
                         int n_max, const int32_t *__restrict__ n_new, const int32_t *__restrict__ suffix_len,
                         float *k_scale, float *v_scale) {
  const int t = blockIdx.x, b = blockIdx.y;
  int n = n_max;
  if (n_new) {
    n = __ldg(n_new + b);
    n = n < 0 ? 0 : n > n_max ? n_max : n;
  }
  if (t >= n) return;
  const int s0 = __ldg(suffix_len + b);
  if (s0 < 0 || (long long)s0 + n > (long long)p.max_sp * kPage) return;   // (reported when the lengths move)
  const int s = s0 + t, slot = s & 15;
  const int page = __ldg(p.suffix_pages + (size_t)b * p.max_sp + (s >> 4));
  if ((unsigned)page >= (unsigned)p.num_pages) {
    if (threadIdx.x == 0) latch(p, kDevBadPage);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t_open = t - slot;   // the batch's token that opens this page, if it is in the batch
  uint8_t *kp = reinterpret_cast<uint8_t *>(const_cast<void *>(p.k_pool));
  uint8_t *vp = reinterpret_cast<uint8_t *>(const_cast<void *>(p.v_pool));
  for (int h = warp; h < p.Hkv; h += 8) {
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      const __nv_bfloat16 *base = (which ? v_new : k_new) + ((size_t)b * n_max * p.Hkv + h) * D + 4 * lane;
      const uint2 w = *reinterpret_cast<const uint2 *>(base + (size_t)t * p.Hkv * D);
      const float x0 = __uint_as_float(w.x << 16), x1 = __uint_as_float(w.x & 0xffff0000u);
      const float x2 = __uint_as_float(w.y << 16), x3 = __uint_as_float(w.y & 0xffff0000u);
      float *scale_ptr = (which ? v_scale : k_scale) + (size_t)page * p.Hkv + h;
      float scale;
      if (t_open >= 0) {
        const uint2 o = *reinterpret_cast<const uint2 *>(base + (size_t)t_open * p.Hkv * D);
        float amax = fmaxf(fmaxf(fabsf(__uint_as_float(o.x << 16)), fabsf(__uint_as_float(o.x & 0xffff0000u))),
                           fmaxf(fabsf(__uint_as_float(o.y << 16)), fabsf(__uint_as_float(o.y & 0xffff0000u))));
#pragma unroll
        for (int sh = 16; sh >= 1; sh >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, sh));
        scale = amax > 0.f ? __fdiv_rn(amax * 2.f, 448.f) : 1.f;
        if (slot == 0 && lane == 0) *scale_ptr = scale;
      } else {
        scale = *scale_ptr;
      }
      const uint32_t codes = encode4(__fdiv_rn(x0, scale), __fdiv_rn(x1, scale), __fdiv_rn(x2, scale), __fdiv_rn(x3, scale));
      uint8_t *dst = (which ? vp : kp) + (((size_t)page * p.Hkv + h) * kPage + slot) * D + 4 * lane;
      *reinterpret_cast<uint32_t *>(dst) = codes;
    }
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Both byte pools in one map: the (page, kv head) slabs of the pool at the lower address and, `distance` bytes above
// each, the same slab of the other pool.  One 4 KB box = [pool][16 tokens][128 bytes] of one (page, kv head).
bool encode_kv8_pair_map(CUtensorMap *map, const void *lower_pool, unsigned long long distance, int num_pages, int Hkv) {
  if (distance == 0 || (distance & 15ull) != 0 || distance >= (1ull << 40)) return false;
  void *sym = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !sym)
    return false;
  EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(sym);
  const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)kPage, (cuuint64_t)num_pages * (cuuint64_t)Hkv, 2};
  const cuuint64_t strides[3] = {(cuuint64_t)D, (cuuint64_t)kPage * D, (cuuint64_t)distance};
  const cuuint32_t box[4] = {(cuuint32_t)D, (cuuint32_t)kPage, 1, 2};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(lower_pool), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

struct Fp8Plan {
  CUtensorMap kv_map;
  uint32_t k_off, v_off;   // where a stage holds the K slab and the V slab
  long long wait_cycles;   // limit of every device-side wait
  // the prefix levels widened to bf16 for the tensor-core prefix pass (null: not made)
  __nv_bfloat16 *kx, *vx;
  float *kx_scale;
  int32_t *xpages;         // expanded page ids, level after level, [G_k][max_pages_k] each
  int x_pages;             // pages in kx / vx
};

int fp8_items_per_cta() { return kW; }

bool fp8_supported(const Params &p) { return p.d == D && p.g >= 1 && p.g <= 8 && p.k_scale && p.v_scale; }

Fp8Plan *fp8_plan(const Params &p) {
  if (!fp8_supported(p)) return nullptr;
  Fp8Plan *plan = new Fp8Plan();
  const uintptr_t ka = reinterpret_cast<uintptr_t>(p.k_pool), va = reinterpret_cast<uintptr_t>(p.v_pool);
  plan->k_off = ka < va ? 0u : kSlabBytes;
  plan->v_off = ka < va ? kSlabBytes : 0u;
  plan->wait_cycles = wait_limit_cycles();
  plan->kx = plan->vx = nullptr;
  plan->kx_scale = nullptr;
  plan->xpages = nullptr;
  plan->x_pages = 0;
  if ((long long)p.num_pages * p.Hkv > 0x7fffffffLL ||
      !encode_kv8_pair_map(&plan->kv_map, ka < va ? p.k_pool : p.v_pool, (unsigned long long)(ka < va ? va - ka : ka - va),
                           p.num_pages, p.Hkv) ||
      cudaFuncSetAttribute(attn_fp8_kernel<kPrefix>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Smem)) !=
          cudaSuccess ||
      cudaFuncSetAttribute(attn_fp8_kernel<kSuffix>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Smem)) !=
          cudaSuccess) {
    (void)cudaGetLastError();
    delete plan;
    return nullptr;
  }
  return plan;
}

void fp8_plan_free(Fp8Plan *plan) {
  if (!plan) return;
  cudaFree(plan->kx);
  cudaFree(plan->vx);
  cudaFree(plan->kx_scale);
  cudaFree(plan->xpages);
  delete plan;
}

// Allocates the expanded pools for `n_levels` prefix levels and fills `expanded[k]` with level k seen through them
// (pools, page table, page count, scale array; everything else as in levels[k]).  false: out of memory or too large.
bool fp8_expand_alloc(Fp8Plan *plan, const Params *levels, int n_levels, Params *expanded) {
  long long total = 0;
  for (int k = 0; k < n_levels; ++k) total += (long long)levels[k].G * levels[k].max_pp;
  if (total < 1 || total > 0x7fffffffLL / levels[0].Hkv) return false;
  const size_t pool_bytes = (size_t)total * levels[0].Hkv * kPage * D * sizeof(__nv_bfloat16);
  if (cudaMalloc(&plan->kx, pool_bytes) != cudaSuccess || cudaMalloc(&plan->vx, pool_bytes) != cudaSuccess ||
      cudaMalloc(&plan->kx_scale, (size_t)total * levels[0].Hkv * sizeof(float)) != cudaSuccess ||
      cudaMalloc(&plan->xpages, (size_t)total * sizeof(int32_t)) != cudaSuccess) {
    (void)cudaGetLastError();
    cudaFree(plan->kx); cudaFree(plan->vx); cudaFree(plan->kx_scale); cudaFree(plan->xpages);
    plan->kx = plan->vx = nullptr;
    plan->kx_scale = nullptr;
    plan->xpages = nullptr;
    return false;
  }
  plan->x_pages = (int)total;
  long long base = 0;
  for (int k = 0; k < n_levels; ++k) {
    expanded[k] = levels[k];
    expanded[k].k_pool = plan->kx;
    expanded[k].v_pool = plan->vx;
    expanded[k].num_pages = plan->x_pages;
    expanded[k].prefix_pages = plan->xpages + base;
    expanded[k].k_scale = plan->kx_scale;
    expanded[k].v_scale = nullptr;
    base += (long long)levels[k].G * levels[k].max_pp;
  }
  return true;
}

const float *fp8_expanded_k_scale(const Fp8Plan *plan) { return plan ? plan->kx_scale : nullptr; }

// (Re)writes the expanded pools from the levels' pages as they are now; asynchronous on `stream`.
mc_status_t fp8_expand_launch(const Fp8Plan *plan, const Params *levels, int n_levels, cudaStream_t stream) {
  if (!plan->kx) return MC_OK;
  long long base = 0;
  for (int k = 0; k < n_levels; ++k) {
    const long long n = (long long)levels[k].G * levels[k].max_pp;
    expand_prefix_kernel<<<(unsigned)n, 256, 0, stream>>>(levels[k], (int)base, plan->kx, plan->vx, plan->kx_scale,
                                                          plan->xpages + base);
    count_launch();
    base += n;
  }
  return check_launch();
}

mc_status_t launch_fp8(const Params &p, const Fp8Plan *plan, int mode, const void *q, float scale, float *o_part,
                       float *lse_part, cudaStream_t stream, bool beside_previous) {
  const int nparts_mode = mode == kPrefix ? p.n_prefix_parts : p.n_parts - p.suffix_part_base;
  const long long n_items = (long long)p.B * p.Hkv * nparts_mode;
  if (n_items == 0) return MC_OK;
  const __nv_bfloat16 *qb = reinterpret_cast<const __nv_bfloat16 *>(q);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((n_items + kW - 1) / kW));
  cfg.blockDim = dim3(kW * 32);
  cfg.dynamicSmemBytes = sizeof(Smem);
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = beside_previous && mode == kSuffix ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, mode == kPrefix ? attn_fp8_kernel<kPrefix> : attn_fp8_kernel<kSuffix>, p,
                                           plan->kv_map, plan->k_off, plan->v_off, qb, scale * kLog2e, o_part, lse_part,
                                           plan->wait_cycles);
  count_launch();
  return e == cudaSuccess ? check_launch() : MC_ERR_CUDA;
}

mc_status_t launch_append_tokens_fp8(const Params &p, const void *k_new, const void *v_new, int n_max,
                                     const int32_t *n_new, const int32_t *suffix_len, cudaStream_t stream) {
  append_tokens_fp8_kernel<<<dim3((unsigned)n_max, (unsigned)p.B), 256, 0, stream>>>(
      p, reinterpret_cast<const __nv_bfloat16 *>(k_new), reinterpret_cast<const __nv_bfloat16 *>(v_new), n_max, n_new,
      suffix_len, const_cast<float *>(p.k_scale), const_cast<float *>(p.v_scale));
  count_launch();
  return check_launch();
}

mc_status_t launch_append_fp8(const Params &p, const void *k_new, const void *v_new, int32_t *suffix_len,
                              cudaStream_t stream) {
  append_fp8_kernel<<<p.B, 256, 0, stream>>>(p, reinterpret_cast<const __nv_bfloat16 *>(k_new),
                                             reinterpret_cast<const __nv_bfloat16 *>(v_new), suffix_len,
                                             const_cast<float *>(p.k_scale), const_cast<float *>(p.v_scale));
  count_launch();
  return check_launch();
}

}  // namespace mc
