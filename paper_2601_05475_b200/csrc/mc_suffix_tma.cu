// Suffix pass, bf16, d = 128, g <= 8: split-KV attention with one warp per (candidate, kv head, chunk) whose
// K/V pages arrive through a private shared-memory ring filled by TMA.
//
// A warp that loads its pages into registers (the warp-level kernel in mc_mma.cu) has one page in flight and
// spends a page's whole dependent chain (eight chained MMAs, cross-lane maxima, exponentials, the second
// product) before it can ask for the page after next: measured, that chain and not HBM sets its pace, so the
// pass needs every warp slot of every SM to reach the memory roofline and loses speed as soon as another
// kernel holds some of them.  Here the loads are asynchronous copies that cost no registers:
//   * each warp owns a ring of kStages page stages (K slab 4 KB + V slab 4 KB each); one lane issues the TMA
//     copy of a page (128-byte swizzle, so that the fragment loads below are free of bank conflicts)
//     kStages pages ahead of the page being computed, and an mbarrier per stage counts the bytes in;
//   * fragments come from shared memory with ldmatrix (K as the A operand of S = K_page Q^T, V transposed
//     as the A operand of O^T += V_page^T P^T), so nothing is permuted in registers;
//   * an iteration takes two pages: two independent score chains, and the running maximum is only refreshed
//     (a cross-lane reduction and a rescale of the accumulators) when some score exceeds it by more than
//     2^8; otherwise the stale maximum is used, which changes no result beyond rounding because the same
//     reference enters the numerator and the denominator.
// Output format, item numbering and masking rules are those of the warp-level kernel.
#include <cstdlib>

#include "mc_internal.cuh"

namespace mc {
namespace {

constexpr int D = 128;
constexpr int kW = 2;                      // warps (items) per CTA
constexpr int kStages = 4;                 // page stages per warp: two being computed, two in flight
constexpr uint32_t kSlabBytes = kPage * D * 2;       // one (page, kv head) slab of K or of V
constexpr uint32_t kStageBytes = 2 * kSlabBytes;
constexpr long long kDrainCycles = 2000000ll;        // ~1 ms: what a warp that gives up grants its copies in flight

struct __align__(1024) Smem {
  uint8_t ring[kW][kStages][kStageBytes];   // [warp][stage][K slab | V slab], each slab [d half][16 tokens][64], swizzled
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
// Private suffix data is read exactly once per step: evict-first in L2, so that it does not push out the
// shared prefix, which every step re-reads.
__device__ __forceinline__ uint64_t l2_stream_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(pol));
  return pol;
}
// The K slab and the V slab of one (page, kv head), 8 KB, as one box: lands as [pool][d half][16 tokens][64 elements]
// with the 128-byte swizzle.  `slab` = page * Hkv + kv head.
__device__ __forceinline__ void tma_load_stage(uint32_t dst, const CUtensorMap *map, int slab, uint64_t *bar,
                                               uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%2, %3, %4, %5, %6}], [%7], %8;\n"
      ::"r"(dst), "l"(map), "r"(0), "r"(0), "r"(0), "r"(slab), "r"(0), "r"(smem_u32(bar)), "l"(policy)
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
__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t transpose8x8(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void
suffix_tma_body(const Params &p, const CUtensorMap &kv_map, uint32_t k_off, uint32_t v_off,
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
  // A kernel launched behind this one as its programmatic dependent (the merge, which waits for this grid's
  // completion before it reads anything) may take its place on the SMs once every CTA of this grid has started.
  if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");

  const int n_chunks = p.n_parts - p.suffix_part_base;
  const long long n_items = (long long)p.B * p.Hkv * n_chunks;
  const long long cta = p.suffix_order ? __ldg(p.suffix_order + blockIdx.x) : blockIdx.x;
  const long long item = cta * kW + warp;
  if (item >= n_items) return;
  // kv heads of one page are adjacent in the pool: neighbouring warps stream neighbouring slabs
  const int h = (int)(item % p.Hkv);
  const int part = (int)((item / p.Hkv) % n_chunks);
  const int b = (int)(item / ((long long)p.Hkv * n_chunks));

  // The chunk's first page ids depend only on the chunk index, not on the sequence length: their loads, the
  // length's and the queries' are issued together.  Entries of a page-table row beyond the sequence are read
  // here but never used as page ids.
  const int first_pg = part * (p.suffix_part_tokens >> 4);
  const int32_t *row_pages = p.suffix_pages + (size_t)b * p.max_sp + first_pg;
  const int row_left = p.max_sp - first_pg;                  // table entries from the chunk's first page on
  auto load_ids = [&](int blk) -> int {
    const int o = blk * 32 + lane;
    return o < row_left ? __ldg(row_pages + o) : -1;
  };
  int ids0 = load_ids(0), ids1 = load_ids(1);                // page ids of ordinals [0,32) and [32,64) of the chunk
  // B operand of the first product: Q^T, column n = head gid, k-step kk covers d in [16 kk, 16 kk + 16)
  uint32_t qf[8][2];
  {
    const uint32_t *qrow = reinterpret_cast<const uint32_t *>(q + ((size_t)b * p.Hq + (size_t)h * p.g + gid) * D);
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      qf[kk][0] = gid < p.g ? __ldg(qrow + 8 * kk + tig) : 0u;
      qf[kk][1] = gid < p.g ? __ldg(qrow + 8 * kk + 4 + tig) : 0u;
    }
  }
  const Span sp = resolve_span<kSuffix>(p, b, part);
  const int g = p.g;
  const size_t row0 = (size_t)b * p.Hq + (size_t)h * g;
  if (sp.lo >= sp.hi) {
    if (lane < g) lse_part[(row0 + lane) * p.n_parts + sp.part] = -INFINITY;
    return;
  }
  const int n_pages = ((sp.hi + 15) >> 4) - (sp.lo >> 4);    // >= 1
  const int n_ord = (n_pages + 1) & ~1;                      // an odd count is padded with a masked repeat of the last page
  // which of a block's 32 pages have an id inside the pool (pages past the chunk count as good: never computed unmasked)
  auto good_mask = [&](int blk, int id) -> uint32_t {
    const int o = blk * 32 + lane;
    const bool good = o >= n_pages || (unsigned)id < (unsigned)p.num_pages;
    if (!good) latch(p, kDevBadPage);
    return __ballot_sync(0xffffffffu, good);
  };
  uint32_t good0 = good_mask(0, ids0), good1 = good_mask(1, ids1);

  const uint64_t pol = l2_stream_policy();
  uint8_t(*ring)[kStageBytes] = sm.ring[warp];
  uint64_t *full = sm.full[warp];
  // Pages o and o + 1 (o even), each issued by the lane that holds its id, both in one predicated instruction
  // stream.  The pad page and a page with a bad id are loaded from a page that exists (finite data) and masked
  // when computed.
  auto issue_pair = [&](int o) {
    if ((lane & 30) != (o & 30)) return;
    o += lane & 1;
    int id = (o >> 5) & 1 ? ids1 : ids0;
    if (o >= n_pages) id = __ldg(row_pages + n_pages - 1);
    if ((unsigned)id >= (unsigned)p.num_pages) id = 0;
    const int s = o % kStages;
    mbar_expect_tx(&full[s], kStageBytes);
    tma_load_stage(smem_u32(ring[s]), &kv_map, (int)slab_index(p, id, h), &full[s], pol);
  };
#pragma unroll 1
  for (int o = 0; o < kStages && o < n_ord; o += 2) issue_pair(o);

  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // heads 2tig and 2tig+1 (l: this lane's share)
  float acc[8][4];   // acc[i]: d tile i; [0],[1]: d = 16i + gid, heads 2tig, 2tig+1; [2],[3]: d = 16i + 8 + gid
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;

  // ldmatrix lane addressing inside a slab.  Matrix mat = lane >> 3, row r = lane & 7 of that matrix.
  //   K (A of S = K Q^T):  mat 0/1: tokens r / r + 8, first 16-byte chunk of the k-step;  mat 2/3: second chunk
  //   V (A of O^T += V^T P^T, transposed on load):  mat 0/1: tokens r, chunks dc / dc + 1;  mat 2/3: tokens r + 8
  const int lm = lane >> 3, lr = lane & 7;
  const int k_tok = lr + 8 * (lm & 1), k_chunk = lm >> 1;
  const int v_tok = lr + 8 * (lm >> 1), v_chunk = lm & 1;
  const uint32_t k_row = k_off + (uint32_t)k_tok * 128u, v_row = v_off + (uint32_t)v_tok * 128u;

  bool alive = true;
#pragma unroll 1
  for (int o = 0; o < n_ord; o += 2) {
    const int s0 = o % kStages, s1 = (o + 1) % kStages;
    alive = mbar_wait(p, &full[s0], (o / kStages) & 1, wait_cycles) &&
            mbar_wait(p, &full[s1], ((o + 1) / kStages) & 1, wait_cycles);
    alive = __all_sync(0xffffffffu, alive);
    if (!alive) break;
    const uint32_t base0 = smem_u32(ring[s0]), base1 = smem_u32(ring[s1]);
    // ---- scores of both pages: four independent chains (page x even/odd k-step).  Fragment loads run eight
    // slots ahead of the MMAs that use them (slot j: k-step j / 2 of page j % 2), so that no MMA waits for shared memory.
    float sa[2][4], sb[2][4];
#pragma unroll
    for (int e = 0; e < 2; ++e)
#pragma unroll
      for (int c = 0; c < 4; ++c) sa[e][c] = sb[e][c] = 0.f;
    uint32_t f[8][4];
    auto k_load = [&](int j) {
      const int kk = j >> 1;
      const uint32_t off = (uint32_t)(kk >> 2) * 2048u + k_row + ((((uint32_t)(2 * (kk & 3) + k_chunk)) ^ (uint32_t)(k_tok & 7)) << 4);
      ldsm_x4(((j & 1) ? base1 : base0) + off, f[j & 7][0], f[j & 7][1], f[j & 7][2], f[j & 7][3]);
    };
#pragma unroll
    for (int j = 0; j < 8; ++j) k_load(j);
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int kk = j >> 1;
      if (j & 1) mma16816(sb[kk & 1], f[j & 7][0], f[j & 7][1], f[j & 7][2], f[j & 7][3], qf[kk][0], qf[kk][1]);
      else mma16816(sa[kk & 1], f[j & 7][0], f[j & 7][1], f[j & 7][2], f[j & 7][3], qf[kk][0], qf[kk][1]);
      if (j + 8 < 16) k_load(j + 8);
    }
    // V fragments of the first four d tiles are requested now and arrive while the softmax below runs.
    // Slot j: d tile 4 (j / 8) + j % 4 of page (j % 8) / 4; a tile's two MMAs (one per page) are four slots apart.
    auto v_load = [&](int j) {
      const int i = 4 * (j >> 3) + (j & 3);
      const uint32_t off = (uint32_t)(i >> 2) * 2048u + v_row + ((((uint32_t)(2 * (i & 3) + v_chunk)) ^ (uint32_t)(v_tok & 7)) << 4);
      ldsm_x4_trans((((j & 7) >> 2) ? base1 : base0) + off, f[j & 7][0], f[j & 7][1], f[j & 7][2], f[j & 7][3]);
    };
#pragma unroll
    for (int j = 0; j < 8; ++j) v_load(j);
    // ---- masks: tokens at or beyond the chunk's end, the pad page, pages with a bad id
    const int tok0 = sp.lo + o * kPage;
    const uint32_t gm = (o >> 5) & 1 ? good1 : good0;   // o is even: o and o + 1 lie in the same block of 32
    const int hi0 = (gm >> (o & 31)) & 1u ? sp.hi : 0;
    const int hi1 = (o + 1 < n_pages) && ((gm >> ((o + 1) & 31)) & 1u) ? sp.hi : 0;
    float x[2][2][2];   // [page][row: token gid / gid + 8][head 2tig / 2tig + 1], scaled scores in log2 units
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        x[0][r][e] = tok0 + gid + 8 * r < hi0 ? (sa[0][2 * r + e] + sa[1][2 * r + e]) * sl2 : -INFINITY;
        x[1][r][e] = tok0 + kPage + gid + 8 * r < hi1 ? (sb[0][2 * r + e] + sb[1][2 * r + e]) * sl2 : -INFINITY;
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
    const float r0 = m0 == -INFINITY ? 0.f : m0, r1 = m1 == -INFINITY ? 0.f : m1;
    uint32_t pb[2][2];   // [page][token half]: P^T as the B operand of the second product
#pragma unroll
    for (int pg = 0; pg < 2; ++pg)
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const float e0 = fast_exp2(x[pg][r][0] - r0), e1 = fast_exp2(x[pg][r][1] - r1);
        l0 += e0;
        l1 += e1;
        pb[pg][r] = transpose8x8(pack_bf16x2(e0, e1));
      }
    // ---- O^T += V^T P^T for both pages
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int i = 4 * (j >> 3) + (j & 3), pg = (j & 7) >> 2;
      mma16816(acc[i], f[j & 7][0], f[j & 7][1], f[j & 7][2], f[j & 7][3], pb[pg][0], pb[pg][1]);
      if (j + 8 < 16) v_load(j + 8);
    }
    __syncwarp();   // every lane has read both stages before they are refilled
    if (o + kStages < n_ord) issue_pair(o + kStages);
    // Page ids: block k's register is reloaded with block k+2 once block k is consumed; the validity mask of the
    // new ids is taken half a block later, when the load has long returned.
    const int done = o + 2;
    const int nb = (done >> 5) + 1;   // the block whose ids are (re)loaded during block nb - 1
    if ((done & 31) == 0) {
      if (nb & 1) ids1 = load_ids(nb); else ids0 = load_ids(nb);
    }
    if ((done & 31) == 16 && done >= 32) {
      if (nb & 1) good1 = good_mask(nb, ids1); else good0 = good_mask(nb, ids0);
    }
  }
  if (!alive) {
    // A wait ran out: the warp writes no result.  Copies into its ring may still be in flight; they get a bounded
    // time to land before the warp leaves and the CTA's shared memory can go to another CTA.
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
      float *dst = o_part + slot * D + gid;   // the 8 lanes of a column write 32 contiguous bytes
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        dst[16 * i] = acc[i][e] * inv;
        dst[16 * i + 8] = acc[i][2 + e] * inv;
      }
    }
  }
}

__global__ void __launch_bounds__(kW * 32)
suffix_tma_kernel(Params p, const __grid_constant__ CUtensorMap kv_map, uint32_t k_off, uint32_t v_off,
                  const __nv_bfloat16 *__restrict__ q, float sl2, float *__restrict__ o_part,
                  float *__restrict__ lse_part, long long wait_cycles) {
  suffix_tma_body(p, kv_map, k_off, v_off, q, sl2, o_part, lse_part, wait_cycles);
  // Launched as the programmatic dependent of the prefix pass, this grid starts before that one ends.  The merge
  // behind it needs both: one thread of the grid (in the CTA that is scheduled last) waits for the prerequisite
  // grid to complete and its writes to be visible before it exits, so this grid cannot complete earlier.  Only
  // that thread waits - a CTA that waited would keep its SM slot from the next CTA of the stream.  Launched the
  // ordinary way there is no prerequisite and the instruction returns at once.
  if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) asm volatile("griddepcontrol.wait;\n" ::: "memory");
}

}  // namespace

struct SuffixTmaPlan {
  CUtensorMap kv_map;
  uint32_t k_off, v_off;   // where a stage holds the K slab and the V slab
  long long wait_cycles;   // limit of every device-side wait
};

int suffix_tma_items_per_cta() { return kW; }

// One tensor map over both pools (one 8 KB box per (page, kv head): its K slab and its V slab).  nullptr when
// unavailable, e.g. when the pools lie 2^40 bytes or more apart.
SuffixTmaPlan *suffix_tma_plan(const Params &p, int dtype) {
  if (dtype != MC_BF16 || p.d != D || p.g < 1 || p.g > 8) return nullptr;
  SuffixTmaPlan *plan = new SuffixTmaPlan();
  const uintptr_t ka = reinterpret_cast<uintptr_t>(p.k_pool), va = reinterpret_cast<uintptr_t>(p.v_pool);
  plan->k_off = ka < va ? 0u : kSlabBytes;
  plan->v_off = ka < va ? kSlabBytes : 0u;
  plan->wait_cycles = wait_limit_cycles();
  if ((long long)p.num_pages * p.Hkv > 0x7fffffffLL ||   // (num_pages counts 16-token unit pages: the map's slabs)
      !encode_kv_pair_map(&plan->kv_map, ka < va ? p.k_pool : p.v_pool, (unsigned long long)(ka < va ? va - ka : ka - va),
                          p.num_pages, p.Hkv) ||
      cudaFuncSetAttribute(suffix_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Smem)) !=
          cudaSuccess) {
    (void)cudaGetLastError();
    delete plan;
    return nullptr;
  }
  return plan;
}

void suffix_tma_plan_free(SuffixTmaPlan *plan) { delete plan; }

mc_status_t launch_suffix_tma(const Params &p, const SuffixTmaPlan *plan, const void *q, float scale, float *o_part,
                              float *lse_part, cudaStream_t stream, bool beside_previous) {
  const long long n_items = (long long)p.B * p.Hkv * (p.n_parts - p.suffix_part_base);
  if (n_items == 0) return MC_OK;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((n_items + kW - 1) / kW));
  cfg.blockDim = dim3(kW * 32);
  cfg.dynamicSmemBytes = sizeof(Smem);
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = beside_previous ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, suffix_tma_kernel, p, plan->kv_map, plan->k_off, plan->v_off,
                                           reinterpret_cast<const __nv_bfloat16 *>(q), scale * kLog2e, o_part, lse_part,
                                           plan->wait_cycles);
  count_launch();
  return e == cudaSuccess ? check_launch() : MC_ERR_CUDA;
}

}  // namespace mc
