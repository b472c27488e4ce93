// Prefix pass on the 5th-generation tensor cores (bf16, d = 128).
//
// For one (group, kv head) the queries of all the group's candidates that map to that kv head are
// stacked into dense 128-row tiles (row = candidate * g + head-in-group), so the group's prefix K/V is
// streamed once for the whole group instead of once per candidate:
//     S = Q_s K^T          128 x 128 tile, tcgen05.mma, operands in shared memory, accumulator in TMEM
//     P = exp2(S*c - m)    one thread per row reads the row of S from TMEM and writes bf16 P over it
//     O += P V             tcgen05.mma, P from TMEM, V in its natural [token][d] layout (MN-major B operand)
// K/V pages reach shared memory by TMA through tensor maps laid over the paged pools (the page id is a TMA
// coordinate): V as one 4 KB box per page, K as two 2 KB boxes per page (one per 64-element d half).
//
// Work item = (group, kv head, prefix split, 128-row tile); every CTA has a list of items.  Inside an item the
// 128-token K/V tiles are dealt alternately to two independent streams ("teams"): each team has its own S and O
// accumulators in TMEM (S0 O0 S1 O1 = 512 columns), its own 128 softmax threads and its own running maximum and
// row sum; the two are merged in the item's epilogue.  While one team
// computes the exponentials of its tile, the tensor pipe runs the other team's products.
// Warp roles: warp 0 and warps 10, 11 issue the TMA copies (warp 0 also stages the next item's query tile), warp 1
// lane 0 issues the MMAs (warp 1 owns the TMEM allocation), warps 2-5 are team 0 and warps 6-9 team 1 (one thread
// per TMEM lane, holding its whole row of 128 scores in registers: twelve warps leave each thread 168 registers,
// and a row needs no exchange between threads): softmax, rescale, epilogue.
// Every mbarrier wait is bounded: on expiry the CTA latches MC_ERR_TIMEOUT, stops issuing work, waits
// (bounded) for its outstanding copies, frees its TMEM and returns.
#include <algorithm>
#include <cstdlib>
#include <functional>
#include <type_traits>
#include <queue>
#include <utility>
#include <vector>

#include "mc_internal.cuh"
#include "mc_tcgen05.cuh"

namespace mc {
namespace {

constexpr int D = 128;
constexpr int kTileM = 128;      // stacked query rows per tile
constexpr int kTileN = 128;      // tokens per K/V tile (8 pages)
constexpr int kKSlots = 3;        // K tiles in flight or in use (TMA, two 2 KB boxes per page: one per d half)
constexpr int kVSlots = 2;        // V tiles (TMA, one 4 KB box per page)
constexpr int kTeams = 2;              // independent tile streams: tile t of an item belongs to team t & 1
constexpr int kSoftmaxThreads = 128;   // per team: one thread per row of the tile
constexpr int kProducers = 3;          // copy-issuing warps: K d-half 0 (+ query staging), K d-half 1, V
constexpr int kThreads = 64 + kTeams * kSoftmaxThreads + (kProducers - 1) * 32;
constexpr uint32_t kHalfBytes = kTileN * 64 * 2;        // one head-dim (or token) half of a 128x128 bf16 tile
constexpr uint32_t kTileBytes = 2 * kHalfBytes;         // 32 KB
constexpr uint32_t kPageBytes = kPage * D * 2;          // one (page, kv head) slab; one TMA box for V
constexpr uint32_t kTmemCols = 512;                     // team T: S at 256 T, O at 256 T + 128; P (bf16 pairs) over S:
                                                        // the thread that owns S columns [64 h, 64 h + 64) writes [64 h, 64 h + 32)
constexpr long long kDrainCycles = 2000000ll;           // ~1 ms: what an aborting CTA grants its copies and products in flight

struct __align__(1024) Smem {   // exactly the 227 KB a CTA may have
  uint8_t q[2][kTileBytes];           // stacked query tile of the current and of the next item
  uint8_t k[kKSlots][kTileBytes];     // [d half][128 tokens][64], 128-byte swizzle
  uint8_t v[kVSlots][kTileBytes];     // [page][d half][16 tokens][64], 128-byte swizzle
  uint64_t full_k[kKSlots], empty_k[kKSlots], full_v[kVSlots], empty_v[kVSlots];
  uint64_t q_ready[2], q_free[2], s_full[kTeams], p_full[kTeams], pv_done[kTeams];
  uint64_t both;                      // the two teams meet here around an item's epilogue
  float xch[kTeams][2][kTileM];       // [team][m, l][row]: the teams show each other their running maximum and row sum
  uint32_t page_ok[8];                // per tile (index kt & 7): which of its 8 pages hold valid data
  float kscale[8][8];                 // per tile (index kt & 7) and page: the K scale of an expanded e4m3 cache
  uint32_t tmem_base;
  volatile int abort;
  long long wait_cycles;              // limit of every wait of this CTA
};

// Bounded wait.  Returns false (and raises the CTA's abort flag) when the limit expires or another
// role has already aborted.
__device__ __forceinline__ bool mbar_wait(Smem &sm, const Params &p, uint64_t *bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    __nanosleep(32);   // a polling warp must not take issue slots from the softmax warps of its scheduler
    if (sm.abort) return false;
    if (clock64() - t0 > sm.wait_cycles) {
      sm.abort = 1;
      latch(p, kDevTimeout);
      return false;
    }
  }
}

// The shared prefix is re-read by every row tile of its group and again at every decode step: its
// lines are asked to stay in L2 (evict-last), while the private suffix streams past them.
__device__ __forceinline__ uint64_t l2_keep_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;\n" : "=l"(pol));
  return pol;
}
// One 16-token slab of V (a unit page of one kv head): both 64-element halves of its 16 token rows, 4 KB, one box.
// `slab` counts 16-token slabs of the pool (slab_index).
__device__ __forceinline__ void tma_load_page(void *dst, const CUtensorMap *map, int slab, uint64_t *bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%2, %3, %4, %5}], [%6], %7;\n"
      ::"r"(smem_u32(dst)), "l"(map), "r"(0), "r"(0), "r"(0), "r"(slab), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
// One d half (64 elements) of the 16 token rows of a slab of K: 2 KB.  The swizzle span caps a box at 64 elements per
// row, and the K-major operand wants each half's 128 token rows contiguous.
__device__ __forceinline__ void tma_load_half_page(void *dst, const CUtensorMap *map, int x, int slab, uint64_t *bar,
                                                   uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%2, %3, %4}], [%5], %6;\n"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(0), "r"(slab), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}

// kind::f16 instruction descriptor: bf16 x bf16 -> f32, M = 128, N = 128
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTileN >> 3) << 17) |
                                ((uint32_t)(kTileM >> 4) << 24);
constexpr uint32_t kIdescQK = kIdescBase;                // A, B both K-major
constexpr uint32_t kIdescPV = kIdescBase | (1u << 16);   // B (= V) MN-major

// One level of the prefix cascade as the kernel sees it; the levels' items are numbered one level after another.
struct TcLevel {
  const int32_t *group_offsets, *prefix_pages, *prefix_len;
  const int32_t *row_limit;   // per candidate: tokens of this level it may see (non-decreasing within a group), or null
  int32_t max_pp, n_splits, part_base, part_tokens, n_mt, item_end;
  int32_t n_groups;
  int32_t chain;   // >= 0: an item of this level also covers, for its rows, the whole prefix of that (coarser) level
};
struct TcLevels {
  int32_t n;
  TcLevel lv[kMaxTcLevels];
};

struct Item {
  int j, h, mt;          // group, kv head, row tile
  int part;              // part slot the result goes to
  int b0, n_cand;        // first candidate of the group, candidates in the group
  int lo, hi;            // token range of this split
  const int32_t *pages;
  const int32_t *limits; // per-candidate token limits of the group (indexed from its first candidate), or null
  // second token range, of the coarser level this level is chained to (lo2 >= hi2: none): the rows of the tile lie
  // in one group of that level, whose prefix the item attends in the same pass, into the same accumulator
  int lo2, hi2, part2;
  const int32_t *pages2, *limits2;
};

// `cand_per_unit`: candidates in one item's rows (one 128-row tile: 128 / g; a pair of row tiles: twice that)
__device__ __forceinline__ Item decode_item(const Params &p, const TcLevels &lvs, int item, int cand_per_unit) {
  int l = 0;
  while (l + 1 < lvs.n && item >= lvs.lv[l].item_end) ++l;
  const TcLevel &L = lvs.lv[l];
  if (l > 0) item -= lvs.lv[l - 1].item_end;
  Item it;
  it.mt = item % L.n_mt;
  int r = item / L.n_mt;
  const int sp = r % L.n_splits;
  r /= L.n_splits;
  it.h = r % p.Hkv;
  it.j = r / p.Hkv;
  it.b0 = __ldg(L.group_offsets + it.j);
  it.n_cand = __ldg(L.group_offsets + it.j + 1) - it.b0;
  int len = __ldg(L.prefix_len + it.j);
  const int cap = L.max_pp * kPage;
  if (len < 0 || len > cap) {
    latch(p, kDevBadPage);
    len = len < 0 ? 0 : cap;
  }
  it.part = L.part_base + sp;
  it.lo = sp * L.part_tokens;
  it.hi = min(len, it.lo + L.part_tokens);
  it.pages = L.prefix_pages + (size_t)it.j * L.max_pp;
  it.limits = nullptr;
  if (L.row_limit) {
    // the limits do not decrease inside a group: no row of this tile sees beyond the limit of its last candidate
    it.limits = L.row_limit + it.b0;
    const int last = min((it.mt + 1) * cand_per_unit, it.n_cand) - 1;
    if (last >= it.mt * cand_per_unit) it.hi = min(it.hi, max(__ldg(it.limits + last), 0));
  }
  it.lo2 = it.hi2 = 0;
  it.part2 = -1;
  it.pages2 = it.limits2 = nullptr;
  if (L.chain >= 0) {
    const TcLevel &C = lvs.lv[L.chain];
    int lo = 0, hi = C.n_groups;   // the coarser level's group that holds this group: offsets[lo] <= b0 < offsets[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (__ldg(C.group_offsets + mid) <= it.b0) lo = mid; else hi = mid;
    }
    int len2 = __ldg(C.prefix_len + lo);
    const int cap2 = C.max_pp * kPage;
    if (len2 < 0 || len2 > cap2) {
      latch(p, kDevBadPage);
      len2 = len2 < 0 ? 0 : cap2;
    }
    it.part2 = C.part_base;
    it.hi2 = len2;
    it.pages2 = C.prefix_pages + (size_t)lo * C.max_pp;
    if (C.row_limit) {
      it.limits2 = C.row_limit + it.b0;
      const int last = min((it.mt + 1) * cand_per_unit, it.n_cand) - 1;
      if (last >= it.mt * cand_per_unit) it.hi2 = min(it.hi2, max(__ldg(it.limits2 + last), 0));
    }
  }
  return it;
}
__device__ __forceinline__ int tiles_of(int lo, int hi) { return lo < hi ? (hi - lo + kTileN - 1) / kTileN : 0; }

// An item with no rows or no tokens is skipped by every role alike.
__device__ __forceinline__ bool item_has_work(const Item &it, int cand_per_tile) {
  return (it.lo < it.hi || it.lo2 < it.hi2) && it.mt * cand_per_tile < it.n_cand;
}

// KSCALE: the pools hold the exact codes of an e4m3 cache widened to bf16 (K) and its dequantised values (V); the
// scores of every page are multiplied by that page's K scale (`k_scale` [page][kv head]) in the softmax.
template <bool KSCALE>
__global__ void __maxnreg__(168)
prefix_tc_kernel(Params p, const __grid_constant__ TcLevels lvs, const __grid_constant__ CUtensorMap k_map,
                 const __grid_constant__ CUtensorMap v_map, const __nv_bfloat16 *__restrict__ q, float sl2,
                 float *__restrict__ o_part, float *__restrict__ lse_part, const int32_t *__restrict__ item_list,
                 const int32_t *__restrict__ cta_begin, __nv_bfloat16 *__restrict__ o_final,
                 float *__restrict__ lse_final, long long wait_cycles, const float *__restrict__ k_scale) {
  // o_final != null: every row gets exactly one part from this launch and none from anywhere else, so the item
  // writes the row's final output (bf16) and log-sum-exp itself and no merge follows.
  const bool direct = o_final != nullptr;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  Smem &sm = *reinterpret_cast<Smem *>(smem_raw);
  if ((smem_u32(smem_raw) & 1023u) != 0) {   // the swizzled tiles need a 1024-byte aligned base
    if (threadIdx.x == 0) latch(p, MC_ERR_CUDA);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = p.g, cand_per_tile = kTileM / g;
  // this CTA's items: a slice of the list made when the layout was created (balanced by the lengths then)
  const int k_begin = __ldg(cta_begin + blockIdx.x), k_end = __ldg(cta_begin + blockIdx.x + 1);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kKSlots; ++s) {
      mbar_init(&sm.full_k[s], 2);   // one arrival per K d half
      mbar_init(&sm.empty_k[s], 1);
    }
    for (int s = 0; s < kVSlots; ++s) {
      mbar_init(&sm.full_v[s], 1);
      mbar_init(&sm.empty_v[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&sm.q_ready[b], 32);
      mbar_init(&sm.q_free[b], 1);
    }
    mbar_init(&sm.both, kTeams * kSoftmaxThreads);
    for (int t = 0; t < kTeams; ++t) {
      mbar_init(&sm.s_full[t], 1);
      mbar_init(&sm.p_full[t], kSoftmaxThreads);
      mbar_init(&sm.pv_done[t], 1);
    }
    sm.abort = 0;
    sm.wait_cycles = wait_cycles;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&sm.tmem_base)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  if (threadIdx.x == kThreads - 1) {
    // This CTA holds its SM now: a kernel launched behind this one as its programmatic dependent (the suffix
    // pass, which needs nothing this kernel writes) may start as soon as every CTA of this grid has said so.
    // When this grid was itself launched as the programmatic dependent of the append, the suffix pass needs what
    // that kernel wrote: the word is given only once the append grid has completed (a short wait, taken by a
    // thread of a copy-issuing warp whose lanes 8-31 have nothing else to do, while the CTA sets itself up).
    // Launched the ordinary way the wait returns at once.
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  }
  // team T: S at columns [256 T, 256 T + 128), O at [256 T + 128, 256 T + 256)

  // Counters advance identically in every role: `kt` counts K/V tiles, `it_n` counts items with work.
  uint32_t kt = 0, it_n = 0;

  if (warp == 0 || warp >= 2 + kTeams * (kSoftmaxThreads / 32)) {
    // ---------------------------------------------------------------- producers (three warps, all 32 lanes)
    // K/V: a tile is 24 TMA boxes (K: 8 pages x 2 head-dim halves of 2 KB, V: 8 pages of 4 KB).  Issuing a box
    //      costs the issuing warp well over a hundred cycles (measured), so the boxes of a tile are shared out:
    //      warp 0 takes K's first d half, the two extra warps K's second d half and V; 8 boxes from 8 lanes each.
    // Q:   warp 0 also stages the stacked query tile of the NEXT item (plain loads, swizzled stores) into the
    //      other Q buffer while the current item is being computed.
    const int prole = warp == 0 ? 0 : warp - (1 + kTeams * (kSoftmaxThreads / 32));   // 0, 1: K d half; 2: V
    const uint64_t policy = l2_keep_policy();
    bool ok = true;

    auto next_item = [&](int from, Item &out) -> int {
      for (int k = from; k < k_end; ++k) {
        out = decode_item(p, lvs, __ldg(item_list + k), cand_per_tile);
        if (item_has_work(out, cand_per_tile)) return k;
      }
      return k_end;
    };
    // Staging of one query tile (128 rows x 16 chunks of 16 bytes) proceeds in 8 rounds of 8 chunks per
    // lane.  Round i's loads are issued in one call and stored (swizzled) in the next, so that their
    // latency hides behind a K/V tile's worth of other work.
    constexpr int kQRounds = 8;
    uint4 qv[8];
    auto q_load = [&](const Item &qi, int round) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int idx = round * 256 + i * 32 + lane, row = idx >> 4, c = idx & 15;
        const int cand = qi.mt * cand_per_tile + row / g;
        qv[i] = make_uint4(0u, 0u, 0u, 0u);
        if (cand < qi.n_cand) {
          const size_t qrow = (size_t)(qi.b0 + cand) * p.Hq + (size_t)qi.h * g + (row % g);
          qv[i] = __ldg(reinterpret_cast<const uint4 *>(q + qrow * D) + c);
        }
      }
    };
    auto q_store = [&](uint8_t *dst, int round) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int idx = round * 256 + i * 32 + lane, row = idx >> 4, c = idx & 15;
        *reinterpret_cast<uint4 *>(dst + (c >> 3) * kHalfBytes + row * 128 + (((c & 7) ^ (row & 7)) << 4)) = qv[i];
      }
    };
    // One step of staging item `qi` (ordinal n among items with work); `round` runs 0..kQRounds.
    auto q_step = [&](const Item &qi, uint32_t n, int &round) -> bool {
      const int buf = n & 1;
      if (round == 0 && n >= 2) {   // the buffer's previous tenant (item n-2) must have finished its first products
        bool w = mbar_wait(sm, p, &sm.q_free[buf], ((n >> 1) - 1) & 1);
        if (!__all_sync(0xffffffffu, w)) return false;
      }
      if (round > 0) q_store(sm.q[buf], round - 1);
      if (round < kQRounds) q_load(qi, round);
      if (round == kQRounds) {
        fence_async_proxy();
        mbar_arrive(&sm.q_ready[buf]);
      }
      ++round;
      return true;
    };

    Item it, nxt;
    int cur = next_item(k_begin, it);
    // (the query tile of the CTA's first item is staged by the softmax warps, which have nothing else to do yet)
    while (ok && cur < k_end && !sm.abort) {
      const int nxt_idx = next_item(cur + 1, nxt);
      int round = nxt_idx < k_end && prole == 0 ? 0 : kQRounds + 1;   // staging state of the next item's query tile
      for (int seg = 0; seg < 2 && ok; ++seg) {
      const int seg_lo = seg ? it.lo2 : it.lo, seg_hi = seg ? it.hi2 : it.hi;
      const int32_t *seg_pages = seg ? it.pages2 : it.pages;
      if (seg_lo >= seg_hi) continue;
      const int last_pg = (seg_hi - 1) >> 4;
      // Page ids are read 32 at a time (four tiles' worth, one per lane) a block ahead of their use, so that no
      // tile waits for a table look-up.  Pages past the end of the prefix repeat the last valid page: finite
      // data, masked later.
      auto load_ids = [&](int blk) -> int { return __ldg(seg_pages + min((seg_lo >> 4) + blk * 32 + lane, last_pg)); };
      int ids_cur = load_ids(0), ids_next = load_ids(1);
      int tile = 0;
      for (int t0 = seg_lo; t0 < seg_hi; t0 += kTileN, ++kt, ++tile) {
        // lane pg (and every lane with the same low three bits) gets the id of the tile's page pg
        int pid = __shfl_sync(0xffffffffu, ids_cur, (tile & 3) * 8 + (lane & 7));
        if ((tile & 3) == 3) {
          ids_cur = ids_next;
          ids_next = load_ids((tile >> 2) + 2);
        }
        const bool in_range = t0 + (lane & 7) * kPage < seg_hi, good = (unsigned)pid < (unsigned)p.num_pages;
        if (lane < 8 && in_range && !good && prole == 0) latch(p, kDevBadPage);
        if (!good) pid = 0;   // a bad page id is replaced by page 0 and its 16 columns are masked
        const uint32_t okmask = __ballot_sync(0xffffffffu, in_range && good) & 0xffu;
        if (prole < 2) {
          // ---- K(t), d half `prole`: 8 boxes of 2 KB (lanes 0-7: page = lane)
          const int sk = kt % kKSlots;
          ok = mbar_wait(sm, p, &sm.empty_k[sk], ((kt / kKSlots) & 1) ^ 1);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          // page_ok is published before this warp's arrive on full_k; the softmax role reads it after s_full of
          // THIS tile, which follows full_k of this tile
          if (KSCALE && prole == 0) {
            if (lane < 8) sm.kscale[kt & 7][lane] = in_range && good ? __ldg(k_scale + (size_t)pid * p.Hkv + it.h) : 1.f;
            __syncwarp();
          }
          if (lane == 0) {
            if (prole == 0) sm.page_ok[kt & 7] = okmask;
            mbar_expect_tx(&sm.full_k[sk], kHalfBytes);
          }
          __syncwarp();
          if (lane < 8)
            tma_load_half_page(sm.k[sk] + prole * kHalfBytes + lane * (kPageBytes / 2), &k_map, prole * 64,
                               (int)slab_index(p, pid, it.h), &sm.full_k[sk], policy);
        } else {
          // ---- V(t): 8 boxes of 4 KB
          const int sv = kt % kVSlots;
          ok = mbar_wait(sm, p, &sm.empty_v[sv], ((kt / kVSlots) & 1) ^ 1);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          if (lane == 0) mbar_expect_tx(&sm.full_v[sv], kTileBytes);
          __syncwarp();
          if (lane < 8)
            tma_load_page(sm.v[sv] + lane * kPageBytes, &v_map, (int)slab_index(p, pid, it.h), &sm.full_v[sv], policy);
        }
        if (round <= kQRounds) {
          ok = q_step(nxt, it_n + 1, round);
          if (!ok) break;
        }
      }
      }   // token ranges of the item
      while (ok && round <= kQRounds) ok = q_step(nxt, it_n + 1, round);   // short item: finish the staging now
      it = nxt;
      cur = nxt_idx;
      ++it_n;
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      uint32_t team_tiles[kTeams] = {0u, 0u};   // tiles of each team whose P has been taken (all items)
      for (int k = k_begin; k < k_end && !sm.abort; ++k) {
        const Item it = decode_item(p, lvs, __ldg(item_list + k), cand_per_tile);
        if (!item_has_work(it, cand_per_tile)) continue;
        const int qb = it_n & 1;
        if (!mbar_wait(sm, p, &sm.q_ready[qb], (it_n >> 1) & 1)) break;
        ++it_n;
        tc_fence_after();
        const uint64_t q_desc = smem_desc(smem_u32(sm.q[qb]), 16, 1024);
        const int n_tiles = tiles_of(it.lo, it.hi) + tiles_of(it.lo2, it.hi2);
        // Tile t belongs to team t & 1.  Per team the order on the tensor pipe is S(t), O += P(t) V(t), S(t+2), ...:
        // P(t) lies over S(t), so S(t+2) may only follow the second product of tile t; the other team's products
        // fill the gaps.  Products complete in issue order.  The first product of the next item follows this item's
        // last second product directly and runs under this item's epilogue.
        bool ok = true;
        auto issue_qk = [&](int t) -> bool {
          const uint32_t ktq = kt + t;
          const int s = ktq % kKSlots;
          if (!mbar_wait(sm, p, &sm.full_k[s], (ktq / kKSlots) & 1)) return false;
          tc_fence_after();
          const uint32_t tmem_s = tmem + (uint32_t)(t & 1) * 256u;
          // the descriptors of the eight k-steps differ only in the start address field (bytes >> 4, no carry out
          // of its 14 bits: shared memory ends below 256 KB)
          const uint64_t k_desc = smem_desc(smem_u32(sm.k[s]), 16, 1024);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t off = ((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4;
            umma_ss(tmem_s, q_desc + off, k_desc + off, kIdescQK, kk > 0);
          }
          umma_commit(&sm.empty_k[s]);   // K(t) is free as soon as the first product has read it
          umma_commit(&sm.s_full[t & 1]);
          if (t == n_tiles - 1) umma_commit(&sm.q_free[qb]);   // last reader of this item's Q tile
          return true;
        };
        ok = issue_qk(0) && (n_tiles < 2 || issue_qk(1));
        for (int t = 0; t < n_tiles && ok; ++t) {
          const int team = t & 1;
          const uint32_t ktp = kt + t;
          const int s = ktp % kVSlots;
          ok = mbar_wait(sm, p, &sm.p_full[team], team_tiles[team] & 1) &&
               mbar_wait(sm, p, &sm.full_v[s], (ktp / kVSlots) & 1);
          if (!ok) break;
          ++team_tiles[team];
          tc_fence_after();
          const uint32_t tmem_s = tmem + (uint32_t)team * 256u, tmem_o = tmem_s + kTileN;
          const uint64_t v_desc = smem_desc(smem_u32(sm.v[s]), kPageBytes / 2, 1024);
          // one k-step per page: its 16 token rows x both 64-element halves (2 KB apart) are one 4 KB box;
          // the P columns of tokens [64 h, 64 h + 64) start at S column 64 h
#pragma unroll
          for (int kk = 0; kk < kTileN / 16; ++kk)
            umma_ts(tmem_o, tmem_s + (kk >> 2) * 64 + (kk & 3) * 8, v_desc + (uint64_t)((kk * kPageBytes) >> 4), kIdescPV,
                    (t >= kTeams) || (kk > 0));
          umma_commit(&sm.empty_v[s]);
          umma_commit(&sm.pv_done[team]);
          if (t + kTeams < n_tiles) ok = issue_qk(t + kTeams);
        }
        if (!ok) break;
        kt += n_tiles;
      }
    }
  } else {
    // ---------------------------------------------------------------- softmax / epilogue (two teams of 128 threads)
    // One thread owns one row of its team's tile: all 128 scores sit in its registers, so the row maximum and the
    // row sum need no exchange between threads.
    const int team = (warp - 2) >> 2;          // which of the item's two tile streams
    const int quad = warp & 3;                 // TMEM lane quadrant this warp may access
    const int r = quad * 32 + lane;            // row of the tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t tmem_s = tmem + (uint32_t)team * 256u, tmem_o = tmem_s + kTileN;
    uint32_t team_tiles = 0;                   // tiles this team has taken so far (all items)
    uint32_t other_tiles = 0;                  // ... and the other team
    uint32_t both_n = 0;                       // completed meetings of the two teams
    // The CTA's first item with work: its stacked query tile (128 rows x 16 chunks of 16 bytes) is staged here by
    // all 256 softmax threads at once, eight chunks each, instead of by the one producer warp in eight rounds -
    // nothing can start before it is in place.  Later items are staged by the producer under the item before.
    {
      int k0 = k_begin;
      Item qi;
      for (; k0 < k_end; ++k0) {
        qi = decode_item(p, lvs, __ldg(item_list + k0), cand_per_tile);
        if (item_has_work(qi, cand_per_tile)) break;
      }
      if (k0 < k_end) {
        const int tid = threadIdx.x - 64;
        constexpr int kPer = kTileM * 16 / (kTeams * kSoftmaxThreads);
        uint4 qv[kPer];
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
          const int idx = i * (kTeams * kSoftmaxThreads) + tid, row = idx >> 4, c = idx & 15;
          const int cand = qi.mt * cand_per_tile + row / g;
          qv[i] = make_uint4(0u, 0u, 0u, 0u);
          if (cand < qi.n_cand) {
            const size_t qrow = (size_t)(qi.b0 + cand) * p.Hq + (size_t)qi.h * g + (row % g);
            qv[i] = __ldg(reinterpret_cast<const uint4 *>(q + qrow * D) + c);
          }
        }
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
          const int idx = i * (kTeams * kSoftmaxThreads) + tid, row = idx >> 4, c = idx & 15;
          *reinterpret_cast<uint4 *>(sm.q[0] + (c >> 3) * kHalfBytes + row * 128 + (((c & 7) ^ (row & 7)) << 4)) = qv[i];
        }
        fence_async_proxy();
        asm volatile("bar.sync 1, %0;\n" ::"n"(kTeams * kSoftmaxThreads) : "memory");   // the softmax warps only
        if (warp == 2) mbar_arrive(&sm.q_ready[0]);                                       // its 32 arrivals
      }
    }
    for (int k = k_begin; k < k_end && !sm.abort; ++k) {
      const Item it = decode_item(p, lvs, __ldg(item_list + k), cand_per_tile);
      if (it.mt * cand_per_tile >= it.n_cand) continue;
      const int cand = it.mt * cand_per_tile + r / g;
      const bool row_ok = cand < it.n_cand;
      const size_t qrow = (size_t)(it.b0 + cand) * p.Hq + (size_t)it.h * g + (r % g);
      const size_t slot = qrow * p.n_parts + it.part;
      const int n_tiles1 = tiles_of(it.lo, it.hi), n_tiles = n_tiles1 + tiles_of(it.lo2, it.hi2);
      // a chained item answers for the coarser level's part slot of its rows too: it stays empty
      if (!direct && row_ok && team == 0 && it.part2 >= 0) lse_part[qrow * p.n_parts + it.part2] = -INFINITY;
      if (n_tiles == 0) {   // no tokens in this split
        if (direct && row_ok) {   // the row's output is zero, its log-sum-exp -infinity; each team writes 64 columns
          uint4 *dst = reinterpret_cast<uint4 *>(o_final + qrow * D + team * 64);
#pragma unroll
          for (int i = 0; i < 8; ++i) dst[i] = make_uint4(0u, 0u, 0u, 0u);
          if (team == 0) lse_final[qrow] = -INFINITY;
        } else if (row_ok && team == 0) {
          lse_part[slot] = -INFINITY;
        }
        continue;
      }
      const int my_tiles = (n_tiles - team + 1) / kTeams, ot_tiles = n_tiles - my_tiles;   // tiles team, team + 2, ...
      float m = -INFINITY, l = 0.f;   // running maximum in log2 units (already multiplied by sl2) and row sum
      // tokens of the item this row may see: the split's end, or less under a per-candidate limit (causal mask)
      const int hi_row1 = it.limits && row_ok ? min(it.hi, __ldg(it.limits + cand)) : it.hi;
      const int hi_row2 = it.limits2 && row_ok ? min(it.hi2, __ldg(it.limits2 + cand)) : it.hi2;
      bool alive = true;
      for (int t = team; t < n_tiles && alive; t += kTeams, ++team_tiles) {
        const int t0 = t < n_tiles1 ? it.lo + t * kTileN : it.lo2 + (t - n_tiles1) * kTileN;
        const int hi_row = t < n_tiles1 ? hi_row1 : hi_row2;
        alive = mbar_wait(sm, p, &sm.s_full[team], team_tiles & 1);
        alive = __all_sync(0xffffffffu, alive);   // also reconverges the warp before the collective TMEM loads
        if (!alive) break;
        tc_fence_after();
        // which of the tile's 8 pages hold valid data (inside the prefix, page id inside the pool)
        const uint32_t page_ok = sm.page_ok[(kt + t) & 7];
        const bool full_tile = page_ok == 0xffu && t0 + kTileN <= hi_row;
        // per-page factor of the scores in log2 units: softmax scale x the page's K scale (sign of sl2 throughout)
        float ck[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) ck[i] = KSCALE ? sl2 * sm.kscale[(kt + t) & 7][i] : sl2;
        // the whole row of S into registers: four loads in flight, one wait
        uint32_t sv[kTileN];
        auto load_row = [&]() {
#pragma unroll
          for (int c = 0; c < kTileN / 32; ++c)
            tmem_ld32(tmem_s + lane_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[c * 32]));
          tmem_wait_ld();
          if (!full_tile) {   // ragged tail or a bad page: masked scores become -inf (sl2 > 0) / +inf (sl2 < 0)
            const uint32_t masked = __float_as_uint(sl2 >= 0.f ? -INFINITY : INFINITY);
#pragma unroll
            for (int col = 0; col < kTileN; ++col) {
              const bool ok = ((page_ok >> (col >> 4)) & 1u) && (t0 + col < hi_row);
              if (!ok) sv[col] = masked;
            }
          }
        };
        load_row();
        // row extremum of the raw scores; times sl2 it is the row maximum of the scaled scores
        float mx;
        if (!KSCALE) {
          float ext;
          float e8[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) e8[i] = __uint_as_float(sv[i]);
          if (sl2 >= 0.f) {
#pragma unroll
            for (int i = 8; i < kTileN; ++i) e8[i & 7] = fmaxf(e8[i & 7], __uint_as_float(sv[i]));
            ext = fmaxf(fmaxf(fmaxf(e8[0], e8[1]), fmaxf(e8[2], e8[3])), fmaxf(fmaxf(e8[4], e8[5]), fmaxf(e8[6], e8[7])));
          } else {
#pragma unroll
            for (int i = 8; i < kTileN; ++i) e8[i & 7] = fminf(e8[i & 7], __uint_as_float(sv[i]));
            ext = fminf(fminf(fminf(e8[0], e8[1]), fminf(e8[2], e8[3])), fminf(fminf(e8[4], e8[5]), fminf(e8[6], e8[7])));
          }
          mx = (ext == INFINITY || ext == -INFINITY) ? -INFINITY : ext * sl2;   // all masked -> -inf
        } else {
          // every page has a factor of its own: the extremum of each page's 16 raw scores, scaled, then the maximum
          mx = -INFINITY;
#pragma unroll
          for (int pg = 0; pg < 8; ++pg) {
            float e4[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) e4[i] = __uint_as_float(sv[16 * pg + i]);
            if (sl2 >= 0.f) {
#pragma unroll
              for (int i = 4; i < 16; ++i) e4[i & 3] = fmaxf(e4[i & 3], __uint_as_float(sv[16 * pg + i]));
              e4[0] = fmaxf(fmaxf(e4[0], e4[1]), fmaxf(e4[2], e4[3]));
            } else {
#pragma unroll
              for (int i = 4; i < 16; ++i) e4[i & 3] = fminf(e4[i & 3], __uint_as_float(sv[16 * pg + i]));
              e4[0] = fminf(fminf(e4[0], e4[1]), fminf(e4[2], e4[3]));
            }
            if (e4[0] != INFINITY && e4[0] != -INFINITY) mx = fmaxf(mx, e4[0] * ck[pg]);   // (all 16 masked: skipped)
          }
        }
        // The running maximum moves only when the new one is clearly larger (2^8): P stays bounded by
        // 2^8 and the accumulator in TMEM is rescaled rarely.
        float m_use = m;
        bool rescale = false;
        if (mx > m + 8.f) {
          m_use = mx;
          rescale = t >= kTeams && m > -INFINITY;
        }
        const float alpha = rescale ? fast_exp2(m - m_use) : 1.f;
        if (__any_sync(0xffffffffu, rescale)) {
          // every earlier product into this team's O must have completed before O is rescaled in place
          alive = mbar_wait(sm, p, &sm.pv_done[team], (team_tiles - 1) & 1);
          alive = __all_sync(0xffffffffu, alive);
          if (!alive) break;
          tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {   // this row of O
            uint32_t v[32];
            tmem_ld32(tmem_o + lane_addr + c * 32, v);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
            tmem_st32(tmem_o + lane_addr + c * 32, v);
          }
          tmem_wait_st();
          load_row();   // the scores are read again rather than kept across this rare path
        }
        l *= alpha;
        m = m_use;
        const float neg_m = m == -INFINITY ? 0.f : -m;
        // P goes to TMEM as the A operand of the second product: lane = row, one column per token pair, written
        // over S (all of it is in registers by now; the team's next first product, which overwrites S, is issued
        // after the second product that reads this P).  Tokens [64 h + 32 c, +32) go to columns [64 h + 16 c, +16).
        float lsum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c = 0; c < kTileN / 32; ++c) {
          uint32_t pw[16];                 // 32 tokens -> 16 packed columns
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float cf = ck[(c * 32 + 2 * j) >> 4];
            const float p0 = fast_exp2(fmaf(__uint_as_float(sv[c * 32 + 2 * j]), cf, neg_m));       // masked: exp2(-inf) = 0
            const float p1 = fast_exp2(fmaf(__uint_as_float(sv[c * 32 + 2 * j + 1]), cf, neg_m));
            lsum[j & 1] += p0;
            lsum[2 + (j & 1)] += p1;
            pw[j] = pack_bf16x2(p0, p1);
          }
          tmem_st16(tmem_s + lane_addr + (c >> 1) * 64 + (c & 1) * 16, pw);
        }
        l += (lsum[0] + lsum[1]) + (lsum[2] + lsum[3]);
        tmem_wait_st();
        tc_fence_before();
        // p_full counts arrivals, not tiles; no thread can arrive for the team's next tile before this phase
        // closes, because that tile's S follows the product that waits for this phase.
        mbar_arrive(&sm.p_full[team]);
      }
      kt += n_tiles;
      other_tiles += ot_tiles;
      if (!alive) break;
      // ---- epilogue: the two streams of the item are merged here, so the item writes one part.
      // Both teams publish (m, l) of every row and meet.
      const float l_row = l;
      sm.xch[team][0][r] = m;
      sm.xch[team][1][r] = l_row;
      auto teams_meet = [&]() -> bool {
        mbar_arrive(&sm.both);
        bool w = mbar_wait(sm, p, &sm.both, both_n & 1);
        ++both_n;
        return __all_sync(0xffffffffu, w);
      };
      alive = teams_meet();
      if (!alive) break;
      const float m_o = sm.xch[team ^ 1][0][r], l_o = sm.xch[team ^ 1][1][r];
      // weights of the two streams in log2 units: exp2(m_T - max) l_T; a stream without tiles or without an
      // unmasked token in this row has weight 0 and its accumulator is not read
      const bool have_me = my_tiles > 0, have_ot = ot_tiles > 0;
      const float m_all = fmaxf(have_me && l_row > 0.f ? m : -INFINITY, have_ot && l_o > 0.f ? m_o : -INFINITY);
      const float a_me = have_me && l_row > 0.f ? fast_exp2(m - m_all) : 0.f;
      const float a_ot = have_ot && l_o > 0.f ? fast_exp2(m_o - m_all) : 0.f;
      const float l_all = a_me * l_row + a_ot * l_o;
      if (have_me) alive = mbar_wait(sm, p, &sm.pv_done[team], (team_tiles - 1) & 1);
      if (have_ot) alive = alive && mbar_wait(sm, p, &sm.pv_done[team ^ 1], (other_tiles - 1) & 1);
      if (!__all_sync(0xffffffffu, alive)) break;
      tc_fence_after();
      const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
      // Each of the row's two threads takes 64 of the 128 output columns, [64 team, +64), 32 at a time.  A thread
      // holds 32 columns (128 bytes) of ONE row; a store instruction issued like that touches 32 rows, 16 bytes of
      // each, which costs the store path 32 cycles an instruction and leaves sectors half written.  So each group
      // of 8 lanes first transposes its 8 rows x 8 pieces of 16 bytes (48 shuffles); a store instruction then
      // writes 4 rows, 128 contiguous bytes of each.
      const uint32_t store_mask = __ballot_sync(0xffffffffu, row_ok && (direct || l_all > 0.f));
      const float w_me = a_me * inv, w_ot = a_ot * inv;
#pragma unroll 1
      for (int cc = 0; cc < 2; ++cc) {
        const int col0 = team * 64 + cc * 32;
        const unsigned long long my_off = (unsigned long long)(direct ? qrow : slot) * D + col0;
        uint32_t v[32];
        if (have_me) {
          tmem_ld32(tmem_o + lane_addr + col0, v);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * w_me);
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = 0u;
        }
        if (have_ot) {
          uint32_t w[32];
          tmem_ld32(tmem + (uint32_t)(team ^ 1) * 256u + kTileN + lane_addr + col0, w);   // the other team's accumulator
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(fmaf(__uint_as_float(w[i]), w_ot, __uint_as_float(v[i])));
        }
        // transpose 8 x 8 blocks of 16-byte pieces inside each group of 8 lanes
#pragma unroll
        for (int s = 4; s >= 1; s >>= 1) {
          const bool up = (lane & s) != 0;
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            if (k & s) continue;
#pragma unroll
            for (int w = 0; w < 4; ++w) {
              const uint32_t send = up ? v[4 * k + w] : v[4 * (k | s) + w];
              const uint32_t got = __shfl_xor_sync(0xffffffffu, send, s);
              if (up) v[4 * k + w] = got; else v[4 * (k | s) + w] = got;
            }
          }
        }
        // piece k of this lane now is (row 8 (lane / 8) + k of this warp's 32 rows, columns col0 + 4 (lane % 8) ...)
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int src = (lane & 24) + k;
          const unsigned long long off = __shfl_sync(0xffffffffu, my_off, src);
          if (!((store_mask >> src) & 1u)) continue;
          if (direct)
            *reinterpret_cast<uint2 *>(o_final + off + 4 * (lane & 7)) =
                make_uint2(pack_bf16x2(__uint_as_float(v[4 * k]), __uint_as_float(v[4 * k + 1])),
                           pack_bf16x2(__uint_as_float(v[4 * k + 2]), __uint_as_float(v[4 * k + 3])));
          else
            *reinterpret_cast<float4 *>(o_part + off + 4 * (lane & 7)) =
                make_float4(__uint_as_float(v[4 * k]), __uint_as_float(v[4 * k + 1]), __uint_as_float(v[4 * k + 2]),
                            __uint_as_float(v[4 * k + 3]));
        }
      }
      if (row_ok && team == 0) (direct ? lse_final[qrow] : lse_part[slot]) = l_all > 0.f ? (m_all + log2f(l_all)) * kLn2 : -INFINITY;
      tc_fence_before();
      // nobody goes on (to overwrite an accumulator or an exchange slot) before everybody has read both
      alive = teams_meet();
      if (!alive) break;
    }
  }

  // ------------------------------------------------------------------ teardown
  if (sm.abort && warp == 0 && lane == 0) {
    // give copies that are still in flight a bounded time to land before the CTA's shared memory goes away
    const long long t0 = clock64();
    while (clock64() - t0 < kDrainCycles) { }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

static_assert(sizeof(Smem) <= 232448, "shared memory of one CTA");

// ================================================================================================
// Row-pair variant.  Where a (group, kv head) has at least two 128-row tiles of stacked queries, an item covers
// TWO of them and the CTA's two teams are the two row tiles: every K/V tile is copied into shared memory once and
// read by both teams' products (half the copies and half the L2 reads of the variant above, where each row tile
// streams the K/V tiles on its own), an item is twice as long (half the per-item cost), and each team owns its rows
// from the first product to the stores (no merging of two streams in the epilogue).  The query tiles arrive by TMA
// through a tensor map laid over q (box = 128 / g candidates x g heads x 64 elements, which IS the stacked row
// order), so no thread stages them.  Per team the order on the tensor pipe is the same chain as above - S(t),
// O += P(t) V(t), S(t+1) - and the other team's products fill the gaps.  With per-candidate limits (scoring) the
// teams see different numbers of tiles; a tile's slot is released by the product of its last user.
// ================================================================================================
struct __align__(1024) SmemRp {
  uint8_t q[kTeams][kTileBytes];      // team T's stacked query tile, [d half][128 rows][64], 128-byte swizzle
  uint8_t k[kKSlots][kTileBytes];
  uint8_t v[kVSlots][kTileBytes];
  uint64_t full_k[kKSlots], empty_k[kKSlots], full_v[kVSlots], empty_v[kVSlots];
  uint64_t q_full[kTeams], q_free[kTeams], s_full[kTeams], p_full[kTeams], pv_done[kTeams];
  uint32_t page_ok[8];
  float kscale[8][8];
  uint32_t tmem_base;
  volatile int abort;
  long long wait_cycles;
};

__device__ __forceinline__ bool mbar_wait_rp(SmemRp &sm, const Params &p, uint64_t *bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    __nanosleep(32);
    if (sm.abort) return false;
    if (clock64() - t0 > sm.wait_cycles) {
      sm.abort = 1;
      latch(p, kDevTimeout);
      return false;
    }
  }
}

// One d half (64 elements) of a stacked query tile: 128 / g candidates x g heads x 64 elements, 16 KB.
__device__ __forceinline__ void tma_load_q_half(void *dst, const CUtensorMap *map, int x, int head, int cand,
                                                uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];\n"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(head), "r"(cand), "r"(smem_u32(bar))
      : "memory");
}

// What one team (row tile 2 mp + T of the item's pair) sees of the item.
struct TeamView {
  bool rows;        // the row tile has candidates
  int hi1, hi2;     // ends of the two token ranges for this tile's rows (its last candidate's limits applied)
  int n1, n2;       // its tiles in the two ranges
};
__device__ __forceinline__ TeamView team_view(const Item &u, int T, int cand_per_tile) {
  TeamView v;
  const int first = (2 * u.mt + T) * cand_per_tile;
  v.rows = first < u.n_cand;
  const int last = min(first + cand_per_tile, u.n_cand) - 1;
  v.hi1 = u.hi;
  v.hi2 = u.hi2;
  if (v.rows && u.limits) v.hi1 = min(v.hi1, max(__ldg(u.limits + last), 0));
  if (v.rows && u.limits2) v.hi2 = min(v.hi2, max(__ldg(u.limits2 + last), 0));
  v.n1 = v.rows ? tiles_of(u.lo, v.hi1) : 0;
  v.n2 = v.rows ? tiles_of(u.lo2, v.hi2) : 0;
  return v;
}

template <bool KSCALE>
__global__ void __maxnreg__(168)
prefix_rp_kernel(Params p, const __grid_constant__ TcLevels lvs, const __grid_constant__ CUtensorMap k_map,
                 const __grid_constant__ CUtensorMap v_map, const __grid_constant__ CUtensorMap q_map, float sl2,
                 float *__restrict__ o_part, float *__restrict__ lse_part, const int32_t *__restrict__ item_list,
                 const int32_t *__restrict__ cta_begin, __nv_bfloat16 *__restrict__ o_final,
                 float *__restrict__ lse_final, long long wait_cycles, const float *__restrict__ k_scale) {
  const bool direct = o_final != nullptr;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  SmemRp &sm = *reinterpret_cast<SmemRp *>(smem_raw);
  if ((smem_u32(smem_raw) & 1023u) != 0) {
    if (threadIdx.x == 0) latch(p, MC_ERR_CUDA);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = p.g, cand_per_tile = kTileM / g, cand_per_unit = 2 * cand_per_tile;
  const int k_begin = __ldg(cta_begin + blockIdx.x), k_end = __ldg(cta_begin + blockIdx.x + 1);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kKSlots; ++s) {
      mbar_init(&sm.full_k[s], 2);
      mbar_init(&sm.empty_k[s], 1);
    }
    for (int s = 0; s < kVSlots; ++s) {
      mbar_init(&sm.full_v[s], 1);
      mbar_init(&sm.empty_v[s], 1);
    }
    for (int t = 0; t < kTeams; ++t) {
      mbar_init(&sm.q_full[t], 1);
      mbar_init(&sm.q_free[t], 1);
      mbar_init(&sm.s_full[t], 1);
      mbar_init(&sm.p_full[t], kSoftmaxThreads);
      mbar_init(&sm.pv_done[t], 1);
    }
    sm.abort = 0;
    sm.wait_cycles = wait_cycles;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&sm.tmem_base)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  if (threadIdx.x == kThreads - 1) {   // (see the kernel above: the append's completion, then the word to the suffix pass)
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  }

  // `kt` counts the K/V tiles of the CTA's stream (an item adds the tiles of the union of its two teams' ranges);
  // every role advances it alike.
  uint32_t kt = 0;

  if (warp == 0 || warp >= 2 + kTeams * (kSoftmaxThreads / 32)) {
    // ---------------------------------------------------------------- producers (three warps)
    const int prole = warp == 0 ? 0 : warp - (1 + kTeams * (kSoftmaxThreads / 32));   // 0, 1: K d half; 2: V
    const uint64_t policy = l2_keep_policy();
    bool ok = true;
    uint32_t q_n[kTeams] = {0u, 0u};   // items in which each team had tiles
    for (int k = k_begin; k < k_end && ok && !sm.abort; ++k) {
      const Item u = decode_item(p, lvs, __ldg(item_list + k), cand_per_unit);
      const TeamView tv0 = team_view(u, 0, cand_per_tile), tv1 = team_view(u, 1, cand_per_tile);
      const int n1 = max(tv0.n1, tv1.n1), n2 = max(tv0.n2, tv1.n2);
      if (n1 + n2 == 0) continue;
      // the teams' query tiles: two boxes each, as soon as the tile's previous tenant has been read for the last time
      if (prole == 0) {
#pragma unroll
        for (int T = 0; T < kTeams; ++T) {
          if (!ok || (T ? tv1.n1 + tv1.n2 : tv0.n1 + tv0.n2) == 0) continue;
          if (q_n[T] > 0) {
            ok = mbar_wait_rp(sm, p, &sm.q_free[T], (q_n[T] - 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) continue;
          }
          if (lane == 0) {
            mbar_expect_tx(&sm.q_full[T], kTileBytes);
            const int cand0 = u.b0 + (2 * u.mt + T) * cand_per_tile;
            tma_load_q_half(sm.q[T], &q_map, 0, u.h * g, cand0, &sm.q_full[T]);
            tma_load_q_half(sm.q[T] + kHalfBytes, &q_map, 64, u.h * g, cand0, &sm.q_full[T]);
          }
          ++q_n[T];
        }
        if (!ok) break;
      }
      for (int seg = 0; seg < 2 && ok; ++seg) {
        const int seg_lo = seg ? u.lo2 : u.lo;
        const int seg_hi = seg ? max(tv0.hi2, tv1.hi2) : max(tv0.hi1, tv1.hi1);
        const int32_t *seg_pages = seg ? u.pages2 : u.pages;
        if ((seg ? n2 : n1) == 0) continue;
        const int last_pg = (seg_hi - 1) >> 4;
        auto load_ids = [&](int blk) -> int { return __ldg(seg_pages + min((seg_lo >> 4) + blk * 32 + lane, last_pg)); };
        int ids_cur = load_ids(0), ids_next = load_ids(1);
        int tile = 0;
        for (int t0 = seg_lo; t0 < seg_hi; t0 += kTileN, ++kt, ++tile) {
          int pid = __shfl_sync(0xffffffffu, ids_cur, (tile & 3) * 8 + (lane & 7));
          if ((tile & 3) == 3) {
            ids_cur = ids_next;
            ids_next = load_ids((tile >> 2) + 2);
          }
          const bool in_range = t0 + (lane & 7) * kPage < seg_hi, good = (unsigned)pid < (unsigned)p.num_pages;
          if (lane < 8 && in_range && !good && prole == 0) latch(p, kDevBadPage);
          if (!good) pid = 0;
          const uint32_t okmask = __ballot_sync(0xffffffffu, in_range && good) & 0xffu;
          if (prole < 2) {
            const int sk = kt % kKSlots;
            ok = mbar_wait_rp(sm, p, &sm.empty_k[sk], ((kt / kKSlots) & 1) ^ 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (KSCALE && prole == 0) {
              if (lane < 8) sm.kscale[kt & 7][lane] = in_range && good ? __ldg(k_scale + (size_t)pid * p.Hkv + u.h) : 1.f;
              __syncwarp();
            }
            if (lane == 0) {
              if (prole == 0) sm.page_ok[kt & 7] = okmask;
              mbar_expect_tx(&sm.full_k[sk], kHalfBytes);
            }
            __syncwarp();
            if (lane < 8)
              tma_load_half_page(sm.k[sk] + prole * kHalfBytes + lane * (kPageBytes / 2), &k_map, prole * 64,
                                 (int)slab_index(p, pid, u.h), &sm.full_k[sk], policy);
          } else {
            const int sv = kt % kVSlots;
            ok = mbar_wait_rp(sm, p, &sm.empty_v[sv], ((kt / kVSlots) & 1) ^ 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (lane == 0) mbar_expect_tx(&sm.full_v[sv], kTileBytes);
            __syncwarp();
            if (lane < 8)
              tma_load_page(sm.v[sv] + lane * kPageBytes, &v_map, (int)slab_index(p, pid, u.h), &sm.full_v[sv], policy);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      uint32_t tt0 = 0u, tt1 = 0u;   // tiles of each team whose P has been taken (all items)
      uint32_t qn0 = 0u, qn1 = 0u;   // items in which each team had tiles
      for (int k = k_begin; k < k_end && !sm.abort; ++k) {
        const Item u = decode_item(p, lvs, __ldg(item_list + k), cand_per_unit);
        const TeamView tv0 = team_view(u, 0, cand_per_tile), tv1 = team_view(u, 1, cand_per_tile);
        const int n1 = max(tv0.n1, tv1.n1), n_all = n1 + max(tv0.n2, tv1.n2);
        if (n_all == 0) continue;
        // The products follow the CTA's K/V stream tile by tile: at tile t, for each team that uses it, the second
        // product of t and then that team's first product of tile t + 1 (so a team's chain is S, P V, S, ... as in the
        // kernel above and no product ever asks for a tile outside the slots in flight).  Team 1 is issued after
        // team 0, so a tile's last user is team 1 where it uses the tile.
        const int n1_0 = tv0.n1, n2_0 = tv0.n2, n1_1 = tv1.n1, n2_1 = tv1.n2;
        auto uses0 = [&](int t) -> bool { return t < n1 ? t < n1_0 : t - n1 < n2_0; };
        auto uses1 = [&](int t) -> bool { return t < n1 ? t < n1_1 : t - n1 < n2_1; };
        const int cnt0 = n1_0 + n2_0, cnt1 = n1_1 + n2_1;
        int s_left0 = cnt0, s_left1 = cnt1, pv0 = 0, pv1 = 0;   // first products still to issue; second products issued
        bool ok = true;
        uint64_t q_desc0 = 0, q_desc1 = 0;
        if (cnt0 > 0) {
          ok = mbar_wait_rp(sm, p, &sm.q_full[0], qn0 & 1);
          ++qn0;
          q_desc0 = smem_desc(smem_u32(sm.q[0]), 16, 1024);
        }
        if (ok && cnt1 > 0) {
          ok = mbar_wait_rp(sm, p, &sm.q_full[1], qn1 & 1);
          ++qn1;
          q_desc1 = smem_desc(smem_u32(sm.q[1]), 16, 1024);
        }
        if (!ok) break;
        tc_fence_after();
        // first product of team T (compile-time) on stream tile t
        auto issue_qk = [&](auto Tc, int t, bool last_user, bool last_of_team) -> bool {
          constexpr int T = decltype(Tc)::value;
          const uint32_t ktq = kt + t;
          const int s = ktq % kKSlots;
          if (!mbar_wait_rp(sm, p, &sm.full_k[s], (ktq / kKSlots) & 1)) return false;
          tc_fence_after();
          const uint32_t tmem_s = tmem + (uint32_t)T * 256u;
          const uint64_t k_desc = smem_desc(smem_u32(sm.k[s]), 16, 1024), q_desc = T ? q_desc1 : q_desc0;
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t off = ((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4;
            umma_ss(tmem_s, q_desc + off, k_desc + off, kIdescQK, kk > 0);
          }
          if (last_user) umma_commit(&sm.empty_k[s]);   // K(t) is free once its last user's product has read it
          umma_commit(&sm.s_full[T]);
          if (last_of_team) umma_commit(&sm.q_free[T]);  // last reader of this team's query tile
          return true;
        };
        auto issue_pv = [&](auto Tc, int t, bool first_of_team, bool last_user, uint32_t done_before) -> bool {
          constexpr int T = decltype(Tc)::value;
          const uint32_t ktp = kt + t;
          const int s = ktp % kVSlots;
          if (!(mbar_wait_rp(sm, p, &sm.p_full[T], done_before & 1) &&
                mbar_wait_rp(sm, p, &sm.full_v[s], (ktp / kVSlots) & 1)))
            return false;
          tc_fence_after();
          const uint32_t tmem_s = tmem + (uint32_t)T * 256u, tmem_o = tmem_s + kTileN;
          const uint64_t v_desc = smem_desc(smem_u32(sm.v[s]), kPageBytes / 2, 1024);
#pragma unroll
          for (int kk = 0; kk < kTileN / 16; ++kk)
            umma_ts(tmem_o, tmem_s + (kk >> 2) * 64 + (kk & 3) * 8, v_desc + (uint64_t)((kk * kPageBytes) >> 4), kIdescPV,
                    !first_of_team || (kk > 0));
          if (last_user) umma_commit(&sm.empty_v[s]);
          umma_commit(&sm.pv_done[T]);
          return true;
        };
        using T0 = std::integral_constant<int, 0>;
        using T1 = std::integral_constant<int, 1>;
        // (both teams use stream tile 0 unless a team's first range is empty; the general rule covers it)
        if (uses0(0)) ok = issue_qk(T0{}, 0, !uses1(0), --s_left0 == 0);
        if (ok && uses1(0)) ok = issue_qk(T1{}, 0, true, --s_left1 == 0);
        for (int t = 0; t < n_all && ok; ++t) {
          const bool u0 = uses0(t), u1 = uses1(t), nx = t + 1 < n_all;
          const bool v0 = nx && uses0(t + 1), v1 = nx && uses1(t + 1);
          if (u0) {
            ok = issue_pv(T0{}, t, pv0 == 0, !u1, tt0);
            ++tt0;
            ++pv0;
          }
          if (ok && v0) ok = issue_qk(T0{}, t + 1, !v1, --s_left0 == 0);
          if (ok && u1) {
            ok = issue_pv(T1{}, t, pv1 == 0, true, tt1);
            ++tt1;
            ++pv1;
          }
          if (ok && v1) ok = issue_qk(T1{}, t + 1, true, --s_left1 == 0);
        }
        if (!ok) break;
        kt += n_all;
      }
    }
  } else {
    // ---------------------------------------------------------------- softmax / epilogue: team T = row tile 2 mp + T
    const int team = (warp - 2) >> 2;
    const int quad = warp & 3;
    const int r = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t tmem_s = tmem + (uint32_t)team * 256u, tmem_o = tmem_s + kTileN;
    uint32_t team_tiles = 0;
    for (int k = k_begin; k < k_end && !sm.abort; ++k) {
      const Item u = decode_item(p, lvs, __ldg(item_list + k), cand_per_unit);
      const TeamView me = team_view(u, team, cand_per_tile), other = team_view(u, team ^ 1, cand_per_tile);
      const int n1 = max(me.n1, other.n1), n_all = n1 + max(me.n2, other.n2);
      if (me.rows) {
        const int cand = (2 * u.mt + team) * cand_per_tile + r / g;
        const bool row_ok = cand < u.n_cand;
        const size_t qrow = (size_t)(u.b0 + cand) * p.Hq + (size_t)u.h * g + (r % g);
        const size_t slot = qrow * p.n_parts + u.part;
        if (!direct && row_ok && u.part2 >= 0) lse_part[qrow * p.n_parts + u.part2] = -INFINITY;
        const int my_tiles = me.n1 + me.n2;
        if (my_tiles == 0) {   // no tokens for these rows in this split
          if (direct && row_ok) {
            uint4 *dst = reinterpret_cast<uint4 *>(o_final + qrow * D);
#pragma unroll
            for (int i = 0; i < 16; ++i) dst[i] = make_uint4(0u, 0u, 0u, 0u);
            lse_final[qrow] = -INFINITY;
          } else if (row_ok) {
            lse_part[slot] = -INFINITY;
          }
        } else {
          float m = -INFINITY, l = 0.f;
          const int hi_row1 = u.limits && row_ok ? min(me.hi1, __ldg(u.limits + cand)) : me.hi1;
          const int hi_row2 = u.limits2 && row_ok ? min(me.hi2, __ldg(u.limits2 + cand)) : me.hi2;
          bool alive = true;
          for (int c = 0; c < my_tiles && alive; ++c, ++team_tiles) {
            const int t = c < me.n1 ? c : n1 + (c - me.n1);                  // tile of the CTA's K/V stream
            const int t0 = c < me.n1 ? u.lo + c * kTileN : u.lo2 + (c - me.n1) * kTileN;
            const int hi_row = c < me.n1 ? hi_row1 : hi_row2;
            alive = mbar_wait_rp(sm, p, &sm.s_full[team], team_tiles & 1);
            alive = __all_sync(0xffffffffu, alive);
            if (!alive) break;
            tc_fence_after();
            const uint32_t page_ok = sm.page_ok[(kt + t) & 7];
            const bool full_tile = page_ok == 0xffu && t0 + kTileN <= hi_row;
            float ck[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) ck[i] = KSCALE ? sl2 * sm.kscale[(kt + t) & 7][i] : sl2;
            uint32_t sv[kTileN];
            auto load_row = [&]() {
#pragma unroll
              for (int cc = 0; cc < kTileN / 32; ++cc)
                tmem_ld32(tmem_s + lane_addr + cc * 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[cc * 32]));
              tmem_wait_ld();
              if (!full_tile) {
                const uint32_t masked = __float_as_uint(sl2 >= 0.f ? -INFINITY : INFINITY);
#pragma unroll
                for (int col = 0; col < kTileN; ++col) {
                  const bool okc = ((page_ok >> (col >> 4)) & 1u) && (t0 + col < hi_row);
                  if (!okc) sv[col] = masked;
                }
              }
            };
            load_row();
            float mx = -INFINITY;
#pragma unroll
            for (int pg = 0; pg < 8; ++pg) {
              float e4[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) e4[i] = __uint_as_float(sv[16 * pg + i]);
              if (sl2 >= 0.f) {
#pragma unroll
                for (int i = 4; i < 16; ++i) e4[i & 3] = fmaxf(e4[i & 3], __uint_as_float(sv[16 * pg + i]));
                e4[0] = fmaxf(fmaxf(e4[0], e4[1]), fmaxf(e4[2], e4[3]));
              } else {
#pragma unroll
                for (int i = 4; i < 16; ++i) e4[i & 3] = fminf(e4[i & 3], __uint_as_float(sv[16 * pg + i]));
                e4[0] = fminf(fminf(e4[0], e4[1]), fminf(e4[2], e4[3]));
              }
              if (e4[0] != INFINITY && e4[0] != -INFINITY) mx = fmaxf(mx, e4[0] * ck[pg]);
            }
            float m_use = m;
            bool rescale = false;
            if (mx > m + 8.f) {
              m_use = mx;
              rescale = c > 0 && m > -INFINITY;
            }
            const float alpha = rescale ? fast_exp2(m - m_use) : 1.f;
            if (__any_sync(0xffffffffu, rescale)) {
              alive = mbar_wait_rp(sm, p, &sm.pv_done[team], (team_tiles - 1) & 1);
              alive = __all_sync(0xffffffffu, alive);
              if (!alive) break;
              tc_fence_after();
#pragma unroll 1
              for (int cc = 0; cc < D / 32; ++cc) {
                uint32_t v[32];
                tmem_ld32(tmem_o + lane_addr + cc * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
                tmem_st32(tmem_o + lane_addr + cc * 32, v);
              }
              tmem_wait_st();
              load_row();
            }
            l *= alpha;
            m = m_use;
            const float neg_m = m == -INFINITY ? 0.f : -m;
            float lsum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int cc = 0; cc < kTileN / 32; ++cc) {
              uint32_t pw[16];
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                const float cf = ck[(cc * 32 + 2 * j) >> 4];
                const float p0 = fast_exp2(fmaf(__uint_as_float(sv[cc * 32 + 2 * j]), cf, neg_m));
                const float p1 = fast_exp2(fmaf(__uint_as_float(sv[cc * 32 + 2 * j + 1]), cf, neg_m));
                lsum[j & 1] += p0;
                lsum[2 + (j & 1)] += p1;
                pw[j] = pack_bf16x2(p0, p1);
              }
              tmem_st16(tmem_s + lane_addr + (cc >> 1) * 64 + (cc & 1) * 16, pw);
            }
            l += (lsum[0] + lsum[1]) + (lsum[2] + lsum[3]);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&sm.p_full[team]);
          }
          if (!alive) break;
          // ---- epilogue of this team's rows: its own accumulator, nothing to merge
          alive = mbar_wait_rp(sm, p, &sm.pv_done[team], (team_tiles - 1) & 1);
          if (!__all_sync(0xffffffffu, alive)) break;
          tc_fence_after();
          const float inv = l > 0.f ? 1.f / l : 0.f;
          const uint32_t store_mask = __ballot_sync(0xffffffffu, row_ok && (direct || l > 0.f));
#pragma unroll 1
          for (int cc = 0; cc < D / 32; ++cc) {
            const int col0 = cc * 32;
            const unsigned long long my_off = (unsigned long long)(direct ? qrow : slot) * D + col0;
            uint32_t v[32];
            tmem_ld32(tmem_o + lane_addr + col0, v);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * inv);
#pragma unroll
            for (int s = 4; s >= 1; s >>= 1) {   // transpose 8 x 8 blocks of 16-byte pieces inside each group of 8 lanes
              const bool up = (lane & s) != 0;
#pragma unroll
              for (int kk = 0; kk < 8; ++kk) {
                if (kk & s) continue;
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                  const uint32_t send = up ? v[4 * kk + w] : v[4 * (kk | s) + w];
                  const uint32_t got = __shfl_xor_sync(0xffffffffu, send, s);
                  if (up) v[4 * kk + w] = got; else v[4 * (kk | s) + w] = got;
                }
              }
            }
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              const int src = (lane & 24) + kk;
              const unsigned long long off = __shfl_sync(0xffffffffu, my_off, src);
              if (!((store_mask >> src) & 1u)) continue;
              if (direct)
                *reinterpret_cast<uint2 *>(o_final + off + 4 * (lane & 7)) =
                    make_uint2(pack_bf16x2(__uint_as_float(v[4 * kk]), __uint_as_float(v[4 * kk + 1])),
                               pack_bf16x2(__uint_as_float(v[4 * kk + 2]), __uint_as_float(v[4 * kk + 3])));
              else
                *reinterpret_cast<float4 *>(o_part + off + 4 * (lane & 7)) =
                    make_float4(__uint_as_float(v[4 * kk]), __uint_as_float(v[4 * kk + 1]), __uint_as_float(v[4 * kk + 2]),
                                __uint_as_float(v[4 * kk + 3]));
            }
          }
          if (row_ok) (direct ? lse_final[qrow] : lse_part[slot]) = l > 0.f ? (m + log2f(l)) * kLn2 : -INFINITY;
          tc_fence_before();
        }
      }
      kt += n_all;
    }
  }

  // ------------------------------------------------------------------ teardown
  if (sm.abort && warp == 0 && lane == 0) {
    const long long t0 = clock64();
    while (clock64() - t0 < kDrainCycles) { }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

static_assert(sizeof(SmemRp) <= 232448, "shared memory of one CTA");

}  // namespace

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool encode_pool_map(CUtensorMap *map, const void *pool, int num_pages, int Hkv, bool whole_page) {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !sym)
      return false;
    fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  // The pool is a sequence of 16-token slabs of 16 x 128 elements (num_pages counts 16-token unit pages, so there
  // are num_pages * Hkv of them, whatever the cache's page size).  V: a slab seen as [token][d half][64]; dimensions
  // innermost first, with the half before the token so that a box lands as [d half][16 tokens][64 elements].
  const cuuint64_t n_slabs = (cuuint64_t)num_pages * (cuuint64_t)Hkv;
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  if (!whole_page) {   // K: one box = 64 elements x 16 tokens of one slab
    const cuuint64_t dims3[3] = {(cuuint64_t)D, (cuuint64_t)kPage, n_slabs};
    const cuuint64_t strides3[2] = {(cuuint64_t)D * 2, (cuuint64_t)kPage * D * 2};
    const cuuint32_t box3[3] = {64, (cuuint32_t)kPage, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(pool), dims3, strides3, box3, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  }
  const cuuint64_t dims[4] = {64, (cuuint64_t)kPage, 2, n_slabs};
  const cuuint64_t strides[3] = {(cuuint64_t)D * 2, 128, (cuuint64_t)kPage * D * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)kPage, 2, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(pool), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Both pools in one map: the (page, kv head) slabs of the pool at the lower address and, `distance` bytes above
// each, the same slab of the other pool.  One 8 KB box = [pool][d half][16 tokens][64] of one (page, kv head).
bool encode_kv_pair_map(CUtensorMap *map, const void *lower_pool, unsigned long long distance, int num_pages, int Hkv) {
  if (distance == 0 || (distance & 15ull) != 0 || distance >= (1ull << 40)) return false;
  void *sym = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !sym)
    return false;
  EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(sym);
  const cuuint64_t dims[5] = {64, (cuuint64_t)kPage, 2, (cuuint64_t)num_pages * (cuuint64_t)Hkv, 2};
  const cuuint64_t strides[4] = {(cuuint64_t)D * 2, 128, (cuuint64_t)kPage * D * 2, (cuuint64_t)distance};
  const cuuint32_t box[5] = {64, (cuuint32_t)kPage, 2, 1, 2};
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(lower_pool), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// q [B][Hq][128] (bf16) as boxes of 128 / g candidates x g heads x 64 elements, 128-byte swizzle.
bool encode_q_map(CUtensorMap *map, const void *q, int B, int Hq, int g) {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !sym)
      return false;
    fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)Hq, (cuuint64_t)B};
  const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)Hq * D * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)g, (cuuint32_t)(kTileM / g)};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(q), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct PrefixTcPlan {
  CUtensorMap k_map, v_map;
  TcLevels levels;
  int n_items, grid;
  bool one_part_per_row;   // every row gets exactly one part from this pass: one single-split level, or two chained
  long long wait_cycles;   // limit of every device-side wait
  const float *k_scale;    // non-null: the pools are an expanded e4m3 cache, one K scale per (page, kv head)
  bool row_pairs;          // items are pairs of row tiles: the row-pair kernel runs the pass
  int32_t *dev_lists;   // device: cta_begin[grid + 1], then item_list[n_items]
};

bool prefix_tc_shape_supported(const Params &p, int dtype) {
  return dtype == MC_BF16 && p.d == D && p.g >= 1 && p.g <= kTileM && kTileM % p.g == 0;
}

bool prefix_tc_supported(const Params &p, int dtype) {
  return prefix_tc_shape_supported(p, dtype) && p.prefix_part_tokens % kTileN == 0;
}

namespace {

bool env_chain_levels() {
  const char *e = std::getenv("MC_PREFIX_CHAIN");
  return !(e && *e == '0');
}
bool env_row_pairs() {
  const char *e = std::getenv("MC_PREFIX_PAIRS");
  return !(e && *e == '0');
}

// Longest-processing-time-first assignment of items (sorted by cost, descending) to `grid` CTAs; returns the
// largest CTA load and, if asked, which CTA each item went to.
double lpt_assign(const std::vector<int> &by_cost, const std::vector<double> &cost, int grid, std::vector<int> *owner) {
  typedef std::pair<double, int> Load;   // (load, CTA); the least loaded CTA on top
  std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
  for (int c = 0; c < grid; ++c) heap.push(Load(0.0, c));
  double longest = 0.0;
  for (size_t i = 0; i < by_cost.size(); ++i) {
    Load l = heap.top();
    heap.pop();
    l.first += cost[(size_t)by_cost[i]];
    if (l.first > longest) longest = l.first;
    if (owner) (*owner)[(size_t)by_cost[i]] = l.second;
    heap.push(l);
  }
  return longest;
}

}  // namespace

// Host-side preparation at layout-create time: tensor maps over the two pools, and the items of every level
// (`levels[k]` with at most `max_group[k]` candidates in one group) dealt to the CTAs of one persistent grid.
// An item's cost is estimated from the lengths as they are now (`tile_us` per 128 x 128 tile, `item_us` per item);
// the items are assigned longest first to the least loaded CTA, and the grid is the smallest (at least 8 CTAs, at
// most 7/16 of the SMs: the suffix pass, which cannot share an SM with this kernel's CTAs, reaches the memory
// roofline from the rest) whose most loaded CTA stays within `target_us` - or `fixed_ctas` CTAs if that is positive.  The lists stay
// valid when the lengths change later; only their balance is the create-time one.  nullptr when unavailable.
PrefixTcPlan *prefix_tc_plan(const Params *levels, const int *max_group, int n_levels, int sm_count, int fixed_ctas,
                             double target_us, double tile_us, double item_us, const float *k_scale) {
  if (n_levels < 1 || n_levels > kMaxTcLevels) return nullptr;
  PrefixTcPlan *plan = new PrefixTcPlan();
  plan->dev_lists = nullptr;
  plan->k_scale = k_scale;
  plan->wait_cycles = wait_limit_cycles();
  const Params &p = levels[0];
  if ((long long)p.num_pages * p.Hkv > 0x7fffffffLL ||
      !encode_pool_map(&plan->k_map, p.k_pool, p.num_pages, p.Hkv, false) ||
      !encode_pool_map(&plan->v_map, p.v_pool, p.num_pages, p.Hkv, true)) {
    delete plan;
    return nullptr;
  }
  long long items = 0;
  plan->levels.n = n_levels;
  std::vector<double> cost;
  // Where every level stacks at least two 128-row tiles per (group, kv head), an item is a pair of row tiles (the
  // row-pair kernel); otherwise one row tile (MC_PREFIX_PAIRS=0: always one).
  bool pairs = env_row_pairs();
  for (int k = 0; k < n_levels; ++k) pairs = pairs && (max_group[k] * levels[k].g + kTileM - 1) / kTileM >= 2;
  plan->row_pairs = pairs;
  const int unit_rows = pairs ? 2 * kTileM : kTileM;
  // Two single-split levels of which one's groups nest in the other's, with as many 128-row tiles: the finer level's
  // items take the coarser level's tokens along (one item, one accumulator, one part per row tile instead of two
  // items and two parts), and the coarser level gets no items of its own.
  int fine = -1, coarse = -1;
  std::vector<int32_t> coarse_len, coarse_go;
  if (n_levels == 2 && levels[0].n_prefix_parts == 1 && levels[1].n_prefix_parts == 1 && env_chain_levels()) {
    std::vector<int32_t> go[2];
    bool known = true;
    for (int k = 0; k < 2; ++k) {
      go[k].resize((size_t)levels[k].G + 1);
      known = known && cudaMemcpy(go[k].data(), levels[k].group_offsets, sizeof(int32_t) * go[k].size(),
                                  cudaMemcpyDeviceToHost) == cudaSuccess;
    }
    (void)cudaGetLastError();
    for (int f = 0; f < 2 && known && fine < 0; ++f) {
      const int c = 1 - f;
      if (levels[f].G < levels[c].G) continue;
      // every boundary of the coarser level is a boundary of the finer one, and the row tiles add up to as many
      bool nested = true;
      size_t i = 0;
      long long tiles_f = 0, tiles_c = 0;
      for (int j = 0; j <= levels[c].G && nested; ++j) {
        while (i < go[f].size() && go[f][i] < go[c][(size_t)j]) ++i;
        nested = i < go[f].size() && go[f][i] == go[c][(size_t)j];
      }
      for (int j = 0; j < levels[f].G; ++j) tiles_f += ((long long)(go[f][(size_t)j + 1] - go[f][(size_t)j]) * p.g + unit_rows - 1) / unit_rows;
      for (int j = 0; j < levels[c].G; ++j) tiles_c += ((long long)(go[c][(size_t)j + 1] - go[c][(size_t)j]) * p.g + unit_rows - 1) / unit_rows;
      if (nested && tiles_f <= tiles_c) {
        coarse_len.resize((size_t)levels[c].G);
        if (cudaMemcpy(coarse_len.data(), levels[c].prefix_len, sizeof(int32_t) * coarse_len.size(),
                       cudaMemcpyDeviceToHost) == cudaSuccess) {
          fine = f;
          coarse = c;
          coarse_go = go[c];
        }
        (void)cudaGetLastError();
      }
    }
  }
  for (int k = 0; k < n_levels; ++k) {
    const Params &pk = levels[k];
    TcLevel &lv = plan->levels.lv[k];
    lv.group_offsets = pk.group_offsets;
    lv.prefix_pages = pk.prefix_pages;
    lv.prefix_len = pk.prefix_len;
    lv.row_limit = pk.row_limit;
    lv.max_pp = pk.max_pp;
    lv.n_splits = pk.n_prefix_parts;
    lv.part_base = pk.prefix_part_base;
    lv.part_tokens = pk.prefix_part_tokens;
    lv.n_groups = pk.G;
    lv.chain = k == fine ? coarse : -1;
    lv.n_mt = (max_group[k] * pk.g + unit_rows - 1) / unit_rows;   // row units (tiles, or pairs of tiles) per (group, kv head, split)
    const long long level_items = (long long)pk.G * pk.Hkv * lv.n_splits * lv.n_mt;
    items += level_items;
    if (items > (1ll << 24)) {
      delete plan;
      return nullptr;
    }
    lv.item_end = (int32_t)items;
    // cost of each item of the level, in the kernel's numbering (row tile fastest, then split, kv head, group)
    std::vector<int32_t> go((size_t)pk.G + 1), len((size_t)pk.G);
    const bool known =
        cudaMemcpy(go.data(), pk.group_offsets, sizeof(int32_t) * go.size(), cudaMemcpyDeviceToHost) == cudaSuccess &&
        cudaMemcpy(len.data(), pk.prefix_len, sizeof(int32_t) * len.size(), cudaMemcpyDeviceToHost) == cudaSuccess;
    (void)cudaGetLastError();
    const int cand_per_tile = unit_rows / pk.g;   // candidates per row unit
    for (long long it = 0; it < level_items; ++it) {
      const int mt = (int)(it % lv.n_mt);
      long long r = it / lv.n_mt;
      const int sp = (int)(r % lv.n_splits);
      r /= lv.n_splits;
      const int j = (int)(r / pk.Hkv);
      const int n_cand = known ? go[(size_t)j + 1] - go[(size_t)j] : max_group[k];
      const long long cap = (long long)pk.max_pp * kPage;
      long long l = known ? len[(size_t)j] : cap;
      l = l < 0 ? 0 : l > cap ? cap : l;
      const long long lo = (long long)sp * lv.part_tokens;
      const long long tokens = (l < lo + lv.part_tokens ? l : lo + lv.part_tokens) - lo;
      long long tiles = tokens > 0 ? (tokens + kTileN - 1) / kTileN : 0;
      if (k == fine && known) {   // plus the tokens of the coarser group around this one
        size_t j2 = 0;
        while (j2 + 1 < coarse_go.size() - 1 && coarse_go[j2 + 1] <= go[(size_t)j]) ++j2;
        const long long cap2 = (long long)levels[coarse].max_pp * kPage;
        long long l2 = coarse_len[j2];
        l2 = l2 < 0 ? 0 : l2 > cap2 ? cap2 : l2;
        tiles += (l2 + kTileN - 1) / kTileN;
      }
      double c = 0.0;
      if (k != coarse && tiles > 0 && mt * cand_per_tile < n_cand) {
        const int row_tiles = pairs && (long long)(n_cand - mt * cand_per_tile) * pk.g > kTileM ? 2 : 1;
        c = (double)tiles * row_tiles * tile_us + item_us;
      }
      cost.push_back(c);
    }
  }
  plan->n_items = (int)items;
  const int coarse_begin = coarse < 0 ? 0 : coarse == 0 ? 0 : plan->levels.lv[coarse - 1].item_end;
  const int coarse_end = coarse < 0 ? 0 : plan->levels.lv[coarse].item_end;
  std::vector<int> by_cost;
  by_cost.reserve((size_t)plan->n_items);
  for (int i = 0; i < plan->n_items; ++i)
    if (i < coarse_begin || i >= coarse_end) by_cost.push_back(i);   // the coarser level of a chain has no items
  std::stable_sort(by_cost.begin(), by_cost.end(), [&](int a, int b) { return cost[(size_t)a] > cost[(size_t)b]; });
  int live = 0;
  for (int i = 0; i < plan->n_items; ++i) live += cost[(size_t)i] > 0.0;
  const int most = live < 1 ? 1 : live < sm_count ? live : sm_count;
  int grid;
  if (fixed_ctas > 0) {
    grid = fixed_ctas < most ? fixed_ctas : most;
  } else {
    // (with nothing to run beside - no suffix tokens, as in scoring - the pass may have every SM)
    const int cap = target_us <= 0.0 ? sm_count : sm_count * 7 / 16 > 8 ? sm_count * 7 / 16 : 8;
    int lo = 8 < most ? 8 : most, hi = most < cap ? most : cap;   // smallest grid in [lo, hi] that meets the target (hi if none does)
    while (lo < hi) {
      const int mid = (lo + hi) / 2;
      if (lpt_assign(by_cost, cost, mid, nullptr) <= target_us) hi = mid; else lo = mid + 1;
    }
    grid = lo;
    // A prefix pass that outlasts the suffix pass even on its full share of the SMs (long shared prompts, short
    // private suffixes: the first steps of a round of rollouts) is what the step waits for: it may then have more
    // CTAs, up to every SM.  Estimate of the step with g prefix CTAs: the prefix pass beside the suffix stream (a
    // third longer than alone) against the suffix pass on the SMs that are left (it needs sm_count - cap of them to
    // saturate HBM and slows in proportion below that); with every SM taken the two passes run one after the other.
    const double suffix_us = target_us / 0.09;   // target_us is a tenth of nine tenths of the suffix pass's time
    if (grid == cap && most > cap && target_us > 0.0) {
      double best = lpt_assign(by_cost, cost, cap, nullptr) * 1.3;
      if (best > suffix_us) {
        const int step = most - cap > 32 ? 4 : 1;
        for (int g = cap + step; g <= most; g = (g < most && g + step > most) ? most : g + step) {
          const double load = lpt_assign(by_cost, cost, g, nullptr);
          const double left = (double)(sm_count - g), sat = (double)(sm_count - cap);
          const double est = left < 1.0 ? load + suffix_us
                                        : std::max(load * 1.3, suffix_us * (left >= sat ? 1.0 : sat / left));
          if (est < best * 0.98) {   // (a larger grid must earn its SMs)
            best = est;
            grid = g;
          }
        }
      }
    }
  }
  plan->grid = grid;
  plan->one_part_per_row = (n_levels == 1 && levels[0].n_prefix_parts == 1) || fine >= 0;
  std::vector<int> owner((size_t)plan->n_items, 0);
  lpt_assign(by_cost, cost, grid, &owner);
  std::vector<int32_t> lists((size_t)grid + 1 + by_cost.size(), 0);
  for (size_t i = 0; i < by_cost.size(); ++i) lists[(size_t)owner[(size_t)by_cost[i]] + 1] += 1;
  for (int c = 0; c < grid; ++c) lists[(size_t)c + 1] += lists[(size_t)c];
  std::vector<int32_t> fill(lists.begin(), lists.begin() + grid);
  for (size_t i = 0; i < by_cost.size(); ++i) {   // costliest first within each CTA
    const int it = by_cost[i];
    lists[(size_t)grid + 1 + (size_t)fill[(size_t)owner[(size_t)it]]++] = it;
  }
  if (cudaFuncSetAttribute(prefix_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)sizeof(Smem)) != cudaSuccess ||
      cudaFuncSetAttribute(prefix_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)sizeof(Smem)) != cudaSuccess ||
      cudaFuncSetAttribute(prefix_rp_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)sizeof(SmemRp)) != cudaSuccess ||
      cudaFuncSetAttribute(prefix_rp_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)sizeof(SmemRp)) != cudaSuccess ||
      cudaMalloc(&plan->dev_lists, sizeof(int32_t) * lists.size()) != cudaSuccess ||
      cudaMemcpy(plan->dev_lists, lists.data(), sizeof(int32_t) * lists.size(), cudaMemcpyHostToDevice) != cudaSuccess) {
    (void)cudaGetLastError();
    prefix_tc_plan_free(plan);
    return nullptr;
  }
  return plan;
}

void prefix_tc_plan_free(PrefixTcPlan *plan) {
  if (!plan) return;
  cudaFree(plan->dev_lists);
  delete plan;
}
int prefix_tc_grid(const PrefixTcPlan *plan) { return plan ? plan->grid : 0; }


bool prefix_tc_one_part_per_row(const PrefixTcPlan *plan) { return plan && plan->one_part_per_row; }

// o_final / lse_final non-null (only for a plan with one part per row, and only when no other pass adds parts): the
// pass writes the final bf16 output and log-sum-exp of every row itself instead of partial results.
mc_status_t launch_prefix_tc(const Params &p, const PrefixTcPlan *plan, const void *q, float scale, float *o_part,
                             float *lse_part, cudaStream_t stream, void *o_final, float *lse_final,
                             bool beside_previous) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)plan->grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = plan->row_pairs ? sizeof(SmemRp) : sizeof(Smem);
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = beside_previous ? 1 : 0;
  cudaError_t e;
  if (plan->row_pairs) {
    // the stacked query tiles come by TMA: a map over this call's q, [B][Hq][d] seen as boxes of 128 / g candidates x
    // g heads x 64 elements (rows of the box = the stacked row order); candidates beyond B read as zeros
    CUtensorMap q_map;
    if (!encode_q_map(&q_map, q, p.B, p.Hq, p.g)) return MC_ERR_CUDA;
    e = cudaLaunchKernelEx(&cfg, plan->k_scale ? prefix_rp_kernel<true> : prefix_rp_kernel<false>, p, plan->levels,
                           plan->k_map, plan->v_map, q_map, scale * kLog2e, o_part, lse_part,
                           (const int32_t *)(plan->dev_lists + plan->grid + 1), (const int32_t *)plan->dev_lists,
                           reinterpret_cast<__nv_bfloat16 *>(o_final), lse_final, plan->wait_cycles, plan->k_scale);
  } else {
    e = cudaLaunchKernelEx(
        &cfg, plan->k_scale ? prefix_tc_kernel<true> : prefix_tc_kernel<false>, p, plan->levels, plan->k_map, plan->v_map,
        reinterpret_cast<const __nv_bfloat16 *>(q), scale * kLog2e, o_part, lse_part,
        (const int32_t *)(plan->dev_lists + plan->grid + 1), (const int32_t *)plan->dev_lists,
        reinterpret_cast<__nv_bfloat16 *>(o_final), lse_final, plan->wait_cycles, plan->k_scale);
  }
  count_launch();
  return e == cudaSuccess ? check_launch() : MC_ERR_CUDA;
}

}  // namespace mc
