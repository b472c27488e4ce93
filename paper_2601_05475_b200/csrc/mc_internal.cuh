// Internal declarations shared by the translation units of the library (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "maxcode_attn.h"

namespace mc {

constexpr int kPage = 16;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// status bits latched on the device (first non-zero value wins through atomicCAS)
constexpr int kDevBadPage = MC_ERR_INVALID_ARG;
constexpr int kDevTimeout = MC_ERR_TIMEOUT;

// Everything a kernel needs to walk the paged cache; passed by value.
struct Params {
  const void *k_pool, *v_pool;
  const int32_t *group_offsets, *prefix_pages, *prefix_len, *suffix_pages, *suffix_len;
  int32_t G, B, Hq, Hkv, d, g;
  int32_t num_pages, max_pp, max_sp;                 // in 16-token UNIT pages (a cache page of 32 / 64 tokens is 2 / 4 of them)
  int32_t lr;                                        // log2 of the unit pages per cache page (0, 1, 2)
  int32_t n_parts;                                   // part slots per row (all prefix levels + suffix chunks)
  int32_t n_prefix_parts, prefix_part_base;          // this prefix level's splits and its first part slot
  int32_t suffix_part_base;                          // first part slot of the suffix chunks
  int32_t prefix_part_tokens, suffix_part_tokens;
  const int32_t *row_limit;                          // per candidate: tokens of this prefix level it may see (null: all)
  const int32_t *suffix_order;                       // launch order of the suffix pass's CTAs (null: as numbered)
  int32_t *status;
  const float *k_scale, *v_scale;                    // e4m3 cache only: one scale per (page, kv head), [num_pages][Hkv]
};

enum Mode : int { kPrefix = 0, kSuffix = 1 };

// Which token range an item covers, resolved on the device from the device-resident lengths.
struct Span {
  const int32_t *pages;  // page-table row
  int32_t lo, hi;        // token range [lo, hi) of the sequence, lo a multiple of 16
  int32_t part;          // part slot the result goes to
};

__device__ __forceinline__ int group_of(const Params &p, int b) {
  int lo = 0, hi = p.G;  // invariant: offsets[lo] <= b < offsets[hi]
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (__ldg(p.group_offsets + mid) <= b) lo = mid; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ void latch(const Params &p, int code) { atomicCAS(p.status, 0, code); }

// The kernels walk tables of 16-token unit pages.  Unit id u = cache page id * units per page + unit inside the page;
// the pool is [cache page][kv head][page_size tokens][d], so the 16-token slab of (u, kv head h) is slab number
// ((u >> lr) * Hkv + h) * 2^lr + (u & (2^lr - 1)) in units of 16 * d elements.  With 16-token cache pages: u * Hkv + h.
__device__ __forceinline__ size_t slab_index(const Params &p, int unit, int h) {
  return ((((size_t)(unit >> p.lr)) * p.Hkv + h) << p.lr) + (size_t)(unit & ((1 << p.lr) - 1));
}

template <int MODE>
__device__ __forceinline__ Span resolve_span(const Params &p, int b, int part) {
  Span s;
  int len, cap, tokens;
  if (MODE == kPrefix) {
    int j = group_of(p, b);
    s.pages = p.prefix_pages + (size_t)j * p.max_pp;
    len = __ldg(p.prefix_len + j);
    if (p.row_limit) len = min(len, max(__ldg(p.row_limit + b), 0));
    cap = p.max_pp * kPage;
    tokens = p.prefix_part_tokens;
    s.part = p.prefix_part_base + part;
  } else {
    s.pages = p.suffix_pages + (size_t)b * p.max_sp;
    len = __ldg(p.suffix_len + b);
    cap = p.max_sp * kPage;
    tokens = p.suffix_part_tokens;
    s.part = p.suffix_part_base + part;
  }
  if (len > cap || len < 0) {  // a length the table cannot hold: clamp and report
    latch(p, kDevBadPage);
    len = len < 0 ? 0 : cap;
  }
  s.lo = part * tokens;
  s.hi = min(len, s.lo + tokens);
  return s;
}

struct Layout;  // the opaque handle

void count_launch();
mc_status_t check_launch();
// Limit, in SM clock cycles, of every bounded device-side wait of kernels planned from now on: about one second,
// or MC_WAIT_CYCLES from the environment (tests shorten it to see a wait run out).
long long wait_limit_cycles();

// launchers (each enqueues on `stream` and returns the launch status)
mc_status_t launch_fma(const Params &p, int dtype, int mode, const void *q, float scale, float *o_part,
                       float *lse_part, cudaStream_t stream);
// `beside_previous`: the launch does not wait for the kernel in front of it on the stream to end, only for
// that kernel's CTAs to announce that dependents may start (programmatic dependent launch).
mc_status_t launch_mma(const Params &p, int mode, const void *q, float scale, float *o_part, float *lse_part,
                       cudaStream_t stream, bool beside_previous = false);
mc_status_t launch_merge(const Params &p, int dtype, const float *o_part, const float *lse_part, void *o,
                         float *lse, cudaStream_t stream, bool beside_previous = false);
bool mma_supported(const Params &p, int dtype);
int mma_items_per_cta();

// tensor-core (tcgen05) prefix pass: one persistent grid over the items of all cascade levels
constexpr int kMaxTcLevels = 4;
struct PrefixTcPlan;
bool prefix_tc_supported(const Params &p, int dtype);
// `k_scale` non-null: the levels' pools are an e4m3 cache expanded to bf16 (K: the exact codes, V: dequantised) and
// k_scale [page][kv head] holds each page's K scale, applied to the scores in the softmax.
PrefixTcPlan *prefix_tc_plan(const Params *levels, const int *max_group, int n_levels, int sm_count, int fixed_ctas,
                             double target_us, double tile_us, double item_us, const float *k_scale = nullptr);
void prefix_tc_plan_free(PrefixTcPlan *plan);
int prefix_tc_grid(const PrefixTcPlan *plan);
bool prefix_tc_shape_supported(const Params &p, int dtype);   // everything but the part geometry
bool prefix_tc_one_part_per_row(const PrefixTcPlan *plan);
mc_status_t launch_prefix_tc(const Params &p, const PrefixTcPlan *plan, const void *q, float scale, float *o_part,
                             float *lse_part, cudaStream_t stream, void *o_final = nullptr, float *lse_final = nullptr,
                             bool beside_previous = false);


// Tensor map over a paged pool seen as num_pages * Hkv slabs of [16 tokens][128] (bf16; num_pages counts 16-token
// unit pages; slab_index orders them) for TMA copies with the 128-byte swizzle:
// `whole_page`: one 4 KB box per slab that lands as [d half][16 tokens][64];
// otherwise one 2 KB box per (slab, d half).
bool encode_pool_map(CUtensorMap *map, const void *pool, int num_pages, int Hkv, bool whole_page);
bool encode_kv_pair_map(CUtensorMap *map, const void *lower_pool, unsigned long long distance, int num_pages, int Hkv);

// suffix pass through TMA-fed shared-memory rings (bf16, d = 128, g <= 8)
struct SuffixTmaPlan;
SuffixTmaPlan *suffix_tma_plan(const Params &p, int dtype);
void suffix_tma_plan_free(SuffixTmaPlan *plan);
int suffix_tma_items_per_cta();
mc_status_t launch_suffix_tma(const Params &p, const SuffixTmaPlan *plan, const void *q, float scale, float *o_part,
                              float *lse_part, cudaStream_t stream, bool beside_previous);

// KV cache in e4m3 with per-(page, kv head) scales (bf16 queries and outputs, d = 128, g <= 8): both passes on one
// TMA-fed warp-level kernel, and the quantising append
struct Fp8Plan;
Fp8Plan *fp8_plan(const Params &p);
void fp8_plan_free(Fp8Plan *plan);
int fp8_items_per_cta();
bool fp8_supported(const Params &p);
mc_status_t launch_fp8(const Params &p, const Fp8Plan *plan, int mode, const void *q, float scale, float *o_part,
                       float *lse_part, cudaStream_t stream, bool beside_previous = false);
// the prefix levels widened to bf16 pools of their own, for the tensor-core prefix pass
bool fp8_expand_alloc(Fp8Plan *plan, const Params *levels, int n_levels, Params *expanded);
const float *fp8_expanded_k_scale(const Fp8Plan *plan);
mc_status_t fp8_expand_launch(const Fp8Plan *plan, const Params *levels, int n_levels, cudaStream_t stream);
mc_status_t launch_append_fp8(const Params &p, const void *k_new, const void *v_new, int32_t *suffix_len,
                              cudaStream_t stream);
mc_status_t launch_append_tokens_fp8(const Params &p, const void *k_new, const void *v_new, int n_max,
                                     const int32_t *n_new, const int32_t *suffix_len, cudaStream_t stream);

// The q/k/v projection y = x W^T on the tensor cores (bf16, heads of 128 features).  A persistent grid shares out
// the k-blocks (64 hidden elements) of all head pairs in equal contiguous runs; the fp32 sums of a run's part of a
// head pair are a "piece": partials [piece][row stride][feature stride], in a workspace the plan owns.  The pieces of
// pair r are those of CTAs first(r) .. last(r), piece index = CTA - first(r), where the CTA holding k-block u of
// the numbering pair * kb_per_pair + kb is ((u + 1) * ctas - 1) / (pairs * kb_per_pair).
struct QkvPlan;
QkvPlan *qkv_plan(int B, int heads, int hidden, const void *w, int sms);
void qkv_plan_free(QkvPlan *plan);
int qkv_pieces(const QkvPlan *plan);        // most pieces any head pair has
int qkv_ctas(const QkvPlan *plan);          // CTAs of one pass
int qkv_passes(const QkvPlan *plan);        // passes over the candidates (256 rows each at most)
int qkv_kb_per_pair(const QkvPlan *plan);
int qkv_row_stride(const QkvPlan *plan);
int qkv_feature_stride(const QkvPlan *plan);
size_t qkv_workspace_bytes(const QkvPlan *plan);
const float *qkv_partials(const QkvPlan *plan);
// `beside_previous`: launched as the programmatic dependent of the kernel in front of it, whose completion it awaits
// before it lets its own dependent start
mc_status_t launch_qkv_gemm(const QkvPlan *plan, const void *x, int32_t *status, cudaStream_t stream,
                            bool beside_previous);

}  // namespace mc
