// C-ABI entry points: argument checking, layout object, append, validation, status word, and the
// drivers that enqueue the passes.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "maxcode_qkv.h"
#include "mc_internal.cuh"

namespace mc {

constexpr int kMaxOuterLevels = 3;

struct Layout {
  mc_kv_layout_desc_t desc;
  Params p;
  int32_t *dev_status;   // device int
  int32_t *suffix_order; // device array: launch order of the suffix pass's CTAs, or null
  int32_t *host_status;  // pinned host int, target of the status read-back
  size_t o_part_bytes, lse_part_bytes, staging_off[5], ws_bytes;
  bool use_mma;
  bool has_suffix;            // false: no private tokens (max_suffix_pages = 0), the suffix pass is not launched
  SuffixTmaPlan *sfx_plan;    // non-null: the suffix pass runs on the TMA-fed kernel
  Fp8Plan *fp8;               // non-null: e4m3 cache; its kernel runs the suffix pass and, without tc_plan, the prefix pass
  Params xp;                  // e4m3 cache with tc_plan: the base level seen through the expanded (bf16) prefix pools
  Params x_src[1 + kMaxOuterLevels];   // ... and the levels the expansion reads, outermost first
  int x_n;
  int io_dtype;               // type of q and o: the cache's, or bf16 over an e4m3 cache
  PrefixTcPlan *tc_plan;      // non-null: every prefix level runs on the tcgen05 kernel, as one launch
  int n_outer;                // outer prefix levels of a cascade (shared by more candidates than the base level)
  Params outer_p[kMaxOuterLevels];
  // Cache pages of 32 or 64 tokens: every kernel walks 16-token unit pages through tables the layout derives from
  // the caller's (entry e of a table becomes the units e * r .. e * r + r - 1, r = page_size / 16).
  struct UnitTable { const int32_t *src; int32_t *dst; long long n; };
  UnitTable unit_tab[2 + kMaxOuterLevels];
  int n_unit_tab;
  int32_t *unit_buf;          // the derived tables, one allocation; null with 16-token pages
  cudaStream_t side_stream;   // the suffix pass of mc_decode_attn runs here, beside the prefix pass
  cudaEvent_t fork_ev, join_ev;
  bool pdl;                   // suffix pass launched as the prefix pass's programmatic dependent (MC_PDL=0: off)
};

static std::atomic<uint64_t> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
mc_status_t check_launch() { return cudaPeekAtLastError() == cudaSuccess ? MC_OK : MC_ERR_CUDA; }
long long wait_limit_cycles() {
  const char *s = std::getenv("MC_WAIT_CYCLES");
  if (s && *s) {
    const long long v = std::atoll(s);
    if (v >= 0) return v;
  }
  return 2000000000ll;
}

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
int pow2_floor(int x) { int r = 1; while (r * 2 <= x) r *= 2; return r; }
int env_int(const char *name, int dflt) {
  const char *s = std::getenv(name);
  if (!s || !*s) return dflt;
  int v = std::atoi(s);
  return v >= 0 ? v : dflt;
}

// ------------------------------------------------------------------------------------------------
// append: one block per candidate copies the new token's K and V rows of every kv head
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) append_kernel(Params p, const uint4 *__restrict__ k_new,
                                                     const uint4 *__restrict__ v_new, int32_t *suffix_len,
                                                     int elem_bytes) {
  // The prefix pass, when it is launched behind this kernel as its programmatic dependent, reads nothing this
  // kernel writes and may start at once; it holds back the suffix pass until this grid has completed.
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  const int b = blockIdx.x;
  const int s = suffix_len[b];
  const int pg = s >> 4;
  int page = -1;
  if (s >= 0 && pg < p.max_sp) page = __ldg(p.suffix_pages + (size_t)b * p.max_sp + pg);
  if ((unsigned)page >= (unsigned)p.num_pages) {  // row full, or a bad table entry: leave the candidate alone
    if (threadIdx.x == 0) latch(p, kDevBadPage);
    return;
  }
  const int row_vec = p.d * elem_bytes / 16;  // uint4 per (token, kv head) row
  const int n_vec = p.Hkv * row_vec;
  uint4 *kp = reinterpret_cast<uint4 *>(const_cast<void *>(p.k_pool));
  uint4 *vp = reinterpret_cast<uint4 *>(const_cast<void *>(p.v_pool));
  for (int i = threadIdx.x; i < 2 * n_vec; i += blockDim.x) {
    const int which = i >= n_vec, j = which ? i - n_vec : i;
    const int h = j / row_vec, c = j % row_vec;
    const size_t dst = (slab_index(p, page, h) * kPage + (s & 15)) * row_vec + c;
    const size_t src = ((size_t)b * p.Hkv + h) * row_vec + c;
    if (which) vp[dst] = v_new[src]; else kp[dst] = k_new[src];
  }
  __syncthreads();  // every thread has read s and issued its stores before the length moves
  if (threadIdx.x == 0) suffix_len[b] = s + 1;
}

// ------------------------------------------------------------------------------------------------
// append with rotary position embedding: one block per candidate.  The head's d elements are d/2 complex
// numbers (element i the real, i + d/2 the imaginary part); the one at index i is multiplied by
// exp(j pos theta_i), theta_i = base^(-2 i / d), pos = the token's position in its whole sequence.  The angle is
// formed and reduced in double precision (positions reach 10^5, where a single-precision angle is off by
// 10^-2 radians); the rotation itself is single precision.  K is stored rotated, V as it is, q in place.
// ------------------------------------------------------------------------------------------------
struct RopeLevels {
  int n;
  int G[1 + kMaxOuterLevels];
  const int32_t *group_offsets[1 + kMaxOuterLevels], *prefix_len[1 + kMaxOuterLevels];
};

template <typename T> __device__ __forceinline__ float rope_load(const T *p);
template <> __device__ __forceinline__ float rope_load<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float rope_load<__nv_bfloat16>(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
__device__ __forceinline__ void rope_store(float *p, float v) { *p = v; }
__device__ __forceinline__ void rope_store(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

template <typename T>
__global__ void __launch_bounds__(256) append_rope_kernel(Params p, RopeLevels lv, const T *__restrict__ k_new,
                                                          const uint4 *__restrict__ v_new, T *q,
                                                          const int32_t *__restrict__ pos_offset, double log2_base,
                                                          int32_t *suffix_len) {
  const int b = blockIdx.x;
  const int s = suffix_len[b];
  const int pg = s >> 4;
  int page = -1;
  if (s >= 0 && pg < p.max_sp) page = __ldg(p.suffix_pages + (size_t)b * p.max_sp + pg);
  if ((unsigned)page >= (unsigned)p.num_pages) {  // row full, or a bad table entry: leave the candidate alone
    if (threadIdx.x == 0) latch(p, kDevBadPage);
    return;
  }
  // position of the new token: the tokens before it, on every level of the cascade
  long long pos = s;
  if (pos_offset) {
    pos += __ldg(pos_offset + b);
  } else {
    for (int k = 0; k < lv.n; ++k) {
      int lo = 0, hi = lv.G[k];
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(lv.group_offsets[k] + mid) <= b) lo = mid; else hi = mid;
      }
      pos += max(__ldg(lv.prefix_len[k] + lo), 0);
    }
  }
  const int half = p.d / 2, lanes = blockDim.x / half;   // d/2 divides the block size (d = 64 or 128)
  const int i = threadIdx.x % half, h0 = threadIdx.x / half;
  double sn, cs;
  sincos((double)pos * exp2(-2.0 * i / p.d * log2_base), &sn, &cs);
  const float c = (float)cs, sf = (float)sn;
  T *kp = reinterpret_cast<T *>(const_cast<void *>(p.k_pool));
  for (int h = h0; h < p.Hkv; h += lanes) {
    const T *src = k_new + ((size_t)b * p.Hkv + h) * p.d;
    T *dst = kp + (slab_index(p, page, h) * kPage + (s & 15)) * p.d;
    const float re = rope_load(src + i), im = rope_load(src + i + half);
    rope_store(dst + i, re * c - im * sf);
    rope_store(dst + i + half, re * sf + im * c);
  }
  if (q)
    for (int h = h0; h < p.Hq; h += lanes) {
      T *row = q + ((size_t)b * p.Hq + h) * p.d;
      const float re = rope_load(row + i), im = rope_load(row + i + half);
      rope_store(row + i, re * c - im * sf);
      rope_store(row + i + half, re * sf + im * c);
    }
  const int row_vec = p.d * (int)sizeof(T) / 16, n_vec = p.Hkv * row_vec;
  uint4 *vp = reinterpret_cast<uint4 *>(const_cast<void *>(p.v_pool));
  for (int j = threadIdx.x; j < n_vec; j += blockDim.x) {
    const int h = j / row_vec, cc = j % row_vec;
    vp[(slab_index(p, page, h) * kPage + (s & 15)) * row_vec + cc] = v_new[((size_t)b * p.Hkv + h) * row_vec + cc];
  }
  __syncthreads();  // every thread has read s and issued its stores before the length moves
  if (threadIdx.x == 0) suffix_len[b] = s + 1;
}

// ------------------------------------------------------------------------------------------------
// the q/k/v projection around its product.  Before it: one block per candidate looks up where the new token goes
// (page and slot, from the length and the page table) and how far it turns (cosine and sine of every pair's angle,
// formed in double precision as in append_rope_kernel), leaves both for the finishing kernel and moves the length;
// the product, which needs none of this, runs meanwhile.  After it: block (b, y) adds up, for candidate b and four
// heads, the pieces of the product (fp32 partial sums [piece][row][feature]; the pieces of a head pair are those of
// the CTAs whose runs of k-blocks touch it, in CTA order), adds the bias, rotates the query and key heads, writes
// q and stores k and v in the token's slot.  Heads are 128 features wide: a thread handles four neighbouring
// pairs (i, i + 64) of one of the block's sixteen heads; all its loads (16 bytes each, up to eight pieces) are
// independent of one another and in flight together.
// ------------------------------------------------------------------------------------------------
struct QkvToken { int32_t page, s; };   // page < 0: the candidate has no room (or a bad table entry): q only

__global__ void __launch_bounds__(64) qkv_prep_kernel(Params p, RopeLevels lv, const int32_t *__restrict__ pos_offset,
                                                      double log2_base, int32_t *suffix_len, QkvToken *tok,
                                                      float2 *rot) {
  // the product is launched behind this kernel as its programmatic dependent and may start at once
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  constexpr int kD = 128;
  const int b = blockIdx.x;
  const int s = suffix_len[b];
  const int pg = s >> 4;
  int page = -1;
  if (s >= 0 && pg < p.max_sp) page = __ldg(p.suffix_pages + (size_t)b * p.max_sp + pg);
  const bool store_kv = (unsigned)page < (unsigned)p.num_pages;
  float2 r = make_float2(1.f, 0.f);
  if (log2_base != 0.0) {
    long long pos = s < 0 ? 0 : s;
    if (pos_offset) {
      pos += __ldg(pos_offset + b);
    } else {
      for (int k = 0; k < lv.n; ++k) {
        int lo = 0, hi = lv.G[k];
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (__ldg(lv.group_offsets[k] + mid) <= b) lo = mid; else hi = mid;
        }
        pos += max(__ldg(lv.prefix_len[k] + lo), 0);
      }
    }
    double sn, cs;
    sincos((double)pos * exp2(-2.0 * threadIdx.x / kD * log2_base), &sn, &cs);
    r = make_float2((float)cs, (float)sn);
  }
  rot[(size_t)b * (kD / 2) + threadIdx.x] = r;
  __syncthreads();   // every thread has read the length before it moves
  if (threadIdx.x == 0) {
    tok[b].page = store_kv ? page : -1;
    tok[b].s = s;
    if (store_kv) suffix_len[b] = s + 1; else latch(p, kDevBadPage);
  }
}

__global__ void __launch_bounds__(256) qkv_finish_kernel(Params p, const float *__restrict__ partial, int ctas,
                                                         int kb_per_pair, int n_pairs, int row_stride,
                                                         int feature_stride, const __nv_bfloat16 *__restrict__ bias,
                                                         __nv_bfloat16 *__restrict__ q_out,
                                                         const QkvToken *__restrict__ tok,
                                                         const float2 *__restrict__ rot, int rotate) {
  // launched as the programmatic dependent of the product, which itself completes only after the kernel above has:
  // nothing is read before that
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  constexpr int kD = 128, kHalf = 64, kBatch = 8;
  const int b = blockIdx.x;
  const int i = (threadIdx.x % 16) * 4, head = blockIdx.y * (blockDim.x / 16) + threadIdx.x / 16;
  if (head >= p.Hq + 2 * p.Hkv) return;
  // CTA c of the product holds k-blocks [c T / ctas, (c + 1) T / ctas) of the numbering pair * kb_per_pair + kb
  const size_t n0 = (size_t)head * kD + i;
  const long long total = (long long)n_pairs * kb_per_pair, u0 = (long long)(head >> 1) * kb_per_pair;
  const int pieces = (int)(((u0 + kb_per_pair) * ctas - 1) / total) - (int)(((u0 + 1) * ctas - 1) / total) + 1;
  const float *src = partial + (size_t)b * feature_stride + n0;
  const size_t piece_stride = (size_t)row_stride * feature_stride;
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
  float4 a[kBatch], c8[kBatch];
#pragma unroll
  for (int k = 0; k < kBatch; ++k) {
    a[k] = k < pieces ? *reinterpret_cast<const float4 *>(src + (size_t)k * piece_stride) : zero;
    c8[k] = k < pieces ? *reinterpret_cast<const float4 *>(src + (size_t)k * piece_stride + kHalf) : zero;
  }
  const QkvToken t = tok[b];
  float re[4] = {0.f, 0.f, 0.f, 0.f}, im[4] = {0.f, 0.f, 0.f, 0.f};
  float cs[4] = {1.f, 1.f, 1.f, 1.f}, sn[4] = {0.f, 0.f, 0.f, 0.f};
  if (rotate && head < p.Hq + p.Hkv) {   // queries and keys turn, values do not
    const float4 r01 = *reinterpret_cast<const float4 *>(rot + (size_t)b * kHalf + i);
    const float4 r23 = *reinterpret_cast<const float4 *>(rot + (size_t)b * kHalf + i + 2);
    cs[0] = r01.x; sn[0] = r01.y; cs[1] = r01.z; sn[1] = r01.w;
    cs[2] = r23.x; sn[2] = r23.y; cs[3] = r23.z; sn[3] = r23.w;
  }
#pragma unroll
  for (int k = 0; k < kBatch; ++k) {   // pieces in order
    re[0] += a[k].x; re[1] += a[k].y; re[2] += a[k].z; re[3] += a[k].w;
    im[0] += c8[k].x; im[1] += c8[k].y; im[2] += c8[k].z; im[3] += c8[k].w;
  }
  for (int k = kBatch; k < pieces; ++k) {   // (more than eight pieces: a grid far wider than the stream is long)
    const float4 x = *reinterpret_cast<const float4 *>(src + (size_t)k * piece_stride);
    const float4 y = *reinterpret_cast<const float4 *>(src + (size_t)k * piece_stride + kHalf);
    re[0] += x.x; re[1] += x.y; re[2] += x.z; re[3] += x.w;
    im[0] += y.x; im[1] += y.y; im[2] += y.z; im[3] += y.w;
  }
  if (bias) {   // the sum of the pieces first, then the bias: one order, whatever the number of pieces
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      re[e] += __bfloat162float(bias[n0 + e]);
      im[e] += __bfloat162float(bias[n0 + kHalf + e]);
    }
  }
  __nv_bfloat16 *dst;
  if (head < p.Hq) {
    dst = q_out + ((size_t)b * p.Hq + head) * kD;
  } else {
    if (t.page < 0) return;
    const bool is_k = head < p.Hq + p.Hkv;
    const int h = is_k ? head - p.Hq : head - p.Hq - p.Hkv;
    __nv_bfloat16 *pool = reinterpret_cast<__nv_bfloat16 *>(const_cast<void *>(is_k ? p.k_pool : p.v_pool));
    dst = pool + (slab_index(p, t.page, h) * kPage + (t.s & 15)) * kD;
  }
  float o_re[4], o_im[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    o_re[e] = re[e] * cs[e] - im[e] * sn[e];
    o_im[e] = re[e] * sn[e] + im[e] * cs[e];
  }
  __nv_bfloat162 w0 = __floats2bfloat162_rn(o_re[0], o_re[1]), w1 = __floats2bfloat162_rn(o_re[2], o_re[3]);
  __nv_bfloat162 w2 = __floats2bfloat162_rn(o_im[0], o_im[1]), w3 = __floats2bfloat162_rn(o_im[2], o_im[3]);
  *reinterpret_cast<uint2 *>(dst + i) = make_uint2(*reinterpret_cast<uint32_t *>(&w0), *reinterpret_cast<uint32_t *>(&w1));
  *reinterpret_cast<uint2 *>(dst + i + kHalf) = make_uint2(*reinterpret_cast<uint32_t *>(&w2), *reinterpret_cast<uint32_t *>(&w3));
}

// ------------------------------------------------------------------------------------------------
// append of several tokens per candidate (prompt ingestion, speculated tokens): block (t, b) stores token t of
// candidate b at suffix position suffix_len[b] + t, rotated or not; the lengths move in a second launch, once every
// row is in place.  A candidate whose tokens do not all fit its page row is left alone and reported.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ int tokens_of(const int32_t *n_new, int b, int n_max) {
  if (!n_new) return n_max;
  const int n = __ldg(n_new + b);
  return n < 0 ? 0 : n > n_max ? n_max : n;
}

template <typename T>
__global__ void __launch_bounds__(256) append_tokens_kernel(Params p, RopeLevels lv, const T *__restrict__ k_new,
                                                            const T *__restrict__ v_new, T *q, int n_max,
                                                            const int32_t *__restrict__ n_new,
                                                            const int32_t *__restrict__ pos_offset, double log2_base,
                                                            const int32_t *__restrict__ suffix_len) {
  const int t = blockIdx.x, b = blockIdx.y;
  const int n = tokens_of(n_new, b, n_max);
  if (t >= n) return;
  const int s0 = __ldg(suffix_len + b);
  if (s0 < 0 || (long long)s0 + n > (long long)p.max_sp * kPage) {   // (reported by the kernel that moves the lengths)
    return;
  }
  const int s = s0 + t;
  const int page = __ldg(p.suffix_pages + (size_t)b * p.max_sp + (s >> 4));
  if ((unsigned)page >= (unsigned)p.num_pages) {
    if (threadIdx.x == 0) latch(p, kDevBadPage);
    return;
  }
  const size_t tok = (size_t)b * n_max + t;
  const int row_vec = p.d * (int)sizeof(T) / 16, n_vec = p.Hkv * row_vec;
  uint4 *vp = reinterpret_cast<uint4 *>(const_cast<void *>(p.v_pool));
  const uint4 *vsrc = reinterpret_cast<const uint4 *>(v_new) + tok * n_vec;
  for (int j = threadIdx.x; j < n_vec; j += blockDim.x) {
    const int h = j / row_vec, cc = j % row_vec;
    vp[(slab_index(p, page, h) * kPage + (s & 15)) * row_vec + cc] = vsrc[j];
  }
  if (log2_base == 0.0) {   // keys as they are
    uint4 *kp = reinterpret_cast<uint4 *>(const_cast<void *>(p.k_pool));
    const uint4 *ksrc = reinterpret_cast<const uint4 *>(k_new) + tok * n_vec;
    for (int j = threadIdx.x; j < n_vec; j += blockDim.x) {
      const int h = j / row_vec, cc = j % row_vec;
      kp[(slab_index(p, page, h) * kPage + (s & 15)) * row_vec + cc] = ksrc[j];
    }
    return;
  }
  // rotary position embedding, as in append_rope_kernel: position = the tokens in front of this one
  long long pos = s;
  if (pos_offset) {
    pos += __ldg(pos_offset + b);
  } else {
    for (int k = 0; k < lv.n; ++k) {
      int lo = 0, hi = lv.G[k];
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(lv.group_offsets[k] + mid) <= b) lo = mid; else hi = mid;
      }
      pos += max(__ldg(lv.prefix_len[k] + lo), 0);
    }
  }
  const int half = p.d / 2, lanes = blockDim.x / half;
  const int i = threadIdx.x % half, h0 = threadIdx.x / half;
  double sn, cs;
  sincos((double)pos * exp2(-2.0 * i / p.d * log2_base), &sn, &cs);
  const float c = (float)cs, sf = (float)sn;
  T *kp = reinterpret_cast<T *>(const_cast<void *>(p.k_pool));
  for (int h = h0; h < p.Hkv; h += lanes) {
    const T *src = k_new + (tok * p.Hkv + h) * p.d;
    T *dst = kp + (slab_index(p, page, h) * kPage + (s & 15)) * p.d;
    const float re = rope_load(src + i), im = rope_load(src + i + half);
    rope_store(dst + i, re * c - im * sf);
    rope_store(dst + i + half, re * sf + im * c);
  }
  if (q)
    for (int h = h0; h < p.Hq; h += lanes) {
      T *row = q + (tok * p.Hq + h) * p.d;
      const float re = rope_load(row + i), im = rope_load(row + i + half);
      rope_store(row + i, re * c - im * sf);
      rope_store(row + i + half, re * sf + im * c);
    }
}

__global__ void advance_len_kernel(Params p, int n_max, const int32_t *__restrict__ n_new, int32_t *suffix_len) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= p.B) return;
  const int n = tokens_of(n_new, b, n_max), s0 = suffix_len[b];
  if (n == 0) return;
  bool fits = s0 >= 0 && (long long)s0 + n <= (long long)p.max_sp * kPage;
  for (int pg = s0 >> 4; fits && pg <= (s0 + n - 1) >> 4; ++pg)   // every page the new tokens need is there
    fits = (unsigned)__ldg(p.suffix_pages + (size_t)b * p.max_sp + pg) < (unsigned)p.num_pages;
  if (!fits) {
    latch(p, kDevBadPage);
    return;
  }
  suffix_len[b] = s0 + n;
}

// ------------------------------------------------------------------------------------------------
// page tables of a cache with 32- or 64-token pages, rewritten in 16-token unit pages: entry e of the
// caller's table gives the 2^lr units e * 2^lr + 0 .. 2^lr - 1; a negative entry stays -1, any other entry
// outside the pool becomes an id that no pool has
// ------------------------------------------------------------------------------------------------
__global__ void unit_table_kernel(const int32_t *__restrict__ src, int32_t *__restrict__ dst, long long n_src, int lr,
                                  int src_pages) {
  const long long n = n_src << lr, nth = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += nth) {
    const int e = __ldg(src + (i >> lr));
    dst[i] = e < 0 ? -1 : e >= src_pages ? 0x7fffffff : (e << lr) + (int)(i & ((1 << lr) - 1));
  }
}

mc_status_t launch_unit_tables(const Layout *L, cudaStream_t st);

// ------------------------------------------------------------------------------------------------
// validation
// ------------------------------------------------------------------------------------------------
__global__ void validate_kernel(Params p, int32_t *refs, int with_suffix) {
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
  if (p.row_limit)   // per-candidate limits must not decrease inside a group
    for (int j = tid; j < p.G; j += nth)
      for (int b = __ldg(p.group_offsets + j) + 1; b < __ldg(p.group_offsets + j + 1); ++b)
        if (__ldg(p.row_limit + b) < __ldg(p.row_limit + b - 1)) latch(p, kDevBadPage);
  if (tid == 0) {
    if (__ldg(p.group_offsets) != 0 || __ldg(p.group_offsets + p.G) != p.B) latch(p, kDevBadPage);
    for (int j = 0; j < p.G; ++j)
      if (__ldg(p.group_offsets + j + 1) < __ldg(p.group_offsets + j)) latch(p, kDevBadPage);
  }
  const long long np = (long long)p.G * p.max_pp, ns = with_suffix ? (long long)p.B * p.max_sp : 0;
  for (long long i = tid; i < np + ns; i += nth) {
    int page, used;
    if (i < np) {
      const int j = (int)(i / p.max_pp), k = (int)(i % p.max_pp);
      const int len = __ldg(p.prefix_len + j);
      if (k == 0 && (len < 0 || len > p.max_pp * kPage)) latch(p, kDevBadPage);
      used = k < (len + kPage - 1) / kPage;
      page = __ldg(p.prefix_pages + i);
    } else {
      const long long r = i - np;
      const int b = (int)(r / p.max_sp), k = (int)(r % p.max_sp);
      const int len = __ldg(p.suffix_len + b);
      if (k == 0 && (len < 0 || len > p.max_sp * kPage)) latch(p, kDevBadPage);
      // pages pre-assigned for future appends count as referenced when their id is non-negative
      page = __ldg(p.suffix_pages + r);
      used = k < (len + kPage - 1) / kPage || page >= 0;
    }
    if (!used) continue;
    if ((unsigned)page >= (unsigned)p.num_pages) { latch(p, kDevBadPage); continue; }
    if (atomicAdd(refs + page, 1) != 0) latch(p, kDevBadPage);
  }
}

// ------------------------------------------------------------------------------------------------
// read-only streaming probe: every thread keeps eight 16-byte loads in flight and folds what it reads into
// one word; the word is stored only if it is non-zero, so the loads cannot be optimised away
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512) hbm_read_probe_kernel(const uint4 *__restrict__ buf, size_t n_vec,
                                                             uint32_t *sink) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  uint32_t acc = 0;
  for (; i + 7 * stride < n_vec; i += 8 * stride) {
    uint4 v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k)
      asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                   : "=r"(v[k].x), "=r"(v[k].y), "=r"(v[k].z), "=r"(v[k].w) : "l"(buf + i + k * stride));
#pragma unroll
    for (int k = 0; k < 8; ++k) acc ^= v[k].x ^ v[k].y ^ v[k].z ^ v[k].w;
  }
  for (; i < n_vec; i += stride) {
    const uint4 v = __ldg(buf + i);
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
  if (acc == 0x9e3779b9u) atomicAdd(sink, 1u);   // (practically never: keeps the loads alive)
}

mc_status_t check_q(const Layout *L, const void *q) {
  if (!L || !q) return MC_ERR_INVALID_ARG;
  if (!aligned16(q)) return MC_ERR_INVALID_ARG;
  return MC_OK;
}

mc_status_t run_level(Layout *L, const Params &p, int mode, const void *q, float scale, float *o_part,
                      float *lse_part, cudaStream_t st) {
  if (mode == kSuffix && !L->has_suffix) return MC_OK;
  if (L->fp8) return launch_fp8(p, L->fp8, mode, q, scale, o_part, lse_part, st);
  if (mode == kSuffix && L->sfx_plan) return launch_suffix_tma(p, L->sfx_plan, q, scale, o_part, lse_part, st, false);
  if (L->use_mma) return launch_mma(p, mode, q, scale, o_part, lse_part, st);
  return launch_fma(p, L->io_dtype, mode, q, scale, o_part, lse_part, st);
}

// The prefix pass covers every level of the cascade (outermost first), the suffix pass the private tokens.
mc_status_t run_pass(Layout *L, int mode, const void *q, float scale, float *o_part, float *lse_part,
                     cudaStream_t st) {
  if (mode == kPrefix) {
    if (L->tc_plan && scale != 0.f)
      return launch_prefix_tc(L->fp8 ? L->xp : L->p, L->tc_plan, q, scale, o_part, lse_part, st);
    for (int k = L->n_outer - 1; k >= 0; --k) {
      mc_status_t s = run_level(L, L->outer_p[k], kPrefix, q, scale, o_part, lse_part, st);
      if (s != MC_OK) return s;
    }
  }
  return run_level(L, L->p, mode, q, scale, o_part, lse_part, st);
}

mc_status_t launch_unit_tables(const Layout *L, cudaStream_t st) {
  for (int i = 0; i < L->n_unit_tab; ++i) {
    const Layout::UnitTable &t = L->unit_tab[i];
    const long long n = t.n << L->p.lr;
    const int blocks = (int)(n / 256 + 1 > 1184 ? 1184 : n / 256 + 1);
    unit_table_kernel<<<blocks, 256, 0, st>>>(t.src, t.dst, t.n, L->p.lr, L->desc.num_pages);
    count_launch();
  }
  return check_launch();
}

// Splits and persistent-CTA count of one prefix level (see the comment in mc_kv_layout_create_cascade).
struct LevelWork { long long pairs; double tiles; int max_group; };
constexpr double kTileUs = 1.3, kItemUs = 8.0;   // measured: per 128x128 tile; per item (prologue + epilogue)

// (group, kv head, 128-row tile) pairs and 128-token tiles of one level, from the lengths as they are now.
LevelWork level_work(const Params &p) {
  const int max_p = p.max_pp * kPage;
  LevelWork r;
  r.max_group = (p.B + p.G - 1) / p.G;
  const int rows_per_group = (int)(((long long)p.B * p.g + p.G - 1) / p.G);
  long long pairs = (long long)p.G * p.Hkv * ((rows_per_group + 127) / 128);
  double tiles = (double)pairs * ((max_p + 127) / 128);
  int32_t *go = new (std::nothrow) int32_t[p.G + 1], *pl = new (std::nothrow) int32_t[p.G];
  if (go && pl && cudaMemcpy(go, p.group_offsets, sizeof(int32_t) * (p.G + 1), cudaMemcpyDeviceToHost) == cudaSuccess &&
      cudaMemcpy(pl, p.prefix_len, sizeof(int32_t) * p.G, cudaMemcpyDeviceToHost) == cudaSuccess) {
    pairs = 0;
    tiles = 0.0;
    r.max_group = 1;
    for (int j = 0; j < p.G; ++j) {
      const int c = go[j + 1] - go[j];
      if (c > r.max_group) r.max_group = c;
      const long long pj = (long long)p.Hkv * ((c * p.g + 127) / 128);
      pairs += pj;
      tiles += (double)pj * ((pl[j] + 127) / 128);
    }
  }
  (void)cudaGetLastError();
  delete[] go;
  delete[] pl;
  r.pairs = pairs < 1 ? 1 : pairs;
  r.tiles = tiles;
  return r;
}

// Splits of one level: as few as let its longest item (plus its fixed cost) end within `budget_us`.
int choose_splits(const Params &p, const LevelWork &w, double budget_us) {
  const double max_pair_tiles = (p.max_pp * kPage + 127) / 128;
  int nsp;
  for (nsp = 1; nsp < 8; ++nsp)
    if ((max_pair_tiles + nsp - 1) / nsp * kTileUs + kItemUs <= budget_us) break;
  if (budget_us < kItemUs + kTileUs) nsp = (int)((160 + w.pairs - 1) / w.pairs);   // nothing to hide under: many items
  return nsp > 8 ? 8 : nsp < 1 ? 1 : nsp;
}

}  // namespace
}  // namespace mc

using mc::Layout;

extern "C" {

const char *mc_status_string(mc_status_t s) {
  switch (s) {
    case MC_OK: return "ok";
    case MC_ERR_INVALID_ARG: return "invalid argument";
    case MC_ERR_UNSUPPORTED: return "unsupported configuration";
    case MC_ERR_OUT_OF_MEMORY: return "out of memory";
    case MC_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case MC_ERR_CUDA: return "CUDA runtime error";
    case MC_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

uint64_t mc_launch_count(void) { return mc::g_launches.load(std::memory_order_relaxed); }

mc_status_t mc_hbm_read_probe(const void *buf, size_t bytes, uint32_t *sink, void *stream) {
  if (!buf || !sink || !mc::aligned16(buf) || bytes < 16) return MC_ERR_INVALID_ARG;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    sms = 148;
  (void)cudaGetLastError();
  mc::hbm_read_probe_kernel<<<sms * 4, 512, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const uint4 *>(buf), bytes / 16, sink);
  mc::count_launch();
  return mc::check_launch();
}

mc_status_t mc_kv_layout_create(const mc_kv_layout_desc_t *d, mc_kv_layout_t **out) {
  return mc_kv_layout_create_cascade(d, nullptr, 0, out);
}

mc_status_t mc_kv_layout_create_cascade(const mc_kv_layout_desc_t *d, const mc_prefix_level_t *outer, int32_t n_outer,
                                        mc_kv_layout_t **out) {
  if (out) *out = nullptr;
  if (!d || !out) return MC_ERR_INVALID_ARG;
  if (d->num_groups < 1 || d->batch < 1 || d->num_q_heads < 1 || d->num_kv_heads < 1 || d->num_pages < 1 ||
      d->max_prefix_pages < 1 || d->max_suffix_pages < 0 || d->batch < d->num_groups)
    return MC_ERR_INVALID_ARG;
  if (d->num_q_heads % d->num_kv_heads != 0) return MC_ERR_INVALID_ARG;
  // max_suffix_pages = 0: a layout without private tokens (scoring of whole sequences); no suffix tables, no suffix
  // part slots, no suffix launch, appends refused
  if (!d->k_pool || !d->v_pool || !d->group_offsets || !d->prefix_pages || !d->prefix_len ||
      (d->max_suffix_pages > 0 && (!d->suffix_pages || !d->suffix_len)))
    return MC_ERR_INVALID_ARG;
  if (!mc::aligned16(d->k_pool) || !mc::aligned16(d->v_pool)) return MC_ERR_INVALID_ARG;
  if (n_outer < 0 || n_outer > mc::kMaxOuterLevels || (n_outer > 0 && !outer)) return MC_ERR_INVALID_ARG;
  for (int k = 0; k < n_outer; ++k)
    if (outer[k].num_groups < 1 || outer[k].num_groups > d->batch || outer[k].max_pages < 1 ||
        !outer[k].group_offsets || !outer[k].pages || !outer[k].len)
      return MC_ERR_INVALID_ARG;
  if (d->page_size != 16 && d->page_size != 32 && d->page_size != 64) return MC_ERR_UNSUPPORTED;
  const int lr = d->page_size == 16 ? 0 : d->page_size == 32 ? 1 : 2, upp = 1 << lr;   // unit pages per cache page
  if ((long long)d->num_pages * upp >= 0x7fffffffLL || (long long)d->max_prefix_pages * upp * mc::kPage > 0x7fffffffLL ||
      (long long)d->max_suffix_pages * upp * mc::kPage > 0x7fffffffLL)
    return MC_ERR_UNSUPPORTED;
  for (int k = 0; k < n_outer; ++k)
    if ((long long)outer[k].max_pages * upp * mc::kPage > 0x7fffffffLL) return MC_ERR_UNSUPPORTED;
  if (d->dtype == MC_FP8_E4M3 && lr != 0) return MC_ERR_UNSUPPORTED;   // page scales are per 16-token page
  if (d->dtype != MC_F32 && d->dtype != MC_BF16 && d->dtype != MC_FP8_E4M3) return MC_ERR_UNSUPPORTED;
  if (d->head_dim != 64 && d->head_dim != 128 && d->head_dim != 256) return MC_ERR_UNSUPPORTED;
  if ((long long)d->batch * d->num_q_heads > (1ll << 30)) return MC_ERR_UNSUPPORTED;
  const bool fp8 = d->dtype == MC_FP8_E4M3;
  if (fp8 && (!d->k_scale || !d->v_scale || (reinterpret_cast<uintptr_t>(d->k_scale) & 3u) ||
              (reinterpret_cast<uintptr_t>(d->v_scale) & 3u)))
    return MC_ERR_INVALID_ARG;
  if (fp8 && (d->head_dim != 128 || d->num_q_heads / d->num_kv_heads > 8)) return MC_ERR_UNSUPPORTED;

  Layout *L = new (std::nothrow) Layout();
  if (!L) return MC_ERR_OUT_OF_MEMORY;
  L->desc = *d;
  L->n_outer = n_outer;
  L->io_dtype = fp8 ? MC_BF16 : d->dtype;
  L->fp8 = nullptr;
  L->x_n = 0;
  L->n_unit_tab = 0;
  L->unit_buf = nullptr;
  mc::Params &p = L->p;
  p.k_pool = d->k_pool; p.v_pool = d->v_pool;
  p.group_offsets = d->group_offsets; p.prefix_pages = d->prefix_pages; p.prefix_len = d->prefix_len;
  p.suffix_pages = d->suffix_pages; p.suffix_len = d->suffix_len;
  p.G = d->num_groups; p.B = d->batch; p.Hq = d->num_q_heads; p.Hkv = d->num_kv_heads; p.d = d->head_dim;
  p.g = d->num_q_heads / d->num_kv_heads;
  p.lr = lr;
  p.num_pages = d->num_pages * upp; p.max_pp = d->max_prefix_pages * upp; p.max_sp = d->max_suffix_pages * upp;
  p.row_limit = nullptr;
  p.k_scale = fp8 ? d->k_scale : nullptr;
  p.v_scale = fp8 ? d->v_scale : nullptr;
  for (int k = 0; k < n_outer; ++k) {   // an outer level is the same cache seen through another group map
    mc::Params &po = L->outer_p[k];
    po = p;
    po.G = outer[k].num_groups;
    po.group_offsets = outer[k].group_offsets;
    po.prefix_pages = outer[k].pages;
    po.prefix_len = outer[k].len;
    po.max_pp = outer[k].max_pages * upp;
    po.row_limit = outer[k].row_limit;
  }
  if (lr > 0) {   // tables in unit pages, filled before anything below reads them
    long long total = 0;
    auto add = [&](const int32_t *src, long long n) {
      L->unit_tab[L->n_unit_tab++] = {src, reinterpret_cast<int32_t *>((uintptr_t)total), n};   // dst: offset for now
      total += ((n << lr) + 63) & ~63ll;
    };
    add(d->prefix_pages, (long long)d->num_groups * d->max_prefix_pages);
    if (d->max_suffix_pages > 0) add(d->suffix_pages, (long long)d->batch * d->max_suffix_pages);
    for (int k = 0; k < n_outer; ++k) add(outer[k].pages, (long long)outer[k].num_groups * outer[k].max_pages);
    if (cudaMalloc(&L->unit_buf, sizeof(int32_t) * (size_t)total) != cudaSuccess) {
      (void)cudaGetLastError();
      delete L;
      return MC_ERR_OUT_OF_MEMORY;
    }
    for (int i = 0; i < L->n_unit_tab; ++i)
      L->unit_tab[i].dst = L->unit_buf + reinterpret_cast<uintptr_t>(L->unit_tab[i].dst);
    int i = 0;
    p.prefix_pages = L->unit_tab[i++].dst;
    if (d->max_suffix_pages > 0) p.suffix_pages = L->unit_tab[i++].dst;
    for (int k = 0; k < n_outer; ++k) {
      L->outer_p[k].prefix_pages = L->unit_tab[i++].dst;
      L->outer_p[k].suffix_pages = p.suffix_pages;
    }
    if (mc::launch_unit_tables(L, nullptr) != MC_OK || cudaStreamSynchronize(nullptr) != cudaSuccess) {
      (void)cudaGetLastError();
      cudaFree(L->unit_buf);
      delete L;
      return MC_ERR_CUDA;
    }
  }

  // Part geometry.  Suffix chunks come from the table stride (the lengths live on the device and may grow).
  // Prefix splits and the CTAs of the tensor-core prefix pass are sized once per level from the lengths as they
  // are now.  The prefix pass runs beside the suffix pass and should end well inside the suffix pass's HBM time;
  // every work item (one token range of one 128-row tile) pays a fixed prologue/epilogue, so items should be
  // long: as few splits as still let one item fit that time.  Constants are measured for this kernel pair.
  const int max_s = p.max_sp * mc::kPage;
  double suffix_us = 0.0, suffix_tokens_now = -1.0;
  int32_t *sl = nullptr;
  {
    sl = new (std::nothrow) int32_t[p.B];
    if (sl && max_s > 0 && cudaMemcpy(sl, d->suffix_len, sizeof(int32_t) * p.B, cudaMemcpyDeviceToHost) == cudaSuccess) {
      double suffix_tokens = 0.0;
      for (int b = 0; b < p.B; ++b) suffix_tokens += sl[b] > 0 ? sl[b] : 0;
      suffix_us = suffix_tokens * 2.0 * p.Hkv * p.d * (d->dtype == MC_F32 ? 4 : fp8 ? 1 : 2) / 6.8e6;   // stream at ~6.8 TB/s
      suffix_tokens_now = suffix_tokens;
    } else {
      delete[] sl;
      sl = nullptr;
    }
    (void)cudaGetLastError();
  }
  // A chunk costs its warp about 4 us of start-up and wind-down besides its pages (measured), so chunks are long:
  // about 4 per row, 512..4096 tokens (cfg3: 8.7 % faster with 2048-token chunks than with 512)
  int ts = mc::pow2_floor(max_s / 4 > 512 ? max_s / 4 : 512);
  if (ts > 4096) ts = 4096;
  if (suffix_tokens_now >= 0.0) {
    // A small problem cannot keep every warp slot (6 per SM) busy with chunks of that size: shorter chunks, so that
    // a slot gets about 1.6 full chunks and the partial chunks of the rows fill the end of the launch - to the nearest
    // 128 tokens, down to 4 pages a chunk.
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      sms = 148;
    (void)cudaGetLastError();
    const double per_chunk = suffix_tokens_now * p.Hkv / (6.0 * sms) / 1.6;
    int tpar = per_chunk < 128.0 ? mc::pow2_floor(per_chunk < 64.0 ? 64 : (int)per_chunk)
                                 : per_chunk > 4096.0 ? 4096 : ((int)per_chunk + 64) / 128 * 128;
    if (tpar < ts) ts = tpar;
  }
  if (mc::env_int("MC_SUFFIX_PART_TOKENS", 0) > 0) ts = mc::env_int("MC_SUFFIX_PART_TOKENS", ts) / mc::kPage * mc::kPage;
  if (ts < mc::kPage) ts = mc::kPage;
  // The levels of the cascade share one persistent grid, so every item has the whole budget.
  const bool want_tc = mc::env_int("MC_PREFIX_TC", 1) && !mc::env_int("MC_FORCE_FMA", 0);
  mc::LevelWork work[1 + mc::kMaxOuterLevels];
  int nsp[1 + mc::kMaxOuterLevels];
  const double budget_us = suffix_us * 0.9;
  int part_base = 0;
  for (int k = 0; k <= n_outer; ++k) {   // k = 0: the base level; part slots in this order, then the suffix chunks
    mc::Params &pk = k == 0 ? p : L->outer_p[k - 1];
    work[k] = mc::level_work(pk);
    nsp[k] = mc::choose_splits(pk, work[k], budget_us);
    const int max_p = pk.max_pp * mc::kPage;
    int tp = ((max_p + nsp[k] - 1) / nsp[k] + 127) / 128 * 128;
    if (mc::env_int("MC_PREFIX_PART_TOKENS", 0) > 0)
      tp = mc::env_int("MC_PREFIX_PART_TOKENS", tp) / mc::kPage * mc::kPage;
    if (tp < mc::kPage) tp = mc::kPage;
    pk.prefix_part_tokens = tp;
    pk.n_prefix_parts = (max_p + tp - 1) / tp;
    pk.prefix_part_base = part_base;
    part_base += pk.n_prefix_parts;
  }
  const int n_parts = part_base + (max_s + ts - 1) / ts;
  for (int k = 0; k <= n_outer; ++k) {
    mc::Params &pk = k == 0 ? p : L->outer_p[k - 1];
    pk.suffix_part_tokens = ts;
    pk.suffix_part_base = part_base;
    pk.n_parts = n_parts;
  }
  L->use_mma = mc::mma_supported(p, d->dtype) && !mc::env_int("MC_FORCE_FMA", 0);
  L->has_suffix = n_parts > part_base;
  L->sfx_plan = L->has_suffix && L->use_mma && mc::env_int("MC_SUFFIX_TMA", 1) ? mc::suffix_tma_plan(p, d->dtype) : nullptr;
  if (fp8 && !(L->fp8 = mc::fp8_plan(p))) {
    delete[] sl;
    cudaFree(L->unit_buf);
    delete L;
    return MC_ERR_UNSUPPORTED;
  }
  // Suffix CTAs are launched longest first (by the lengths as they are now; appends change them slowly), so
  // that the launch ends on short items instead of a few long ones.  Without it the order is as numbered.
  L->suffix_order = nullptr;
  if ((L->use_mma || L->fp8) && sl && mc::env_int("MC_SUFFIX_ORDER", 1)) {
    const int per = L->fp8 ? mc::fp8_items_per_cta() : L->sfx_plan ? mc::suffix_tma_items_per_cta() : mc::mma_items_per_cta();
    const int n_chunks = n_parts - part_base;
    const long long n_items = (long long)p.B * p.Hkv * n_chunks, n_ctas = (n_items + per - 1) / per;
    if (n_ctas > 1 && n_ctas < (1ll << 24)) {
      std::vector<int32_t> order((size_t)n_ctas), key((size_t)n_ctas);
      for (long long c = 0; c < n_ctas; ++c) {
        int longest = 0;
        for (long long it = c * per; it < (c + 1) * per && it < n_items; ++it) {   // item = (b, chunk, kv head)
          const int chunk = (int)((it / p.Hkv) % n_chunks), b = (int)(it / ((long long)p.Hkv * n_chunks));
          int tokens = sl[b] - chunk * ts;
          tokens = tokens < 0 ? 0 : tokens > ts ? ts : tokens;
          if (tokens > longest) longest = tokens;
        }
        key[(size_t)c] = longest;
        order[(size_t)c] = (int32_t)c;
      }
      std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return key[a] > key[b]; });
      if (cudaMalloc(&L->suffix_order, sizeof(int32_t) * (size_t)n_ctas) != cudaSuccess ||
          cudaMemcpy(L->suffix_order, order.data(), sizeof(int32_t) * (size_t)n_ctas, cudaMemcpyHostToDevice) !=
              cudaSuccess) {
        cudaFree(L->suffix_order);
        L->suffix_order = nullptr;
        (void)cudaGetLastError();
      }
    }
  }
  delete[] sl;
  p.suffix_order = L->suffix_order;
  for (int k = 0; k < n_outer; ++k) L->outer_p[k].suffix_order = L->suffix_order;

  const size_t rows = (size_t)p.B * p.Hq, e = L->io_dtype == MC_F32 ? 4 : 2;
  L->o_part_bytes = mc::align_up(rows * p.n_parts * p.d * sizeof(float), 256);
  L->lse_part_bytes = mc::align_up(rows * p.n_parts * sizeof(float), 256);
  size_t off = L->o_part_bytes + L->lse_part_bytes;
  const size_t qb = mc::align_up(rows * p.d * e, 256), kvb = mc::align_up((size_t)p.B * p.Hkv * p.d * e, 256);
  const size_t sizes[5] = {qb, kvb, kvb, qb, mc::align_up(rows * sizeof(float), 256)};  // q, k_new, v_new, o, lse
  for (int i = 0; i < 5; ++i) { L->staging_off[i] = off; off += sizes[i]; }
  L->ws_bytes = off;

  if (cudaMalloc(&L->dev_status, 256) != cudaSuccess) {
    cudaFree(L->suffix_order);
    cudaFree(L->unit_buf);
    mc::suffix_tma_plan_free(L->sfx_plan);
    mc::fp8_plan_free(L->fp8);
    delete L;
    return MC_ERR_OUT_OF_MEMORY;
  }
  if (cudaMemset(L->dev_status, 0, 256) != cudaSuccess ||
      cudaMallocHost(&L->host_status, sizeof(int32_t)) != cudaSuccess) {
    cudaFree(L->dev_status);
    cudaFree(L->suffix_order);
    cudaFree(L->unit_buf);
    mc::suffix_tma_plan_free(L->sfx_plan);
    mc::fp8_plan_free(L->fp8);
    delete L;
    return MC_ERR_CUDA;
  }
  *L->host_status = 0;
  p.status = L->dev_status;
  for (int k = 0; k < n_outer; ++k) L->outer_p[k].status = L->dev_status;

  // Tensor-core prefix pass: tensor maps over the pools and the persistent grid of each level.
  L->tc_plan = nullptr;
  if (want_tc) {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess) {
      // outermost level first: its items are the ones with the most rows
      mc::Params levels[1 + mc::kMaxOuterLevels];
      int max_group[1 + mc::kMaxOuterLevels];
      bool all = true;
      for (int k = n_outer, i = 0; k >= 0; --k, ++i) {
        levels[i] = k == 0 ? p : L->outer_p[k - 1];
        max_group[i] = work[k].max_group;
        all = all && mc::prefix_tc_supported(levels[i], MC_BF16) && (fp8 || d->dtype == MC_BF16) && max_group[i] <= p.B;
      }
      // The suffix pass reaches the memory roofline from little more than half of the SMs and cannot share an SM
      // with a prefix CTA, so the prefix pass gets enough CTAs to end early (a tenth of the suffix pass's time,
      // measured alone; beside the suffix stream it runs about a third longer) and frees its SMs for the rest.
      const float *k_scale = nullptr;
      if (all && fp8) {
        // An e4m3 cache: the pass runs on the prefix levels widened once to 16-bit pools of their own (the prefix
        // does not change while candidates decode; mc_kv_layout_refresh_prefix repeats the widening).
        mc::Params widened[1 + mc::kMaxOuterLevels];
        all = mc::fp8_expand_alloc(L->fp8, levels, n_outer + 1, widened) &&
              mc::fp8_expand_launch(L->fp8, levels, n_outer + 1, nullptr) == MC_OK &&
              cudaStreamSynchronize(nullptr) == cudaSuccess;
        if (all) {
          L->x_n = n_outer + 1;
          for (int i = 0; i <= n_outer; ++i) {
            L->x_src[i] = levels[i];
            levels[i] = widened[i];
          }
          L->xp = widened[n_outer];
          k_scale = mc::fp8_expanded_k_scale(L->fp8);
        }
      }
      if (all)
        L->tc_plan = mc::prefix_tc_plan(levels, max_group, n_outer + 1, sms, mc::env_int("MC_PREFIX_CTAS", 0),
                                        0.1 * budget_us, mc::kTileUs, mc::kItemUs, k_scale);
    }
    (void)cudaGetLastError();
  }
  L->pdl = mc::env_int("MC_PDL", 1) != 0;
  if (cudaStreamCreateWithFlags(&L->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&L->fork_ev, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&L->join_ev, cudaEventDisableTiming) != cudaSuccess) {
    mc_kv_layout_destroy(reinterpret_cast<mc_kv_layout_t *>(L));
    return MC_ERR_CUDA;
  }
  *out = reinterpret_cast<mc_kv_layout_t *>(L);
  return MC_OK;
}

mc_status_t mc_kv_layout_destroy(mc_kv_layout_t *layout) {
  Layout *L = reinterpret_cast<Layout *>(layout);
  if (!L) return MC_OK;
  if (L->side_stream) cudaStreamDestroy(L->side_stream);
  if (L->fork_ev) cudaEventDestroy(L->fork_ev);
  if (L->join_ev) cudaEventDestroy(L->join_ev);
  mc::prefix_tc_plan_free(L->tc_plan);
  mc::suffix_tma_plan_free(L->sfx_plan);
  mc::fp8_plan_free(L->fp8);
  cudaFree(L->dev_status);
  cudaFree(L->suffix_order);
  cudaFree(L->unit_buf);
  cudaFreeHost(L->host_status);
  delete L;
  return MC_OK;
}

mc_status_t mc_kv_layout_refresh_tables(mc_kv_layout_t *layout, void *stream) {
  Layout *L = reinterpret_cast<Layout *>(layout);
  if (!L) return MC_ERR_INVALID_ARG;
  if (L->n_unit_tab == 0) return MC_OK;   // 16-token pages: the kernels read the caller's tables themselves
  return mc::launch_unit_tables(L, reinterpret_cast<cudaStream_t>(stream));
}

mc_status_t mc_kv_layout_refresh_prefix(mc_kv_layout_t *layout, void *stream) {
  Layout *L = reinterpret_cast<Layout *>(layout);
  if (!L) return MC_ERR_INVALID_ARG;
  if (!L->fp8 || L->x_n == 0) return MC_OK;   // nothing is kept: every pass reads the pools themselves
  return mc::fp8_expand_launch(L->fp8, L->x_src, L->x_n, reinterpret_cast<cudaStream_t>(stream));
}

mc_status_t mc_kv_layout_geometry(const mc_kv_layout_t *layout, mc_part_geometry_t *g) {
  const Layout *L = reinterpret_cast<const Layout *>(layout);
  if (!L || !g) return MC_ERR_INVALID_ARG;
  g->rows = L->p.B * L->p.Hq;
  g->n_parts = L->p.n_parts;
  g->n_prefix_parts = L->p.suffix_part_base;   // all prefix levels together (base level first)
  g->prefix_part_tokens = L->p.prefix_part_tokens;
  g->suffix_part_tokens = L->p.suffix_part_tokens;
  g->head_dim = L->p.d;
  g->prefix_ctas = mc::prefix_tc_grid(L->tc_plan);
  return MC_OK;
}

size_t mc_workspace_bytes(const mc_kv_layout_t *layout) {
  const Layout *L = reinterpret_cast<const Layout *>(layout);
  return L ? L->ws_bytes : 0;
}

mc_status_t mc_get_last_status(mc_kv_layout_t *layout, void *stream) {
  Layout *L = reinterpret_cast<Layout *>(layout);
  if (!L) return MC_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(L->host_status, L->dev_status, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemsetAsync(L->dev_status, 0, sizeof(int32_t), st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return MC_ERR_CUDA;
  const int32_t v = *L->host_status;
  return v >= MC_OK && v <= MC_ERR_TIMEOUT ? static_cast<mc_status_t>(v) : MC_ERR_CUDA;
}

mc_status_t mc_kv_layout_validate(mc_kv_layout_t *layout, void *scratch, size_t scratch_bytes, void *stream) {
  Layout *L = reinterpret_cast<Layout *>(layout);
  if (!L || !scratch) return MC_ERR_INVALID_ARG;
  if (scratch_bytes < (size_t)L->p.num_pages * sizeof(int32_t)) return MC_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (L->n_unit_tab && mc::launch_unit_tables(L, st) != MC_OK) return MC_ERR_CUDA;   // check the tables as they are now
  if (cudaMemsetAsync(scratch, 0, (size_t)L->p.num_pages * sizeof(int32_t), st) != cudaSuccess) return MC_ERR_CUDA;
  mc::validate_kernel<<<148, 256, 0, st>>>(L->p, reinterpret_cast<int32_t *>(scratch), 1);
  mc::count_launch();
  for (int k = 0; k < L->n_outer; ++k) {   // outer levels: their own prefix tables, same reference counts
    mc::validate_kernel<<<148, 256, 0, st>>>(L->outer_p[k], reinterpret_cast<int32_t *>(scratch), 0);
    mc::count_launch();
  }
  if (mc::check_launch() != MC_OK) return MC_ERR_CUDA;
  return mc_get_last_status(layout, stream);
}

mc_status_t mc_kv_append(mc_kv_layout_t *layout, const void *k_new, const void *v_new, void *stream) {
  Layout *L = reinterpret_cast<Layout *>(layout);
  if (!L || !k_new || !v_new || !mc::aligned16(k_new) || !mc::aligned16(v_new)) return MC_ERR_INVALID_ARG;
  if (!L->has_suffix) return MC_ERR_INVALID_ARG;   // a layout without private tokens has nowhere to append
  if (L->fp8) return mc::launch_append_fp8(L->p, k_new, v_new, L->desc.suffix_len, reinterpret_cast<cudaStream_t>(stream));
  const int e = L->desc.dtype == MC_F32 ? 4 : 2;
  mc::append_kernel<<<L->p.B, 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      L->p, reinterpret_cast<const uint4 *>(k_new), reinterpret_cast<const uint4 *>(v_new), L->desc.suffix_len, e);
  mc::count_launch();
  return mc::check_launch();
}

mc_status_t mc_kv_append_rope(mc_kv_layout_t *layout, const void *k_new, const void *v_new, void *q,
                              const int32_t *pos_offset, double theta_base, void *stream) {
  Layout *L = reinterpret_cast<Layout *>(layout);
  if (!L || !k_new || !v_new || !mc::aligned16(k_new) || !mc::aligned16(v_new) || (q && !mc::aligned16(q)))
    return MC_ERR_INVALID_ARG;
  if (!L->has_suffix || !(theta_base > 0.0) || L->p.d % 2 != 0 || 256 % (L->p.d / 2) != 0) return MC_ERR_INVALID_ARG;
  if (L->fp8) return MC_ERR_UNSUPPORTED;   // the rotary append does not quantise
  mc::RopeLevels lv;
  lv.n = 1 + L->n_outer;
  for (int k = 0; k < lv.n; ++k) {
    const mc::Params &pk = k == 0 ? L->p : L->outer_p[k - 1];
    lv.G[k] = pk.G;
    lv.group_offsets[k] = pk.group_offsets;
    lv.prefix_len[k] = pk.prefix_len;
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const double l2b = std::log2(theta_base);
  if (L->desc.dtype == MC_F32)
    mc::append_rope_kernel<float><<<L->p.B, 256, 0, st>>>(L->p, lv, reinterpret_cast<const float *>(k_new),
                                                          reinterpret_cast<const uint4 *>(v_new),
                                                          reinterpret_cast<float *>(q), pos_offset, l2b,
                                                          L->desc.suffix_len);
  else
    mc::append_rope_kernel<__nv_bfloat16><<<L->p.B, 256, 0, st>>>(
        L->p, lv, reinterpret_cast<const __nv_bfloat16 *>(k_new), reinterpret_cast<const uint4 *>(v_new),
        reinterpret_cast<__nv_bfloat16 *>(q), pos_offset, l2b, L->desc.suffix_len);
  mc::count_launch();
  return mc::check_launch();
}

struct mc_qkv_plan {
  Layout *L;
  mc::QkvPlan *gemm;
  const void *bias;
  void *token_info;       // device: per candidate, where its new token goes (QkvToken [B]) and, 256-byte aligned
                          // behind that, the rotation of its 64 pairs (float2 [B][64])
};

mc_status_t mc_qkv_plan_create(mc_kv_layout_t *layout, const void *w_qkv, const void *bias, int32_t hidden,
                               mc_qkv_plan_t **out) {
  if (out) *out = nullptr;
  Layout *L = reinterpret_cast<Layout *>(layout);
  if (!L || !out || !w_qkv || !mc::aligned16(w_qkv) || (bias && (reinterpret_cast<uintptr_t>(bias) & 1u)))
    return MC_ERR_INVALID_ARG;
  if (hidden < 64 || hidden % 64 != 0) return MC_ERR_INVALID_ARG;
  if (L->desc.dtype != MC_BF16 || L->p.d != 128 || !L->has_suffix) return MC_ERR_UNSUPPORTED;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    sms = 148;
  (void)cudaGetLastError();
  mc_qkv_plan *pl = new (std::nothrow) mc_qkv_plan();
  if (!pl) return MC_ERR_OUT_OF_MEMORY;
  pl->L = L;
  pl->bias = bias;
  pl->gemm = mc::qkv_plan(L->p.B, L->p.Hq + 2 * L->p.Hkv, hidden, w_qkv, sms);
  pl->token_info = nullptr;
  const size_t tok_bytes = mc::align_up(sizeof(mc::QkvToken) * (size_t)L->p.B, 256);
  if (!pl->gemm || cudaMalloc(&pl->token_info, tok_bytes + sizeof(float2) * 64 * (size_t)L->p.B) != cudaSuccess) {
    (void)cudaGetLastError();
    mc::qkv_plan_free(pl->gemm);
    delete pl;
    return MC_ERR_OUT_OF_MEMORY;
  }
  *out = pl;
  return MC_OK;
}

mc_status_t mc_qkv_plan_destroy(mc_qkv_plan_t *plan) {
  if (!plan) return MC_OK;
  mc::qkv_plan_free(plan->gemm);
  cudaFree(plan->token_info);
  delete plan;
  return MC_OK;
}

mc_status_t mc_qkv_plan_geometry(const mc_qkv_plan_t *plan, int32_t *pieces, int32_t *ctas, size_t *workspace_bytes) {
  if (!plan) return MC_ERR_INVALID_ARG;
  if (pieces) *pieces = mc::qkv_pieces(plan->gemm);
  if (ctas) *ctas = mc::qkv_ctas(plan->gemm) * mc::qkv_passes(plan->gemm);
  if (workspace_bytes) *workspace_bytes = mc::qkv_workspace_bytes(plan->gemm);
  return MC_OK;
}

mc_status_t mc_qkv_append(mc_qkv_plan_t *plan, const void *x, void *q_out, const int32_t *pos_offset,
                          double theta_base, void *stream) {
  if (!plan || !x || !q_out || !mc::aligned16(x) || !mc::aligned16(q_out)) return MC_ERR_INVALID_ARG;
  if (theta_base < 0.0 || (theta_base == 0.0 && pos_offset)) return MC_ERR_INVALID_ARG;
  Layout *L = plan->L;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  mc::RopeLevels lv;
  lv.n = 1 + L->n_outer;
  for (int k = 0; k < lv.n; ++k) {
    const mc::Params &pk = k == 0 ? L->p : L->outer_p[k - 1];
    lv.G[k] = pk.G;
    lv.group_offsets[k] = pk.group_offsets;
    lv.prefix_len[k] = pk.prefix_len;
  }
  mc::QkvToken *tok = reinterpret_cast<mc::QkvToken *>(plan->token_info);
  float2 *rot = reinterpret_cast<float2 *>(static_cast<unsigned char *>(plan->token_info) +
                                           mc::align_up(sizeof(mc::QkvToken) * (size_t)L->p.B, 256));
  const bool pdl = mc::env_int("MC_PDL", 1) != 0;
  mc::qkv_prep_kernel<<<L->p.B, 64, 0, st>>>(L->p, lv, pos_offset, theta_base > 0.0 ? std::log2(theta_base) : 0.0,
                                            L->desc.suffix_len, tok, rot);
  mc::count_launch();
  if (mc::check_launch() != MC_OK) return MC_ERR_CUDA;
  mc_status_t s = mc::launch_qkv_gemm(plan->gemm, x, L->dev_status, st, pdl);
  if (s != MC_OK) return s;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)L->p.B, (unsigned)((L->p.Hq + 2 * L->p.Hkv + 15) / 16));
  cfg.blockDim = dim3(256);
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = pdl ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(
      &cfg, mc::qkv_finish_kernel, L->p, mc::qkv_partials(plan->gemm), mc::qkv_ctas(plan->gemm),
      mc::qkv_kb_per_pair(plan->gemm), (L->p.Hq + 2 * L->p.Hkv + 1) / 2, mc::qkv_row_stride(plan->gemm),
      mc::qkv_feature_stride(plan->gemm), reinterpret_cast<const __nv_bfloat16 *>(plan->bias),
      reinterpret_cast<__nv_bfloat16 *>(q_out), static_cast<const mc::QkvToken *>(tok), static_cast<const float2 *>(rot),
      theta_base > 0.0 ? 1 : 0);
  mc::count_launch();
  return e == cudaSuccess ? mc::check_launch() : MC_ERR_CUDA;
}

mc_status_t mc_kv_append_tokens(mc_kv_layout_t *layout, const void *k_new, const void *v_new, int32_t n_max,
                                const int32_t *n_new, void *q, const int32_t *pos_offset, double theta_base,
                                void *stream) {
  Layout *L = reinterpret_cast<Layout *>(layout);
  if (!L || !k_new || !v_new || !mc::aligned16(k_new) || !mc::aligned16(v_new) || (q && !mc::aligned16(q)))
    return MC_ERR_INVALID_ARG;
  if (!L->has_suffix || n_max < 0 || n_max > 65535 || theta_base < 0.0) return MC_ERR_INVALID_ARG;
  if (theta_base == 0.0 && (q || pos_offset)) return MC_ERR_INVALID_ARG;   // they belong to the rotation
  if (theta_base > 0.0 && (L->p.d % 2 != 0 || 256 % (L->p.d / 2) != 0)) return MC_ERR_INVALID_ARG;
  if (n_max == 0) return MC_OK;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (L->fp8) {
    if (theta_base > 0.0) return MC_ERR_UNSUPPORTED;   // the rotary append does not quantise
    const mc_status_t s = mc::launch_append_tokens_fp8(L->p, k_new, v_new, n_max, n_new, L->desc.suffix_len, st);
    if (s != MC_OK) return s;
  } else {
    mc::RopeLevels lv;
    lv.n = 1 + L->n_outer;
    for (int k = 0; k < lv.n; ++k) {
      const mc::Params &pk = k == 0 ? L->p : L->outer_p[k - 1];
      lv.G[k] = pk.G;
      lv.group_offsets[k] = pk.group_offsets;
      lv.prefix_len[k] = pk.prefix_len;
    }
    const double l2b = theta_base > 0.0 ? std::log2(theta_base) : 0.0;
    if (theta_base == 1.0) return MC_ERR_INVALID_ARG;   // log2 = 0 is the "no rotation" mark (and base 1 rotates every pair alike)
    const dim3 grid((unsigned)n_max, (unsigned)L->p.B);
    if (L->desc.dtype == MC_F32)
      mc::append_tokens_kernel<float><<<grid, 256, 0, st>>>(L->p, lv, reinterpret_cast<const float *>(k_new),
                                                            reinterpret_cast<const float *>(v_new),
                                                            reinterpret_cast<float *>(q), n_max, n_new, pos_offset, l2b,
                                                            L->desc.suffix_len);
    else
      mc::append_tokens_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(
          L->p, lv, reinterpret_cast<const __nv_bfloat16 *>(k_new), reinterpret_cast<const __nv_bfloat16 *>(v_new),
          reinterpret_cast<__nv_bfloat16 *>(q), n_max, n_new, pos_offset, l2b, L->desc.suffix_len);
    mc::count_launch();
  }
  mc::advance_len_kernel<<<(L->p.B + 255) / 256, 256, 0, st>>>(L->p, n_max, n_new, L->desc.suffix_len);
  mc::count_launch();
  return mc::check_launch();
}

mc_status_t mc_prefix_attn(mc_kv_layout_t *layout, const void *q, float scale, float *o_part, float *lse_part,
                           void *stream) {
  Layout *L = reinterpret_cast<Layout *>(layout);
  mc_status_t s = mc::check_q(L, q);
  if (s != MC_OK) return s;
  if (!o_part || !lse_part || !mc::aligned16(o_part)) return MC_ERR_INVALID_ARG;
  return mc::run_pass(L, mc::kPrefix, q, scale, o_part, lse_part, reinterpret_cast<cudaStream_t>(stream));
}

mc_status_t mc_suffix_attn(mc_kv_layout_t *layout, const void *q, float scale, float *o_part, float *lse_part,
                           void *stream) {
  Layout *L = reinterpret_cast<Layout *>(layout);
  mc_status_t s = mc::check_q(L, q);
  if (s != MC_OK) return s;
  if (!o_part || !lse_part || !mc::aligned16(o_part)) return MC_ERR_INVALID_ARG;
  return mc::run_pass(L, mc::kSuffix, q, scale, o_part, lse_part, reinterpret_cast<cudaStream_t>(stream));
}

mc_status_t mc_merge_lse(mc_kv_layout_t *layout, const float *o_part, const float *lse_part, void *o, float *lse,
                         void *stream) {
  Layout *L = reinterpret_cast<Layout *>(layout);
  if (!L || !o_part || !lse_part || !o || !lse || !mc::aligned16(o_part) || !mc::aligned16(o))
    return MC_ERR_INVALID_ARG;
  return mc::launch_merge(L->p, L->io_dtype, o_part, lse_part, o, lse, reinterpret_cast<cudaStream_t>(stream));
}

static mc_status_t decode_impl(mc_kv_layout_t *layout, const void *k_new, const void *v_new, const void *q,
                               float scale, void *o, float *lse, void *ws, size_t ws_bytes, void *stream) {
  Layout *L = reinterpret_cast<Layout *>(layout);
  mc_status_t s = mc::check_q(L, q);
  if (s != MC_OK) return s;
  if (!o || !lse || !ws || !mc::aligned16(o)) return MC_ERR_INVALID_ARG;
  if ((k_new == nullptr) != (v_new == nullptr)) return MC_ERR_INVALID_ARG;
  if (k_new && (!mc::aligned16(k_new) || !mc::aligned16(v_new))) return MC_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return MC_ERR_INVALID_ARG;
  if (ws_bytes < L->ws_bytes) return MC_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  float *o_part = reinterpret_cast<float *>(ws);
  float *lse_part = reinterpret_cast<float *>(static_cast<char *>(ws) + L->o_part_bytes);
  // The two passes write disjoint part slots and run side by side.  The prefix pass (tensor-bound, a few
  // persistent CTAs, each needing an SM's whole shared memory) must get its CTAs placed before the suffix pass
  // (HBM-bound, thousands of short CTAs) fills every SM.
  if (L->tc_plan && scale != 0.f && !L->has_suffix && mc::prefix_tc_one_part_per_row(L->tc_plan) &&
      mc::env_int("MC_PREFIX_DIRECT", 1)) {
    // No private tokens and one part per row from the prefix pass: it writes the final output itself, no merge.
    if (k_new) return MC_ERR_INVALID_ARG;   // nowhere to append
    return mc::launch_prefix_tc(L->fp8 ? L->xp : L->p, L->tc_plan, q, scale, o_part, lse_part, st, o, lse);
  }
  if (L->tc_plan && (L->use_mma || L->fp8) && scale != 0.f && L->pdl) {
    // One stream: the suffix pass is launched behind the tensor-core prefix pass as its programmatic
    // dependent, so it starts once every prefix CTA is running, not when they end.  The order holds when
    // the step is replayed from a captured graph.  The merge, launched the ordinary way, waits for both.
    if (k_new && (s = mc_kv_append(layout, k_new, v_new, st)) != MC_OK) return s;
    // Behind an append of its own the prefix pass is launched as that kernel's programmatic dependent: it needs
    // nothing of the append, so its start-up runs beside it; the suffix pass, which does, is released by the
    // prefix CTAs only after they have seen the append grid complete (MC_PDL_APPEND=0: an ordinary launch).
    const bool early = k_new != nullptr && mc::env_int("MC_PDL_APPEND", 1);
    if ((s = mc::launch_prefix_tc(L->fp8 ? L->xp : L->p, L->tc_plan, q, scale, o_part, lse_part, st, nullptr, nullptr,
                                  early)) != MC_OK)
      return s;
    if (L->has_suffix) {
      s = L->fp8        ? mc::launch_fp8(L->p, L->fp8, mc::kSuffix, q, scale, o_part, lse_part, st, true)
          : L->sfx_plan ? mc::launch_suffix_tma(L->p, L->sfx_plan, q, scale, o_part, lse_part, st, true)
                        : mc::launch_mma(L->p, mc::kSuffix, q, scale, o_part, lse_part, st, true);
      if (s != MC_OK) return s;
    }
    // The merge is the suffix pass's programmatic dependent in turn (MC_PDL_MERGE=0: an ordinary launch): its CTAs
    // are resident and waiting when the last suffix CTA ends, instead of being launched then.
    return mc::launch_merge(L->p, L->io_dtype, o_part, lse_part, o, lse, st,
                            L->has_suffix && (L->sfx_plan || L->fp8) && mc::env_int("MC_PDL_MERGE", 1));
  }
  // Otherwise two streams: the prefix pass first, on the caller's stream; the append (it touches only suffix
  // pages and lengths) and the suffix pass on the handle's side stream; the merge joins them.
  if (cudaEventRecord(L->fork_ev, st) != cudaSuccess ||
      cudaStreamWaitEvent(L->side_stream, L->fork_ev, 0) != cudaSuccess)
    return MC_ERR_CUDA;
  if ((s = mc::run_pass(L, mc::kPrefix, q, scale, o_part, lse_part, st)) != MC_OK) return s;
  if (k_new && (s = mc_kv_append(layout, k_new, v_new, L->side_stream)) != MC_OK) return s;
  if ((s = mc::run_pass(L, mc::kSuffix, q, scale, o_part, lse_part, L->side_stream)) != MC_OK) return s;
  if (cudaEventRecord(L->join_ev, L->side_stream) != cudaSuccess ||
      cudaStreamWaitEvent(st, L->join_ev, 0) != cudaSuccess)
    return MC_ERR_CUDA;
  return mc::launch_merge(L->p, L->io_dtype, o_part, lse_part, o, lse, st);
}

mc_status_t mc_decode_attn(mc_kv_layout_t *layout, const void *q, float scale, void *o, float *lse, void *ws,
                           size_t ws_bytes, void *stream) {
  return decode_impl(layout, nullptr, nullptr, q, scale, o, lse, ws, ws_bytes, stream);
}

mc_status_t mc_decode_step(mc_kv_layout_t *layout, const void *k_new, const void *v_new, const void *q, float scale,
                           void *o, float *lse, void *ws, size_t ws_bytes, void *stream) {
  return decode_impl(layout, k_new, v_new, q, scale, o, lse, ws, ws_bytes, stream);
}

mc_status_t mc_decode_step_host(mc_kv_layout_t *layout, const void *k_new_host, const void *v_new_host,
                                const void *q_host, float scale, void *o_host, float *lse_host, void *ws,
                                size_t ws_bytes, void *stream) {
  Layout *L = reinterpret_cast<Layout *>(layout);
  if (!L || !q_host || !o_host || !lse_host || !ws) return MC_ERR_INVALID_ARG;
  if ((k_new_host == nullptr) != (v_new_host == nullptr)) return MC_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return MC_ERR_INVALID_ARG;
  if (ws_bytes < L->ws_bytes) return MC_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  char *base = static_cast<char *>(ws);
  const size_t e = L->io_dtype == MC_F32 ? 4 : 2, rows = (size_t)L->p.B * L->p.Hq;
  const size_t q_bytes = rows * L->p.d * e, kv_bytes = (size_t)L->p.B * L->p.Hkv * L->p.d * e;
  void *q_dev = base + L->staging_off[0], *k_dev = base + L->staging_off[1], *v_dev = base + L->staging_off[2];
  void *o_dev = base + L->staging_off[3];
  float *lse_dev = reinterpret_cast<float *>(base + L->staging_off[4]);
  if (cudaMemcpyAsync(q_dev, q_host, q_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return MC_ERR_CUDA;
  mc_status_t s;
  if (k_new_host) {
    if (cudaMemcpyAsync(k_dev, k_new_host, kv_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(v_dev, v_new_host, kv_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return MC_ERR_CUDA;
  }
  if ((s = mc_decode_step(layout, k_new_host ? k_dev : nullptr, k_new_host ? v_dev : nullptr, q_dev, scale, o_dev,
                          lse_dev, ws, ws_bytes, stream)) != MC_OK)
    return s;
  if (cudaMemcpyAsync(o_host, o_dev, q_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemcpyAsync(lse_host, lse_dev, rows * sizeof(float), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return MC_ERR_CUDA;
  return MC_OK;
}

}  // extern "C"
