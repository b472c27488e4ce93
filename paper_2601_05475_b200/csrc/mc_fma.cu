// Plain-ALU split-KV attention: one warp per (candidate, query head, part), lanes split the head
// dimension, coalesced vector loads of each K/V row, warp-shuffle reduction of the dot product and an
// online softmax.  Serves the fp32 dtype (no tensor-core format keeps 1e-5) and every shape the
// tensor-core kernels do not cover.
#include "mc_internal.cuh"

namespace mc {
namespace {

template <typename T, int VEC>
struct RowLoad;

template <>
struct RowLoad<float, 2> {
  static __device__ __forceinline__ void ld(const float *p, float (&o)[2]) {
    float2 v = __ldg(reinterpret_cast<const float2 *>(p));
    o[0] = v.x; o[1] = v.y;
  }
};
template <>
struct RowLoad<float, 4> {
  static __device__ __forceinline__ void ld(const float *p, float (&o)[4]) {
    float4 v = __ldg(reinterpret_cast<const float4 *>(p));
    o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
  }
};
template <>
struct RowLoad<float, 8> {
  static __device__ __forceinline__ void ld(const float *p, float (&o)[8]) {
    float4 a = __ldg(reinterpret_cast<const float4 *>(p)), b = __ldg(reinterpret_cast<const float4 *>(p) + 1);
    o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w;
    o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
  }
};
__device__ __forceinline__ void unpack_bf16x2(uint32_t w, float &lo, float &hi) {
  lo = __uint_as_float(w << 16);
  hi = __uint_as_float(w & 0xffff0000u);
}
template <>
struct RowLoad<__nv_bfloat16, 2> {
  static __device__ __forceinline__ void ld(const __nv_bfloat16 *p, float (&o)[2]) {
    uint32_t w = __ldg(reinterpret_cast<const uint32_t *>(p));
    unpack_bf16x2(w, o[0], o[1]);
  }
};
template <>
struct RowLoad<__nv_bfloat16, 4> {
  static __device__ __forceinline__ void ld(const __nv_bfloat16 *p, float (&o)[4]) {
    uint2 w = __ldg(reinterpret_cast<const uint2 *>(p));
    unpack_bf16x2(w.x, o[0], o[1]);
    unpack_bf16x2(w.y, o[2], o[3]);
  }
};

template <>
struct RowLoad<__nv_bfloat16, 8> {
  static __device__ __forceinline__ void ld(const __nv_bfloat16 *p, float (&o)[8]) {
    uint4 w = __ldg(reinterpret_cast<const uint4 *>(p));
    unpack_bf16x2(w.x, o[0], o[1]);
    unpack_bf16x2(w.y, o[2], o[3]);
    unpack_bf16x2(w.z, o[4], o[5]);
    unpack_bf16x2(w.w, o[6], o[7]);
  }
};

constexpr int kWarpsPerBlock = 4;
constexpr int kTok = 4;  // tokens per inner iteration (independent shuffle chains)

template <typename T, int D, int MODE>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
attn_fma_kernel(Params p, const T *__restrict__ q, float scale_log2, float *__restrict__ o_part,
                float *__restrict__ lse_part) {
  constexpr int VEC = D / 32;
  const int lane = threadIdx.x & 31;
  const int nparts_mode = MODE == kPrefix ? p.n_prefix_parts : p.n_parts - p.suffix_part_base;
  const long long n_items = (long long)p.B * p.Hq * nparts_mode;
  const long long item = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  if (item >= n_items) return;
  const int part = (int)(item % nparts_mode);
  const int hq = (int)((item / nparts_mode) % p.Hq);
  const int b = (int)(item / ((long long)nparts_mode * p.Hq));
  const int h = hq / p.g;
  const Span sp = resolve_span<MODE>(p, b, part);
  const size_t row = (size_t)b * p.Hq + hq;
  float *o_dst = o_part + (row * p.n_parts + sp.part) * D + lane * VEC;
  float *lse_dst = lse_part + row * p.n_parts + sp.part;
  if (sp.lo >= sp.hi) {
    if (lane == 0) *lse_dst = -INFINITY;
    return;
  }
  float qv[VEC];
  RowLoad<T, VEC>::ld(q + row * D + lane * VEC, qv);
  const T *kp = reinterpret_cast<const T *>(p.k_pool);
  const T *vp = reinterpret_cast<const T *>(p.v_pool);

  float m = -INFINITY, l = 0.f, acc[VEC];
#pragma unroll
  for (int c = 0; c < VEC; ++c) acc[c] = 0.f;

  for (int t0 = sp.lo; t0 < sp.hi; t0 += kTok) {
    float s[kTok], vv[kTok][VEC];
    bool valid[kTok];
#pragma unroll
    for (int u = 0; u < kTok; ++u) {
      const int t = t0 + u;
      s[u] = 0.f;
#pragma unroll
      for (int c = 0; c < VEC; ++c) vv[u][c] = 0.f;
      bool ok = t < sp.hi;
      int page = ok ? __ldg(sp.pages + (t >> 4)) : 0;
      if (ok && (unsigned)page >= (unsigned)p.num_pages) {
        latch(p, kDevBadPage);
        ok = false;
      }
      if (ok) {
        const size_t off = (slab_index(p, page, h) * kPage + (t & 15)) * D + lane * VEC;
        float kv[VEC];
        RowLoad<T, VEC>::ld(kp + off, kv);
        RowLoad<T, VEC>::ld(vp + off, vv[u]);
#pragma unroll
        for (int c = 0; c < VEC; ++c) s[u] = fmaf(qv[c], kv[c], s[u]);
      }
      valid[u] = ok;  // warp-uniform
    }
#pragma unroll
    for (int sh = 16; sh >= 1; sh >>= 1) {
#pragma unroll
      for (int u = 0; u < kTok; ++u) s[u] += __shfl_xor_sync(0xffffffffu, s[u], sh);
    }
    float mx = m;
#pragma unroll
    for (int u = 0; u < kTok; ++u) {
      s[u] = valid[u] ? s[u] * scale_log2 : -INFINITY;
      mx = fmaxf(mx, s[u]);
    }
    if (mx == -INFINITY) continue;  // nothing valid seen yet (only bad pages so far)
    const float alpha = exp2f(m - mx);
    l *= alpha;
#pragma unroll
    for (int c = 0; c < VEC; ++c) acc[c] *= alpha;
#pragma unroll
    for (int u = 0; u < kTok; ++u) {
      const float pu = exp2f(s[u] - mx);
      l += pu;
#pragma unroll
      for (int c = 0; c < VEC; ++c) acc[c] = fmaf(pu, vv[u][c], acc[c]);
    }
    m = mx;
  }
  if (l > 0.f) {
    const float inv = 1.f / l;
#pragma unroll
    for (int c = 0; c < VEC; ++c) o_dst[c] = acc[c] * inv;
    if (lane == 0) *lse_dst = (m + log2f(l)) * kLn2;
  } else if (lane == 0) {
    *lse_dst = -INFINITY;
  }
}

template <typename T, int D>
mc_status_t launch_t(const Params &p, int mode, const void *q, float scale, float *o_part, float *lse_part,
                     cudaStream_t stream) {
  const int nparts_mode = mode == kPrefix ? p.n_prefix_parts : p.n_parts - p.suffix_part_base;
  const long long n_items = (long long)p.B * p.Hq * nparts_mode;
  if (n_items == 0) return MC_OK;
  const unsigned grid = (unsigned)((n_items + kWarpsPerBlock - 1) / kWarpsPerBlock);
  const float sl2 = scale * kLog2e;
  if (mode == kPrefix)
    attn_fma_kernel<T, D, kPrefix><<<grid, kWarpsPerBlock * 32, 0, stream>>>(p, (const T *)q, sl2, o_part, lse_part);
  else
    attn_fma_kernel<T, D, kSuffix><<<grid, kWarpsPerBlock * 32, 0, stream>>>(p, (const T *)q, sl2, o_part, lse_part);
  count_launch();
  return check_launch();
}

}  // namespace

mc_status_t launch_fma(const Params &p, int dtype, int mode, const void *q, float scale, float *o_part,
                       float *lse_part, cudaStream_t stream) {
  if (dtype == MC_F32) {
    if (p.d == 64) return launch_t<float, 64>(p, mode, q, scale, o_part, lse_part, stream);
    if (p.d == 128) return launch_t<float, 128>(p, mode, q, scale, o_part, lse_part, stream);
    if (p.d == 256) return launch_t<float, 256>(p, mode, q, scale, o_part, lse_part, stream);
  } else if (dtype == MC_BF16) {
    if (p.d == 64) return launch_t<__nv_bfloat16, 64>(p, mode, q, scale, o_part, lse_part, stream);
    if (p.d == 128) return launch_t<__nv_bfloat16, 128>(p, mode, q, scale, o_part, lse_part, stream);
    if (p.d == 256) return launch_t<__nv_bfloat16, 256>(p, mode, q, scale, o_part, lse_part, stream);
  }
  return MC_ERR_UNSUPPORTED;
}

}  // namespace mc
