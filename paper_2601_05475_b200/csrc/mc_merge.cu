// Log-sum-exp merge of the per-part partial results: one warp per output row, lanes split the head
// dimension.  Reads only the parts whose lse is finite, several of them at a time.
#include "mc_internal.cuh"

namespace mc {
namespace {

constexpr int kWarpsPerBlock = 4;

template <typename T, int VEC>
__device__ __forceinline__ void store_row(T *dst, const float (&v)[VEC]);

template <>
__device__ __forceinline__ void store_row<float, 2>(float *dst, const float (&v)[2]) {
  *reinterpret_cast<float2 *>(dst) = make_float2(v[0], v[1]);
}
template <>
__device__ __forceinline__ void store_row<float, 4>(float *dst, const float (&v)[4]) {
  *reinterpret_cast<float4 *>(dst) = make_float4(v[0], v[1], v[2], v[3]);
}
template <>
__device__ __forceinline__ void store_row<float, 8>(float *dst, const float (&v)[8]) {
  reinterpret_cast<float4 *>(dst)[0] = make_float4(v[0], v[1], v[2], v[3]);
  reinterpret_cast<float4 *>(dst)[1] = make_float4(v[4], v[5], v[6], v[7]);
}
template <>
__device__ __forceinline__ void store_row<__nv_bfloat16, 2>(__nv_bfloat16 *dst, const float (&v)[2]) {
  *reinterpret_cast<__nv_bfloat162 *>(dst) = __floats2bfloat162_rn(v[0], v[1]);
}
template <>
__device__ __forceinline__ void store_row<__nv_bfloat16, 4>(__nv_bfloat16 *dst, const float (&v)[4]) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
  uint2 w;
  w.x = *reinterpret_cast<uint32_t *>(&a);
  w.y = *reinterpret_cast<uint32_t *>(&b);
  *reinterpret_cast<uint2 *>(dst) = w;
}

template <>
__device__ __forceinline__ void store_row<__nv_bfloat16, 8>(__nv_bfloat16 *dst, const float (&v)[8]) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
  __nv_bfloat162 c = __floats2bfloat162_rn(v[4], v[5]), d = __floats2bfloat162_rn(v[6], v[7]);
  uint4 w;
  w.x = *reinterpret_cast<uint32_t *>(&a);
  w.y = *reinterpret_cast<uint32_t *>(&b);
  w.z = *reinterpret_cast<uint32_t *>(&c);
  w.w = *reinterpret_cast<uint32_t *>(&d);
  *reinterpret_cast<uint4 *>(dst) = w;
}

template <typename T, int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
merge_lse_kernel(int rows, int n_parts, const float *__restrict__ o_part, const float *__restrict__ lse_part,
                 T *__restrict__ o, float *__restrict__ lse) {
  constexpr int VEC = D / 32;
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  // Launched as the programmatic dependent of the suffix pass, this grid's CTAs may become resident while that
  // pass's last CTAs still run; nothing is read before the prerequisite grid has completed and its writes are
  // visible (and through the suffix grid's own wait, the prefix pass's).  Launched the ordinary way, this
  // returns at once.
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  if (row >= rows) return;
  const float *lp = lse_part + (size_t)row * n_parts;
  float m = -INFINITY;
  for (int i = lane; i < n_parts; i += 32) m = fmaxf(m, lp[i]);
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, sh));
  float acc[VEC];
#pragma unroll
  for (int c = 0; c < VEC; ++c) acc[c] = 0.f;
  float s = 0.f;
  if (m > -INFINITY) {
    // Lane i of a batch holds the weight of part base + i; the rows of up to kBatch parts are then fetched together,
    // so the merge pays one memory round trip per batch and not one per part.  An empty part has weight 0 and its
    // row (which may hold anything) is not read.
    constexpr int kBatch = 8;
    const float *op = o_part + (size_t)row * n_parts * D + lane * VEC;
    for (int base = 0; base < n_parts; base += 32) {
      const float li = base + lane < n_parts ? lp[base + lane] : -INFINITY;
      const float w = li == -INFINITY ? 0.f : expf(li - m);
      s += w;
      const int cnt = min(32, n_parts - base);
      for (int i0 = 0; i0 < cnt; i0 += kBatch) {
        float wi[kBatch], v[kBatch][VEC];
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
          wi[k] = __shfl_sync(0xffffffffu, w, (i0 + k) & 31);   // lanes past the last part hold 0
          const float *src = op + (size_t)(base + i0 + k) * D;
          if constexpr (VEC == 8) {
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f), t2 = t;
            if (wi[k] != 0.f) {
              t = reinterpret_cast<const float4 *>(src)[0];
              t2 = reinterpret_cast<const float4 *>(src)[1];
            }
            v[k][0] = t.x; v[k][1] = t.y; v[k][2] = t.z; v[k][3] = t.w;
            v[k][4] = t2.x; v[k][5] = t2.y; v[k][6] = t2.z; v[k][7] = t2.w;
          } else if constexpr (VEC == 4) {
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            if (wi[k] != 0.f) t = *reinterpret_cast<const float4 *>(src);
            v[k][0] = t.x; v[k][1] = t.y; v[k][2] = t.z; v[k][3] = t.w;
          } else {
            float2 t = make_float2(0.f, 0.f);
            if (wi[k] != 0.f) t = *reinterpret_cast<const float2 *>(src);
            v[k][0] = t.x; v[k][1] = t.y;
          }
        }
#pragma unroll
        for (int k = 0; k < kBatch; ++k)
#pragma unroll
          for (int c = 0; c < VEC; ++c) acc[c] = fmaf(wi[k], v[k][c], acc[c]);
      }
    }
#pragma unroll
    for (int sh = 16; sh >= 1; sh >>= 1) s += __shfl_xor_sync(0xffffffffu, s, sh);
    const float inv = 1.f / s;
#pragma unroll
    for (int c = 0; c < VEC; ++c) acc[c] *= inv;
  }
  store_row<T, VEC>(o + (size_t)row * D + lane * VEC, acc);
  if (lane == 0) lse[row] = m > -INFINITY ? m + logf(s) : -INFINITY;
}

template <typename T, int D>
mc_status_t launch_t(const Params &p, const float *o_part, const float *lse_part, void *o, float *lse,
                     cudaStream_t stream, bool beside_previous) {
  const int rows = p.B * p.Hq;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((rows + kWarpsPerBlock - 1) / kWarpsPerBlock));
  cfg.blockDim = dim3(kWarpsPerBlock * 32);
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = beside_previous ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, merge_lse_kernel<T, D>, rows, (int)p.n_parts, o_part, lse_part,
                                           (T *)o, lse);
  count_launch();
  return e == cudaSuccess ? check_launch() : MC_ERR_CUDA;
}

}  // namespace

mc_status_t launch_merge(const Params &p, int dtype, const float *o_part, const float *lse_part, void *o,
                         float *lse, cudaStream_t stream, bool beside_previous) {
  if (dtype == MC_F32) {
    if (p.d == 64) return launch_t<float, 64>(p, o_part, lse_part, o, lse, stream, beside_previous);
    if (p.d == 128) return launch_t<float, 128>(p, o_part, lse_part, o, lse, stream, beside_previous);
    if (p.d == 256) return launch_t<float, 256>(p, o_part, lse_part, o, lse, stream, beside_previous);
  } else if (dtype == MC_BF16) {
    if (p.d == 64) return launch_t<__nv_bfloat16, 64>(p, o_part, lse_part, o, lse, stream, beside_previous);
    if (p.d == 128) return launch_t<__nv_bfloat16, 128>(p, o_part, lse_part, o, lse, stream, beside_previous);
    if (p.d == 256) return launch_t<__nv_bfloat16, 256>(p, o_part, lse_part, o, lse, stream, beside_previous);
  }
  return MC_ERR_UNSUPPORTED;
}

}  // namespace mc
