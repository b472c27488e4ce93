// Query/key/value projection of a decode step on the 5th-generation tensor cores: y = x W^T, bf16 operands, fp32 sums.
//
// With B = 64..256 candidates the product reads every weight once and uses it B times: it is bound by the stream
// of W from HBM (N x hidden x 2 bytes), not by the tensor pipe.  The shape of the kernel follows from that:
//   * one CTA = one head (128 output features: one 128-wide B operand tile, and the rotation that follows pairs
//     features inside a head) x one piece of the hidden dimension x up to 256 candidates (one or two 128-row A
//     tiles, accumulators of 128 TMEM columns each);
//   * the hidden dimension is split into `splits` pieces per head so that the grid has about as many CTAs as the
//     GPU has room for at once: all of them resident, each with two or three 64-wide k-blocks in flight, together
//     well over the bytes HBM needs in flight;
//   * a k-block is one TMA box of W (128 features x 64 hidden = 16 KB, streamed, evict-first) and one box of x per
//     row tile (re-read by every CTA from L2, evict-last), both with the 128-byte swizzle, consumed by four
//     tcgen05.mma (k = 16) per row tile;
//   * the epilogue stores the fp32 partial sums [split][row][feature]; the kernel that rotates and appends adds
//     the splits up in a fixed order (no atomics: the result does not depend on the order CTAs finish in).
// Warp roles: warp 0 lane 0 issues the copies, warp 1 lane 0 the products (warp 1 owns the TMEM allocation),
// warps 2-5 read the accumulators back (one thread per TMEM lane = per candidate row).  Every mbarrier wait is
// bounded: on expiry the CTA latches MC_ERR_TIMEOUT, stops issuing, waits (bounded) for its copies in flight, frees
// its TMEM and returns.
#include <cstdlib>
#include <new>

#include "mc_internal.cuh"
#include "mc_tcgen05.cuh"

namespace mc {
namespace {

constexpr int kHead = 128;                   // features per head = N tile
constexpr int kRows = 128;                   // candidate rows per A tile
constexpr int kKb = 64;                      // hidden elements per k-block (one 128-byte swizzle span of bf16)
constexpr uint32_t kBoxBytes = kRows * kKb * 2;   // 16 KB: one box of x or of W
constexpr int kThreadsQ = 192;
constexpr long long kDrainCyclesQ = 2000000ll;

template <int N_MT> struct QkvCfg {
  static constexpr int kStages = N_MT == 1 ? 3 : 2;                       // 96 KB either way: two CTAs per SM
  static constexpr uint32_t kStageBytes = (N_MT + 1) * kBoxBytes;         // x tiles, then the W tile
  static constexpr uint32_t kTmemCols = N_MT == 1 ? 128 : 256;
};

template <int N_MT> struct __align__(1024) SmemQ {
  uint8_t stage[QkvCfg<N_MT>::kStages][QkvCfg<N_MT>::kStageBytes];
  uint64_t full[QkvCfg<N_MT>::kStages], empty[QkvCfg<N_MT>::kStages], acc_full;
  uint32_t tmem_base;
  volatile int abort;
  long long wait_cycles;
};

template <int N_MT>
__device__ __forceinline__ bool mbar_wait_q(SmemQ<N_MT> &sm, int32_t *status, uint64_t *bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    __nanosleep(32);
    if (sm.abort) return false;
    if (clock64() - t0 > sm.wait_cycles) {
      sm.abort = 1;
      atomicCAS(status, 0, (int32_t)kDevTimeout);
      return false;
    }
  }
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%2, %3}], [%4], %5;\n"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}

// kind::f16 instruction descriptor: bf16 x bf16 -> f32, M = 128, N = 128, both operands K-major
constexpr uint32_t kIdescQ = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kHead >> 3) << 17) |
                             ((uint32_t)(kRows >> 4) << 24);

// grid.x = head * splits + piece, grid.y = pass over the candidates (N_MT * 128 rows each)
template <int N_MT>
__global__ void __launch_bounds__(kThreadsQ)
qkv_gemm_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap w_map,
                float *__restrict__ partial, int B, int N, int kb_total, int splits, int m_pad, int32_t *status,
                long long wait_cycles) {
  using C = QkvCfg<N_MT>;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  SmemQ<N_MT> &sm = *reinterpret_cast<SmemQ<N_MT> *>(smem_raw);
  if ((smem_u32(smem_raw) & 1023u) != 0) {   // the swizzled tiles need a 1024-byte aligned base
    if (threadIdx.x == 0) atomicCAS(status, 0, (int32_t)MC_ERR_CUDA);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int head = blockIdx.x / splits, piece = blockIdx.x % splits;
  const int m0 = blockIdx.y * (N_MT * kRows);
  const int kb_lo = (int)((long long)piece * kb_total / splits), kb_hi = (int)((long long)(piece + 1) * kb_total / splits);

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&sm.full[s], 1);
      mbar_init(&sm.empty[s], 1);
    }
    mbar_init(&sm.acc_full, 1);
    sm.abort = 0;
    sm.wait_cycles = wait_cycles;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&sm.tmem_base)),
                 "r"(C::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  // The kernel that adds the pieces up is launched behind this one as its programmatic dependent: its CTAs may take
  // their places early and wait there for this grid to complete.
  if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");

  if (warp == 0) {
    // ---------------------------------------------------------------- copies
    if (lane == 0) {
      uint64_t keep, stream;
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;\n" : "=l"(keep));
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(stream));
      for (int kb = kb_lo; kb < kb_hi; ++kb) {
        const uint32_t n = (uint32_t)(kb - kb_lo);
        const int s = n % C::kStages;
        if (!mbar_wait_q(sm, status, &sm.empty[s], ((n / C::kStages) & 1) ^ 1)) break;
        mbar_expect_tx(&sm.full[s], C::kStageBytes);
#pragma unroll
        for (int mt = 0; mt < N_MT; ++mt)   // rows past the last candidate lie outside the map and arrive as zeros
          tma_load_2d(sm.stage[s] + mt * kBoxBytes, &x_map, kb * kKb, m0 + mt * kRows, &sm.full[s], keep);
        tma_load_2d(sm.stage[s] + N_MT * kBoxBytes, &w_map, kb * kKb, head * kHead, &sm.full[s], stream);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- products
    if (lane == 0) {
      bool ok = true;
      for (int kb = kb_lo; kb < kb_hi; ++kb) {
        const uint32_t n = (uint32_t)(kb - kb_lo);
        const int s = n % C::kStages;
        if (!(ok = mbar_wait_q(sm, status, &sm.full[s], (n / C::kStages) & 1))) break;
        tc_fence_after();
        const uint64_t w_desc = smem_desc(smem_u32(sm.stage[s] + N_MT * kBoxBytes), 16, 1024);
#pragma unroll
        for (int mt = 0; mt < N_MT; ++mt) {
          const uint64_t x_desc = smem_desc(smem_u32(sm.stage[s] + mt * kBoxBytes), 16, 1024);
#pragma unroll
          for (int kk = 0; kk < kKb / 16; ++kk)   // 32 bytes further along the swizzle span per k-step
            umma_ss(tmem + (uint32_t)mt * kHead, x_desc + (uint64_t)(kk * 2), w_desc + (uint64_t)(kk * 2), kIdescQ,
                    (kb > kb_lo) || (kk > 0));
        }
        umma_commit(&sm.empty[s]);
      }
      if (ok) umma_commit(&sm.acc_full);   // arrives once every product issued so far has completed
    }
  } else {
    // ---------------------------------------------------------------- accumulators -> partial sums
    const int quad = warp & 3, r = quad * 32 + lane;
    bool ok = kb_hi > kb_lo ? mbar_wait_q(sm, status, &sm.acc_full, 0) : true;
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
#pragma unroll
      for (int mt = 0; mt < N_MT; ++mt) {
        const int row = m0 + mt * kRows + r;
        float *dst = partial + ((size_t)piece * m_pad + row) * N + (size_t)head * kHead;
#pragma unroll
        for (int c = 0; c < kHead / 32; ++c) {
          uint32_t v[32];
          if (kb_hi > kb_lo) {
            tmem_ld32(tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)(mt * kHead + c * 32), v);
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = 0u;   // a piece without k-blocks (more pieces than k-blocks) adds nothing
          }
          if (row < B) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
              reinterpret_cast<uint4 *>(dst + c * 32)[i] = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
          }
        }
      }
    }
  }

  // An aborting CTA grants its copies in flight a bounded time to land before its shared memory is given back.
  if (sm.abort && warp == 0 && lane == 0) {
    const long long t0 = clock64();
    while (clock64() - t0 < kDrainCyclesQ) { }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(C::kTmemCols) : "memory");
  }
}

typedef CUresult (*EncodeTiledFnQ)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Map over a row-major bf16 matrix [rows][cols]: one box = 64 columns of 128 rows, 128-byte swizzle; rows beyond
// the matrix read as zeros.
bool encode_matrix_map(CUtensorMap *map, const void *base, long long rows, long long cols) {
  static EncodeTiledFnQ fn = nullptr;
  if (!fn) {
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !sym)
      return false;
    fn = reinterpret_cast<EncodeTiledFnQ>(sym);
  }
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kKb, (cuuint32_t)kRows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int env_int_q(const char *name, int dflt) {
  const char *s = std::getenv(name);
  if (!s || !*s) return dflt;
  const int v = std::atoi(s);
  return v >= 0 ? v : dflt;
}

}  // namespace

struct QkvPlan {
  CUtensorMap w_map;
  int B, N, hidden, kb_total, heads, splits, n_mt, passes, m_pad;
  float *partial;
  size_t ws_bytes;
  long long wait_cycles;
};

QkvPlan *qkv_plan(int B, int heads, int hidden, const void *w, int sms) {
  if (B < 1 || heads < 1 || hidden < kKb || hidden % kKb != 0) return nullptr;
  QkvPlan *pl = new (std::nothrow) QkvPlan();
  if (!pl) return nullptr;
  pl->B = B;
  pl->heads = heads;
  pl->N = heads * kHead;
  pl->hidden = hidden;
  pl->kb_total = hidden / kKb;
  pl->n_mt = B > kRows ? 2 : 1;
  pl->passes = (B + pl->n_mt * kRows - 1) / (pl->n_mt * kRows);
  pl->m_pad = pl->passes * pl->n_mt * kRows;
  // Two CTAs fit an SM (96 KB of stages each; 2 x 256 TMEM columns at most).  As many pieces per head as keep the
  // whole grid resident at once, so that no CTA waits for a slot while HBM idles; at least 4 k-blocks a piece.
  const int slots = 2 * sms;
  int splits = slots / (heads * pl->passes);
  if (splits > pl->kb_total / 4) splits = pl->kb_total / 4;
  if (splits > 16) splits = 16;
  if (splits < 1) splits = 1;
  const int forced = env_int_q("MC_QKV_SPLITS", 0);
  if (forced > 0) splits = forced > 64 ? 64 : forced;
  pl->splits = splits;
  pl->wait_cycles = wait_limit_cycles();
  pl->ws_bytes = (size_t)splits * pl->m_pad * pl->N * sizeof(float);
  pl->partial = nullptr;
  if (!encode_matrix_map(&pl->w_map, w, pl->N, hidden) ||
      cudaFuncSetAttribute(qkv_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(SmemQ<1>)) != cudaSuccess ||
      cudaFuncSetAttribute(qkv_gemm_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(SmemQ<2>)) != cudaSuccess ||
      cudaMalloc(&pl->partial, pl->ws_bytes) != cudaSuccess) {
    (void)cudaGetLastError();
    delete pl;
    return nullptr;
  }
  return pl;
}

void qkv_plan_free(QkvPlan *pl) {
  if (!pl) return;
  cudaFree(pl->partial);
  delete pl;
}

int qkv_splits(const QkvPlan *pl) { return pl->splits; }
int qkv_ctas(const QkvPlan *pl) { return pl->heads * pl->splits * pl->passes; }
int qkv_row_stride(const QkvPlan *pl) { return pl->m_pad; }
size_t qkv_workspace_bytes(const QkvPlan *pl) { return pl->ws_bytes; }
const float *qkv_partials(const QkvPlan *pl) { return pl->partial; }

mc_status_t launch_qkv_gemm(const QkvPlan *pl, const void *x, int32_t *status, cudaStream_t stream) {
  CUtensorMap x_map;
  if (!encode_matrix_map(&x_map, x, pl->B, pl->hidden)) return MC_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(pl->heads * pl->splits), (unsigned)pl->passes);
  cfg.blockDim = dim3(kThreadsQ);
  cfg.stream = stream;
  cudaError_t e;
  if (pl->n_mt == 1) {
    cfg.dynamicSmemBytes = sizeof(SmemQ<1>);
    e = cudaLaunchKernelEx(&cfg, qkv_gemm_kernel<1>, x_map, pl->w_map, pl->partial, pl->B, pl->N, pl->kb_total,
                           pl->splits, pl->m_pad, status, pl->wait_cycles);
  } else {
    cfg.dynamicSmemBytes = sizeof(SmemQ<2>);
    e = cudaLaunchKernelEx(&cfg, qkv_gemm_kernel<2>, x_map, pl->w_map, pl->partial, pl->B, pl->N, pl->kb_total,
                           pl->splits, pl->m_pad, status, pl->wait_cycles);
  }
  count_launch();
  return e == cudaSuccess ? check_launch() : MC_ERR_CUDA;
}

}  // namespace mc
