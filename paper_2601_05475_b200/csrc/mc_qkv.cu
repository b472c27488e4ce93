// Query/key/value projection of a decode step on the 5th-generation tensor cores: y = x W^T, bf16 operands, fp32 sums.
//
// With B = 64..256 candidates the product reads every weight once and uses it B times: it is bound by the stream
// of W from HBM (N x hidden x 2 bytes), not by the tensor pipe.  The shape of the kernel follows from that:
//   * the work is the sequence of all k-blocks (64 hidden elements) of all head pairs (256 output features: one
//     256-wide B operand tile; the rotation that follows pairs features inside a head), and every CTA of a
//     persistent grid (one per SM) takes an equal, contiguous share of that sequence - so every SM pulls on HBM
//     from the first to the last microsecond, whatever the number of heads;
//   * a k-block is one TMA box of W (256 features x 64 hidden = 32 KB, streamed, evict-first) and one box of x per
//     128-row tile (re-read by every CTA from L2, evict-last), both with the 128-byte swizzle, consumed by four
//     tcgen05.mma (M = 128, N = 256, k = 16) per row tile; four stages (three with two row tiles) keep 96-128 KB
//     of W in flight per SM;
//   * what bounds it is the bytes an SM can have on their way: a copy issued while HBM runs near its rate arrives
//     about 3 us later (x, from L2, about half that), shared memory holds four k-blocks of 48 KB, and four k-blocks
//     per 3 us per SM is the 5 TB/s the kernel reaches - level with the library GEMM of the same shape.  Tried and
//     measured, none faster: W re-tiled into contiguous 32 KB boxes (the same: DRAM locality is not the limit),
//     the x copies left out (the same: the SM's intake is not the limit), separate rings of five W boxes and two x
//     slots (slower: two slots do not cover x's latency).  What would help is a smaller share of x per byte of W
//     in shared memory: x shared between SMs (cluster multicast or CTA pairs) or between two W tiles;
//   * where a CTA's share crosses from one head pair to the next, it stores the fp32 sums of the piece it has
//     ([piece][row][feature]; piece = the CTA's ordinal among the CTAs that share the pair) and starts over; the
//     kernel that rotates and appends adds the pieces of a pair up in that fixed order (no atomics: the result does
//     not depend on the order CTAs finish in).
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

constexpr int kPairN = 256;                  // features per B operand tile: two heads
constexpr int kRows = 128;                   // candidate rows per A tile
constexpr int kKb = 64;                      // hidden elements per k-block (one 128-byte swizzle span of bf16)
constexpr uint32_t kXBoxBytes = kRows * kKb * 2;    // 16 KB
constexpr uint32_t kWBoxBytes = kPairN * kKb * 2;   // 32 KB
constexpr int kThreadsQ = 192;
constexpr long long kDrainCyclesQ = 2000000ll;

template <int N_MT> struct QkvCfg {
  static constexpr int kStages = N_MT == 1 ? 4 : 3;                          // 192 KB either way: one CTA per SM
  static constexpr uint32_t kStageBytes = N_MT * kXBoxBytes + kWBoxBytes;     // x tiles, then the W tile
  static constexpr int kAccBufs = N_MT == 1 ? 2 : 1;    // accumulator sets: with one row tile the next piece's
                                                        // products run while the epilogue reads this one's sums
  static constexpr uint32_t kTmemCols = 512;
};
constexpr int kTrRow = 36;   // floats per row of the epilogue's transposing buffer (32 + 4: 16-byte rows, no bank conflicts)

template <int N_MT> struct __align__(1024) SmemQ {
  uint8_t stage[QkvCfg<N_MT>::kStages][QkvCfg<N_MT>::kStageBytes];
  float tr[4][32 * kTrRow];     // per epilogue warp: 32 rows x 32 columns on their way from TMEM to coalesced stores
  uint64_t full[QkvCfg<N_MT>::kStages], empty[QkvCfg<N_MT>::kStages];
  uint64_t acc_full[QkvCfg<N_MT>::kAccBufs], acc_empty[QkvCfg<N_MT>::kAccBufs];
  uint32_t tmem_base;
  volatile int abort;
  long long wait_cycles;
};

// (mbarrier.try_wait may suspend the thread for a while before it answers; test_wait answers at once)
__device__ __forceinline__ bool mbar_test_wait_q(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false (and raises the CTA's abort flag) when the limit expires or another role has
// already aborted.  Limits under a millisecond are polled without suspending, so that they mean what they say.
template <int N_MT>
__device__ __forceinline__ bool mbar_wait_q(SmemQ<N_MT> &sm, int32_t *status, uint64_t *bar, uint32_t parity) {
  const bool polled = sm.wait_cycles < 2000000ll;
  if (polled ? mbar_test_wait_q(bar, parity) : mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (polled ? mbar_test_wait_q(bar, parity) : mbar_try_wait(bar, parity)) return true;
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

// kind::f16 instruction descriptor: bf16 x bf16 -> f32, M = 128, N = 256, both operands K-major
constexpr uint32_t kIdescQ = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kPairN >> 3) << 17) |
                             ((uint32_t)(kRows >> 4) << 24);

// grid.x = persistent CTAs, grid.y = pass over the candidates (N_MT * 128 rows each).  The k-blocks of all head
// pairs are numbered pair * kb_per_pair + kb; CTA c takes [c T / n, (c + 1) T / n).
template <int N_MT>
__global__ void __launch_bounds__(kThreadsQ)
qkv_gemm_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap w_map,
                float *__restrict__ partial, int B, int n_pad, int kb_per_pair, int n_pairs, int m_pad, int32_t *status,
                long long wait_cycles) {
  using C = QkvCfg<N_MT>;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  SmemQ<N_MT> &sm = *reinterpret_cast<SmemQ<N_MT> *>(smem_raw);
  if ((smem_u32(smem_raw) & 1023u) != 0) {   // the swizzled tiles need a 1024-byte aligned base
    if (threadIdx.x == 0) atomicCAS(status, 0, (int32_t)MC_ERR_CUDA);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.y * (N_MT * kRows);
  const long long total = (long long)n_pairs * kb_per_pair;
  const int u_lo = (int)(blockIdx.x * total / gridDim.x), u_hi = (int)((blockIdx.x + 1) * total / gridDim.x);

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&sm.full[s], 1);
      mbar_init(&sm.empty[s], 1);
    }
    for (int a = 0; a < C::kAccBufs; ++a) {
      mbar_init(&sm.acc_full[a], 1);
      mbar_init(&sm.acc_empty[a], kThreadsQ - 64);
    }
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
  // their places early and wait there for this grid to complete.  It also needs what the kernel in front of this
  // one wrote (where the tokens go), which this kernel does not: a thread of the epilogue, idle until the first
  // piece is done, waits for that grid before it gives the word.  Launched the ordinary way the wait returns at once.
  if (threadIdx.x == kThreadsQ - 1) {
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  }

  if (warp == 0) {
    // ---------------------------------------------------------------- copies
    if (lane == 0) {
      uint64_t keep, stream;
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;\n" : "=l"(keep));
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(stream));
      for (int u = u_lo; u < u_hi; ++u) {
        const uint32_t n = (uint32_t)(u - u_lo);
        const int s = n % C::kStages;
        const int pair = u / kb_per_pair, kb = u - pair * kb_per_pair;
        if (!mbar_wait_q(sm, status, &sm.empty[s], ((n / C::kStages) & 1) ^ 1)) break;
        mbar_expect_tx(&sm.full[s], C::kStageBytes);
        // (rows past the last candidate or past the last feature lie outside the maps and arrive as zeros)
        tma_load_2d(sm.stage[s] + N_MT * kXBoxBytes, &w_map, kb * kKb, pair * kPairN, &sm.full[s], stream);
#pragma unroll
        for (int mt = 0; mt < N_MT; ++mt)
          tma_load_2d(sm.stage[s] + mt * kXBoxBytes, &x_map, kb * kKb, m0 + mt * kRows, &sm.full[s], keep);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- products
    if (lane == 0) {
      uint32_t seg = 0;   // pieces this CTA has started
      for (int u = u_lo; u < u_hi; ++u) {
        const uint32_t n = (uint32_t)(u - u_lo);
        const int s = n % C::kStages;
        const int kb = u % kb_per_pair;
        const bool first = u == u_lo || kb == 0, last = u == u_hi - 1 || kb == kb_per_pair - 1;
        const uint32_t buf = seg % C::kAccBufs, use = seg / C::kAccBufs;   // accumulator set and its use count
        if (first && use > 0) {   // the set still holds an earlier piece until the epilogue has read it
          if (!mbar_wait_q(sm, status, &sm.acc_empty[buf], (use - 1) & 1)) break;
          tc_fence_after();
        }
        if (!mbar_wait_q(sm, status, &sm.full[s], (n / C::kStages) & 1)) break;
        tc_fence_after();
        const uint32_t acc = tmem + buf * (uint32_t)(N_MT * kPairN);
        const uint64_t w_desc = smem_desc(smem_u32(sm.stage[s] + N_MT * kXBoxBytes), 16, 1024);
#pragma unroll
        for (int mt = 0; mt < N_MT; ++mt) {
          const uint64_t x_desc = smem_desc(smem_u32(sm.stage[s] + mt * kXBoxBytes), 16, 1024);
#pragma unroll
          for (int kk = 0; kk < kKb / 16; ++kk)   // 32 bytes further along the swizzle span per k-step
            umma_ss(acc + (uint32_t)mt * kPairN, x_desc + (uint64_t)(kk * 2), w_desc + (uint64_t)(kk * 2), kIdescQ,
                    !first || (kk > 0));
        }
        umma_commit(&sm.empty[s]);
        if (last) {
          umma_commit(&sm.acc_full[buf]);   // arrives once every product issued so far has completed
          ++seg;
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- accumulators -> partial sums
    // A thread reads its row of the accumulator (TMEM lane = candidate row); stored like that, a warp's store
    // would touch 32 rows 16 bytes at a time.  Each 32 x 32 block therefore goes through the warp's transposing
    // buffer and leaves as 8 stores of 4 rows x 128 contiguous bytes.
    const int quad = warp & 3;
    float *tr = sm.tr[quad];
    uint32_t seg = 0;
    for (int u = u_lo; u < u_hi; ++seg) {
      const int pair = u / kb_per_pair;
      const int u_end = min(u_hi, (pair + 1) * kb_per_pair);   // the piece is [u, u_end)
      // this CTA's ordinal among the CTAs that share the pair: the first of them holds k-block pair * kb_per_pair
      const int first_cta = (int)((((long long)pair * kb_per_pair + 1) * gridDim.x - 1) / total);
      const int piece = (int)blockIdx.x - first_cta;
      const uint32_t buf = seg % C::kAccBufs, use = seg / C::kAccBufs;
      bool ok = mbar_wait_q(sm, status, &sm.acc_full[buf], use & 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t acc = tmem + buf * (uint32_t)(N_MT * kPairN) + ((uint32_t)(quad * 32) << 16);
#pragma unroll 1
      for (int mt = 0; mt < N_MT; ++mt) {
        const int row0 = m0 + mt * kRows + quad * 32;   // first of this warp's 32 rows
        float *dst = partial + ((size_t)piece * m_pad + row0) * n_pad + (size_t)pair * kPairN;
#pragma unroll 1
        for (int c = 0; c < kPairN / 32; ++c) {
          uint32_t v[32];
          tmem_ld32(acc + (uint32_t)(mt * kPairN + c * 32), v);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 8; ++i)
            *reinterpret_cast<uint4 *>(tr + lane * kTrRow + 4 * i) = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 8; ++j) {   // rows 4 j .. 4 j + 3, eight lanes (128 bytes) each
            const int rr = 4 * j + (lane >> 3);
            const uint4 t = *reinterpret_cast<const uint4 *>(tr + rr * kTrRow + 4 * (lane & 7));
            if (row0 + rr < B) *reinterpret_cast<uint4 *>(dst + (size_t)rr * n_pad + c * 32 + 4 * (lane & 7)) = t;
          }
          __syncwarp();
        }
      }
      tc_fence_before();
      mbar_arrive(&sm.acc_empty[buf]);   // the accumulators may be overwritten
      u = u_end;
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

static_assert(sizeof(SmemQ<1>) <= 232448 && sizeof(SmemQ<2>) <= 232448, "shared memory of one CTA");

typedef CUresult (*EncodeTiledFnQ)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Map over a row-major bf16 matrix [rows][cols]: one box = 64 columns of `box_rows` rows, 128-byte swizzle; rows
// beyond the matrix read as zeros.
bool encode_matrix_map(CUtensorMap *map, const void *base, long long rows, long long cols, int box_rows) {
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
  const cuuint32_t box[2] = {(cuuint32_t)kKb, (cuuint32_t)box_rows};
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
  int B, N, hidden, kb_per_pair, n_pairs, n_pad, n_mt, passes, m_pad, ctas, pieces;
  float *partial;
  size_t ws_bytes;
  long long wait_cycles;
};

// The CTA whose share [c T / n, (c + 1) T / n) holds k-block u.
static int qkv_cta_of(long long u, int n, long long total) { return (int)(((u + 1) * n - 1) / total); }

QkvPlan *qkv_plan(int B, int heads, int hidden, const void *w, int sms) {
  if (B < 1 || heads < 1 || hidden < kKb || hidden % kKb != 0) return nullptr;
  QkvPlan *pl = new (std::nothrow) QkvPlan();
  if (!pl) return nullptr;
  pl->B = B;
  pl->N = heads * 128;
  pl->hidden = hidden;
  pl->kb_per_pair = hidden / kKb;
  pl->n_pairs = (heads + 1) / 2;
  pl->n_pad = pl->n_pairs * kPairN;
  pl->n_mt = B > kRows ? 2 : 1;
  pl->passes = (B + pl->n_mt * kRows - 1) / (pl->n_mt * kRows);
  pl->m_pad = pl->passes * pl->n_mt * kRows;
  const long long total = (long long)pl->n_pairs * pl->kb_per_pair;
  int ctas = env_int_q("MC_QKV_CTAS", 0);
  if (ctas <= 0) ctas = sms;
  if (ctas > total) ctas = (int)total;   // at least one k-block each
  pl->ctas = ctas;
  pl->pieces = 1;
  for (int pr = 0; pr < pl->n_pairs; ++pr) {
    const int n = qkv_cta_of((long long)(pr + 1) * pl->kb_per_pair - 1, ctas, total) -
                  qkv_cta_of((long long)pr * pl->kb_per_pair, ctas, total) + 1;
    if (n > pl->pieces) pl->pieces = n;
  }
  pl->wait_cycles = wait_limit_cycles();
  pl->ws_bytes = (size_t)pl->pieces * pl->m_pad * pl->n_pad * sizeof(float);
  pl->partial = nullptr;
  if (!encode_matrix_map(&pl->w_map, w, pl->N, hidden, kPairN) ||
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

int qkv_pieces(const QkvPlan *pl) { return pl->pieces; }
int qkv_ctas(const QkvPlan *pl) { return pl->ctas; }
int qkv_passes(const QkvPlan *pl) { return pl->passes; }
int qkv_kb_per_pair(const QkvPlan *pl) { return pl->kb_per_pair; }
int qkv_row_stride(const QkvPlan *pl) { return pl->m_pad; }
int qkv_feature_stride(const QkvPlan *pl) { return pl->n_pad; }
size_t qkv_workspace_bytes(const QkvPlan *pl) { return pl->ws_bytes; }
const float *qkv_partials(const QkvPlan *pl) { return pl->partial; }

mc_status_t launch_qkv_gemm(const QkvPlan *pl, const void *x, int32_t *status, cudaStream_t stream,
                            bool beside_previous) {
  CUtensorMap x_map;
  if (!encode_matrix_map(&x_map, x, pl->B, pl->hidden, kRows)) return MC_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)pl->ctas, (unsigned)pl->passes);
  cfg.blockDim = dim3(kThreadsQ);
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = beside_previous ? 1 : 0;
  cudaError_t e;
  if (pl->n_mt == 1) {
    cfg.dynamicSmemBytes = sizeof(SmemQ<1>);
    e = cudaLaunchKernelEx(&cfg, qkv_gemm_kernel<1>, x_map, pl->w_map, pl->partial, pl->B, pl->n_pad, pl->kb_per_pair,
                           pl->n_pairs, pl->m_pad, status, pl->wait_cycles);
  } else {
    cfg.dynamicSmemBytes = sizeof(SmemQ<2>);
    e = cudaLaunchKernelEx(&cfg, qkv_gemm_kernel<2>, x_map, pl->w_map, pl->partial, pl->B, pl->n_pad, pl->kb_per_pair,
                           pl->n_pairs, pl->m_pad, status, pl->wait_cycles);
  }
  count_launch();
  return e == cudaSuccess ? check_launch() : MC_ERR_CUDA;
}

}  // namespace mc
