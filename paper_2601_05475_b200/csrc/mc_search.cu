// Batched max-reward search bookkeeping: categorical rewards, best-so-far, value targets, labels, trajectory
// returns, the value head's softmax and mean, and the per-group argmax.  All of it is a few flops per element:
// the kernels are bound by HBM, so every array is touched once, with consecutive threads on consecutive
// trajectories of the step-major arrays.
#include <cuda_runtime.h>
#include <stdint.h>

#include "maxcode_search.h"
#include "mc_internal.cuh"

namespace mc {
namespace {

__device__ __forceinline__ int reward_class(float speedup_pct, bool correct, float s1, float s2, float s3) {
  if (!correct || !(speedup_pct > 100.f)) return 0;
  return speedup_pct <= s1 ? 1 : speedup_pct <= s2 ? 2 : speedup_pct <= s3 ? 3 : 4;
}

// One thread per trajectory.  TMAX > 0: the whole trajectory (T <= TMAX steps) is held in registers between the
// forward sweep (u_t, G) and the backward sweep (future maxima), so inputs are read once.  TMAX = 0: any T, the
// backward sweep reads the inputs a second time.
template <int TMAX>
__global__ void __launch_bounds__(256)
search_returns_kernel(const float *__restrict__ speedup, const uint8_t *__restrict__ correct,
                      const int32_t *__restrict__ len, int N, int T, float s1, float s2, float s3, float gamma,
                      uint8_t *__restrict__ reward, float *__restrict__ best_so_far, float *__restrict__ value_target,
                      uint8_t *__restrict__ label, float *__restrict__ traj_return) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= N) return;
  int L = len ? __ldg(len + n) : T;
  L = L < 0 ? 0 : L > T ? T : L;
  const float inv_gamma = 1.f / gamma;
  if (TMAX > 0) {
    float raw[TMAX > 0 ? TMAX : 1], u[TMAX > 0 ? TMAX : 1];
    int r[TMAX > 0 ? TMAX : 1];
    float best = 0.f, pw = 1.f;   // rewards are >= 0, so 0 is the identity of the running maximum
#pragma unroll
    for (int t = 0; t < TMAX; ++t) {
      raw[t] = 0.f; r[t] = 0; u[t] = 0.f;
      if (t < L) {
        const size_t i = (size_t)t * N + n;
        const float s = __ldg(speedup + i);
        const bool ok = __ldg(correct + i) != 0;
        r[t] = reward_class(s, ok, s1, s2, s3);
        raw[t] = ok ? s : 0.f;
        best = fmaxf(best, pw * (float)r[t]);
        u[t] = best;
        pw *= gamma;
      }
    }
    if (traj_return) traj_return[n] = best;
    float m = 0.f, mraw = 0.f;
#pragma unroll
    for (int t = TMAX - 1; t >= 0; --t) {
      if (t >= T) continue;
      const size_t i = (size_t)t * N + n;
      const bool live = t < L;
      if (live) {
        m = t == L - 1 ? (float)r[t] : fmaxf((float)r[t], gamma * m);
        mraw = t == L - 1 ? raw[t] : fmaxf(raw[t], gamma * mraw);
      }
      if (reward) reward[i] = (uint8_t)(live ? r[t] : 0);
      if (best_so_far) best_so_far[i] = live ? u[t] : 0.f;
      if (value_target) value_target[i] = live ? fmaxf(u[t] * inv_gamma, m) : 0.f;
      if (label) label[i] = (uint8_t)(live ? reward_class(mraw, true, s1, s2, s3) : 0);
    }
  } else {
    float best = 0.f, pw = 1.f;
    for (int t = 0; t < L; ++t) {
      const size_t i = (size_t)t * N + n;
      const int r = reward_class(__ldg(speedup + i), __ldg(correct + i) != 0, s1, s2, s3);
      best = fmaxf(best, pw * (float)r);
      pw *= gamma;
      if (best_so_far) best_so_far[i] = best;
    }
    if (traj_return) traj_return[n] = best;
    // backward sweep: u_t comes from the array the forward sweep wrote, or, if the caller did not ask for that
    // array, from repeating the forward sweep up to t
    float m = 0.f, mraw = 0.f;
    for (int t = T - 1; t >= 0; --t) {
      const size_t i = (size_t)t * N + n;
      const bool live = t < L;
      int r = 0;
      float u = 0.f;
      if (live) {
        const float s = __ldg(speedup + i);
        const bool ok = __ldg(correct + i) != 0;
        r = reward_class(s, ok, s1, s2, s3);
        const float raw = ok ? s : 0.f;
        m = t == L - 1 ? (float)r : fmaxf((float)r, gamma * m);
        mraw = t == L - 1 ? raw : fmaxf(raw, gamma * mraw);
        if (value_target) {
          if (best_so_far) {
            u = best_so_far[i];   // written by this thread above
          } else {
            float b = 0.f, q = 1.f;
            for (int k = 0; k <= t; ++k) {
              const size_t j = (size_t)k * N + n;
              b = fmaxf(b, q * (float)reward_class(__ldg(speedup + j), __ldg(correct + j) != 0, s1, s2, s3));
              q *= gamma;
            }
            u = b;
          }
        }
      }
      if (reward) reward[i] = (uint8_t)r;
      if (!live && best_so_far) best_so_far[i] = 0.f;
      if (value_target) value_target[i] = live ? fmaxf(u * inv_gamma, m) : 0.f;
      if (label) label[i] = (uint8_t)(live ? reward_class(mraw, true, s1, s2, s3) : 0);
    }
  }
}

// The same for T <= 8 (the depth of the paper's searches) with four neighbouring trajectories per thread: every
// access is a 16-byte vector (4 bytes for the uint8 arrays), a quarter of the instructions of the kernel above.
// N must be a multiple of 4 and every array 16-byte aligned.
__global__ void __launch_bounds__(128)
search_returns_x4_kernel(const float4 *__restrict__ speedup, const uchar4 *__restrict__ correct,
                         const int4 *__restrict__ len, int N4, int T, float s1, float s2, float s3, float gamma,
                         uchar4 *__restrict__ reward, float4 *__restrict__ best_so_far, float4 *__restrict__ value_target,
                         uchar4 *__restrict__ label, float4 *__restrict__ traj_return) {
  constexpr int TMAX = 8;
  const int n4 = blockIdx.x * blockDim.x + threadIdx.x;
  if (n4 >= N4) return;
  int L[4] = {T, T, T, T};
  if (len) {
    const int4 l = __ldg(len + n4);
    L[0] = l.x; L[1] = l.y; L[2] = l.z; L[3] = l.w;
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) L[j] = L[j] < 0 ? 0 : L[j] > T ? T : L[j];
  const float inv_gamma = 1.f / gamma;
  float raw[TMAX][4], u[TMAX][4];
  unsigned char r[TMAX][4];
  float best[4] = {0.f, 0.f, 0.f, 0.f}, pw = 1.f;
#pragma unroll
  for (int t = 0; t < TMAX; ++t) {
    float s[4] = {0.f, 0.f, 0.f, 0.f};
    unsigned char c[4] = {0, 0, 0, 0};
    if (t < T) {
      const float4 sv = __ldg(speedup + (size_t)t * N4 + n4);
      const uchar4 cv = __ldg(correct + (size_t)t * N4 + n4);
      s[0] = sv.x; s[1] = sv.y; s[2] = sv.z; s[3] = sv.w;
      c[0] = cv.x; c[1] = cv.y; c[2] = cv.z; c[3] = cv.w;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      // a step past the trajectory's end counts as reward 0, which changes no maximum (rewards are >= 0)
      const bool ok = t < L[j] && c[j] != 0;
      const int rc = reward_class(s[j], ok, s1, s2, s3);
      r[t][j] = (unsigned char)rc;
      raw[t][j] = ok ? s[j] : 0.f;
      best[j] = fmaxf(best[j], pw * (float)rc);
      u[t][j] = best[j];
    }
    pw *= gamma;
  }
  if (traj_return) traj_return[n4] = make_float4(best[0], best[1], best[2], best[3]);
  float m[4] = {0.f, 0.f, 0.f, 0.f}, mraw[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int t = TMAX - 1; t >= 0; --t) {
    if (t >= T) continue;
    float v[4];
    unsigned char lab[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const bool live = t < L[j];
      m[j] = fmaxf((float)r[t][j], gamma * m[j]);
      mraw[j] = fmaxf(raw[t][j], gamma * mraw[j]);
      v[j] = live ? fmaxf(u[t][j] * inv_gamma, m[j]) : 0.f;
      lab[j] = (unsigned char)reward_class(mraw[j], true, s1, s2, s3);   // 0 past the end: mraw is still 0 there
      if (!live) u[t][j] = 0.f;
    }
    const size_t i = (size_t)t * N4 + n4;
    if (reward) reward[i] = make_uchar4(r[t][0], r[t][1], r[t][2], r[t][3]);
    if (best_so_far) best_so_far[i] = make_float4(u[t][0], u[t][1], u[t][2], u[t][3]);
    if (value_target) value_target[i] = make_float4(v[0], v[1], v[2], v[3]);
    if (label) label[i] = make_uchar4(lab[0], lab[1], lab[2], lab[3]);
  }
}

__global__ void __launch_bounds__(256)
value_head_kernel(const float *__restrict__ logits, int N, float *__restrict__ prob, float *__restrict__ expected) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= N) return;
  float z[5];
#pragma unroll
  for (int q = 0; q < 5; ++q) z[q] = __ldg(logits + (size_t)n * 5 + q);
  const float mx = fmaxf(fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3])), z[4]);
  float sum = 0.f;
#pragma unroll
  for (int q = 0; q < 5; ++q) {
    z[q] = expf(z[q] - mx);
    sum += z[q];
  }
  const float inv = 1.f / sum;
  float e = 0.f;
#pragma unroll
  for (int q = 0; q < 5; ++q) {
    const float pq = z[q] * inv;
    if (prob) prob[(size_t)n * 5 + q] = pq;
    e = fmaf((float)q, pq, e);
  }
  expected[n] = e;
}

// Eight lanes per group (the paper samples k = 8 candidates per state; larger groups are walked in steps of eight);
// (value, index) pairs ordered by larger value, then smaller index.
constexpr int kLanesPerGroup = 8;
__global__ void __launch_bounds__(256)
group_argmax_kernel(const float *__restrict__ values, const int32_t *__restrict__ group_offsets, int P,
                    int32_t *__restrict__ best) {
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long j = tid / kLanesPerGroup;
  const int sub = (int)(tid % kLanesPerGroup);
  const bool active = j < P;   // whole warps stay in the shuffles below
  const int lo = active ? __ldg(group_offsets + j) : 0, hi = active ? __ldg(group_offsets + j + 1) : 0;
  float bv = -INFINITY;
  int bi = -1;
  for (int i = lo + sub; i < hi; i += kLanesPerGroup) {
    const float v = __ldg(values + i);
    if (bi < 0 ? v == v : v > bv) {   // the first non-NaN entry, then strictly larger ones (indices rise)
      bv = v;
      bi = i;
    }
  }
#pragma unroll
  for (int sh = kLanesPerGroup / 2; sh >= 1; sh >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, sh);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, sh);
    if (oi >= 0 && (bi < 0 || ov > bv || (ov == bv && oi < bi))) {
      bv = ov;
      bi = oi;
    }
  }
  if (active && sub == 0) best[j] = bi;
}

// Value head and both selections of a group in one pass: eight lanes per group; every lane forms the value head of
// its entries (softmax over the five class logits, its mean), keeps the best mean and the best return it has seen,
// and the eight lanes reduce both (value, index) pairs.  Nothing is read twice and nothing needs a second launch.
__device__ __forceinline__ void take_better(float &bv, int &bi, float v, int i) {
  if (i >= 0 && (bi < 0 ? v == v : (v > bv || (v == bv && i < bi)))) {
    bv = v;
    bi = i;
  }
}

__global__ void __launch_bounds__(256)
select_kernel(const float *__restrict__ logits, const float *__restrict__ traj_return,
              const int32_t *__restrict__ group_offsets, int P, float *__restrict__ prob, float *__restrict__ expected,
              int32_t *__restrict__ best_return, int32_t *__restrict__ best_expected) {
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long j = tid / kLanesPerGroup;
  const int sub = (int)(tid % kLanesPerGroup);
  const bool active = j < P;   // whole warps stay in the shuffles below
  const int lo = active ? __ldg(group_offsets + j) : 0, hi = active ? __ldg(group_offsets + j + 1) : 0;
  float ev = -INFINITY, gv = -INFINITY;
  int ei = -1, gi = -1;
  for (int i = lo + sub; i < hi; i += kLanesPerGroup) {
    float z[5];
#pragma unroll
    for (int q = 0; q < 5; ++q) z[q] = __ldg(logits + (size_t)i * 5 + q);
    const float mx = fmaxf(fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3])), z[4]);
    float sum = 0.f;
#pragma unroll
    for (int q = 0; q < 5; ++q) {
      z[q] = expf(z[q] - mx);
      sum += z[q];
    }
    const float inv = 1.f / sum;
    float e = 0.f;
#pragma unroll
    for (int q = 0; q < 5; ++q) {
      const float pq = z[q] * inv;
      if (prob) prob[(size_t)i * 5 + q] = pq;
      e = fmaf((float)q, pq, e);
    }
    if (expected) expected[i] = e;
    if (e == e) take_better(ev, ei, e, i);                        // (indices rise: an equal value never replaces)
    if (traj_return) {
      const float g = __ldg(traj_return + i);
      if (g == g) take_better(gv, gi, g, i);
    }
  }
#pragma unroll
  for (int sh = kLanesPerGroup / 2; sh >= 1; sh >>= 1) {
    const float oev = __shfl_xor_sync(0xffffffffu, ev, sh), ogv = __shfl_xor_sync(0xffffffffu, gv, sh);
    const int oei = __shfl_xor_sync(0xffffffffu, ei, sh), ogi = __shfl_xor_sync(0xffffffffu, gi, sh);
    take_better(ev, ei, oev, oei);
    take_better(gv, gi, ogv, ogi);
  }
  if (active && sub == 0) {
    if (best_expected) best_expected[j] = ei;
    if (best_return) best_return[j] = gi;
  }
}

}  // namespace
}  // namespace mc

extern "C" {

mc_status_t mc_search_returns(const float *speedup_pct, const uint8_t *correct, const int32_t *len, int32_t N, int32_t T,
                              float s1, float s2, float s3, float gamma, uint8_t *reward, float *best_so_far,
                              float *value_target, uint8_t *label, float *traj_return, void *stream) {
  if (!speedup_pct || !correct || N < 1 || T < 1) return MC_ERR_INVALID_ARG;
  if (!(100.f < s1 && s1 < s2 && s2 < s3) || !(gamma > 0.f && gamma <= 1.f)) return MC_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const unsigned grid = (unsigned)((N + 255) / 256);
#define MC_SEARCH_LAUNCH(TM)                                                                                        \
  mc::search_returns_kernel<TM><<<grid, 256, 0, st>>>(speedup_pct, correct, len, N, T, s1, s2, s3, gamma, reward, \
                                                      best_so_far, value_target, label, traj_return)
  const uintptr_t align = reinterpret_cast<uintptr_t>(speedup_pct) | reinterpret_cast<uintptr_t>(correct) |
                          reinterpret_cast<uintptr_t>(len) | reinterpret_cast<uintptr_t>(reward) |
                          reinterpret_cast<uintptr_t>(best_so_far) | reinterpret_cast<uintptr_t>(value_target) |
                          reinterpret_cast<uintptr_t>(label) | reinterpret_cast<uintptr_t>(traj_return);
  if (T <= 8 && N % 4 == 0 && (align & 15u) == 0)
    mc::search_returns_x4_kernel<<<(unsigned)((N / 4 + 127) / 128), 128, 0, st>>>(
        reinterpret_cast<const float4 *>(speedup_pct), reinterpret_cast<const uchar4 *>(correct),
        reinterpret_cast<const int4 *>(len), N / 4, T, s1, s2, s3, gamma, reinterpret_cast<uchar4 *>(reward),
        reinterpret_cast<float4 *>(best_so_far), reinterpret_cast<float4 *>(value_target),
        reinterpret_cast<uchar4 *>(label), reinterpret_cast<float4 *>(traj_return));
  else if (T <= 8) MC_SEARCH_LAUNCH(8);
  else if (T <= 16) MC_SEARCH_LAUNCH(16);
  else if (T <= 32) MC_SEARCH_LAUNCH(32);
  else MC_SEARCH_LAUNCH(0);
#undef MC_SEARCH_LAUNCH
  mc::count_launch();
  return mc::check_launch();
}

mc_status_t mc_search_value_head(const float *logits, int32_t N, float *prob, float *expected, void *stream) {
  if (!logits || !expected || N < 1) return MC_ERR_INVALID_ARG;
  mc::value_head_kernel<<<(unsigned)((N + 255) / 256), 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(logits, N, prob,
                                                                                                        expected);
  mc::count_launch();
  return mc::check_launch();
}

mc_status_t mc_search_group_argmax(const float *values, const int32_t *group_offsets, int32_t P, int32_t *best,
                                   void *stream) {
  if (!values || !group_offsets || !best || P < 1) return MC_ERR_INVALID_ARG;
  const long long threads = (long long)P * mc::kLanesPerGroup;
  mc::group_argmax_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      values, group_offsets, P, best);
  mc::count_launch();
  return mc::check_launch();
}

mc_status_t mc_search_select(const float *logits, const float *traj_return, const int32_t *group_offsets, int32_t P,
                             float *prob, float *expected, int32_t *best_return, int32_t *best_expected, void *stream) {
  if (!logits || !group_offsets || P < 1 || (!best_expected && !best_return && !expected && !prob))
    return MC_ERR_INVALID_ARG;
  if ((best_return != nullptr) != (traj_return != nullptr)) return MC_ERR_INVALID_ARG;
  const long long threads = (long long)P * mc::kLanesPerGroup;
  mc::select_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      logits, traj_return, group_offsets, P, prob, expected, best_return, best_expected);
  mc::count_launch();
  return mc::check_launch();
}

}  // extern "C"
