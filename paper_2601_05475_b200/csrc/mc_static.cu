// mc_decode_attn_static: the whole decode-attention step for callers that must not allocate.
//
// The partial results that the prefix and suffix passes hand to the merge normally live in a workspace
// the caller allocates, and the layout handle allocates a status word.  This entry point needs neither:
// its scratch is the file-scope device array below, which every GPU that loads the library holds until
// the process exits.  All calls share that one array.
#include <mutex>

#include "mc_internal.cuh"

namespace mc {
namespace {

constexpr size_t kStaticScratchBytes = 16u << 20;   // 16 MiB per GPU
constexpr size_t kStatusBytes = 256;                // the first bytes hold the device status word
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel can use:
// the device address is looked up once per device, with that device current.
std::mutex g_mu;
void *g_scratch_dev[kMaxDevices] = {nullptr};

mc_status_t scratch_for_current_device(unsigned char **out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return MC_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return MC_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_dev[dev]) {
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
      (void)cudaGetLastError();
      return MC_ERR_CUDA;
    }
    g_scratch_dev[dev] = ptr;
  }
  *out = static_cast<unsigned char *>(g_scratch_dev[dev]);
  return MC_OK;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
int pow2_floor(int x) { int r = 1; while (r * 2 <= x) r *= 2; return r; }

}  // namespace
}  // namespace mc

extern "C" {

size_t mc_static_scratch_bytes(void) { return mc::kStaticScratchBytes; }

mc_status_t mc_decode_attn_static(const mc_kv_layout_desc_t *d, const void *q, float scale, void *o, float *lse,
                                  int32_t *dev_status, void *stream) {
  if (!d || !q || !o || !lse) return MC_ERR_INVALID_ARG;
  if (d->num_groups < 1 || d->batch < 1 || d->num_q_heads < 1 || d->num_kv_heads < 1 || d->num_pages < 1 ||
      d->max_prefix_pages < 1 || d->max_suffix_pages < 1 || d->batch < d->num_groups ||
      d->num_q_heads % d->num_kv_heads != 0)
    return MC_ERR_INVALID_ARG;
  if (!d->k_pool || !d->v_pool || !d->group_offsets || !d->prefix_pages || !d->prefix_len || !d->suffix_pages ||
      !d->suffix_len)
    return MC_ERR_INVALID_ARG;
  const uintptr_t ptr_bits = reinterpret_cast<uintptr_t>(d->k_pool) | reinterpret_cast<uintptr_t>(d->v_pool) |
                             reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(o);
  if (ptr_bits & 15u) return MC_ERR_INVALID_ARG;
  if (d->page_size != mc::kPage || (d->dtype != MC_F32 && d->dtype != MC_BF16) ||
      (d->head_dim != 64 && d->head_dim != 128))
    return MC_ERR_UNSUPPORTED;

  mc::Params p;
  p.suffix_order = nullptr;
  p.row_limit = nullptr;
  p.k_scale = p.v_scale = nullptr;
  p.lr = 0;
  p.k_pool = d->k_pool; p.v_pool = d->v_pool;
  p.group_offsets = d->group_offsets; p.prefix_pages = d->prefix_pages; p.prefix_len = d->prefix_len;
  p.suffix_pages = d->suffix_pages; p.suffix_len = d->suffix_len;
  p.G = d->num_groups; p.B = d->batch; p.Hq = d->num_q_heads; p.Hkv = d->num_kv_heads; p.d = d->head_dim;
  p.g = d->num_q_heads / d->num_kv_heads;
  p.num_pages = d->num_pages; p.max_pp = d->max_prefix_pages; p.max_sp = d->max_suffix_pages;
  // fixed part geometry: about 8 prefix splits and 16 suffix chunks per row, 256..4096 tokens each
  const long long max_p = (long long)d->max_prefix_pages * mc::kPage, max_s = (long long)d->max_suffix_pages * mc::kPage;
  int tp = mc::pow2_floor((int)(max_p / 8 > 256 ? max_p / 8 : 256)), ts = mc::pow2_floor((int)(max_s / 16 > 256 ? max_s / 16 : 256));
  if (tp > 4096) tp = 4096;
  if (ts > 4096) ts = 4096;
  p.prefix_part_tokens = tp;
  p.suffix_part_tokens = ts;
  const long long n_prefix = (max_p + tp - 1) / tp, n_parts = n_prefix + (max_s + ts - 1) / ts;
  const long long rows = (long long)p.B * p.Hq;
  // The one thing this entry point cannot do is grow its scratch: larger problems are refused.
  if (rows > (1ll << 30) || n_parts > (1ll << 20)) return MC_ERR_WORKSPACE_TOO_SMALL;
  const size_t o_bytes = mc::align_up((size_t)rows * n_parts * p.d * sizeof(float), 256);
  const size_t l_bytes = mc::align_up((size_t)rows * n_parts * sizeof(float), 256);
  if (mc::kStatusBytes + o_bytes + l_bytes > mc::kStaticScratchBytes) return MC_ERR_WORKSPACE_TOO_SMALL;
  p.n_prefix_parts = (int)n_prefix;
  p.prefix_part_base = 0;
  p.suffix_part_base = (int)n_prefix;
  p.n_parts = (int)n_parts;

  unsigned char *scratch = nullptr;
  mc_status_t s = mc::scratch_for_current_device(&scratch);
  if (s != MC_OK) return s;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int32_t *status = dev_status ? dev_status : reinterpret_cast<int32_t *>(scratch);
  // The array still holds whatever the previous call left: the status word must start at zero.  The part
  // slots need no clearing, every slot of every row is rewritten by the two passes below.
  if (cudaMemsetAsync(status, 0, sizeof(int32_t), st) != cudaSuccess) return MC_ERR_CUDA;
  p.status = status;
  float *o_part = reinterpret_cast<float *>(scratch + mc::kStatusBytes);
  float *lse_part = reinterpret_cast<float *>(scratch + mc::kStatusBytes + o_bytes);
  const bool mma = mc::mma_supported(p, d->dtype);
  for (int mode = 0; mode < 2; ++mode) {
    s = mma ? mc::launch_mma(p, mode, q, scale, o_part, lse_part, st)
            : mc::launch_fma(p, d->dtype, mode, q, scale, o_part, lse_part, st);
    if (s != MC_OK) return s;
  }
  return mc::launch_merge(p, d->dtype, o_part, lse_part, o, lse, st);
}

}  // extern "C"
