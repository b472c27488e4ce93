// bf16, d = 128 or 64, g <= 8: split-KV attention with one warp per (candidate, kv head, part).
//
// A warp streams its token range page by page (16 tokens).  Per page and kv head it reads the 4 KB K
// slab and the 4 KB V slab exactly once with 128-bit loads straight into the register fragments of
// warp-level m16n8k16 MMAs; nothing is staged, nothing is re-read:
//   S[16 tokens][8 heads]  = K_page (16 x 128) . Q^T (128 x 8)          8 MMAs
//   O^T[128][8 heads]     += V_page^T (128 x 16) . P^T (16 x 8)         8 MMAs
// The contraction over d may visit the columns in any order, so each lane takes whole 16-byte chunks
// of a K row (and the matching chunks of its query row) as the k-columns of two consecutive MMAs.  For
// V the rows of the MMA tile are head-dim values owned by the lane group, and the token pairs the
// fragment wants are assembled from two token rows with byte permutes.  The 16x8 probability tile is
// moved from accumulator layout to B-operand layout with two 8x8 matrix transposes.
// Softmax statistics are kept per lane for the two heads the lane's accumulators belong to.
#include <cstdlib>

#include "mc_internal.cuh"

namespace mc {
namespace {

constexpr int kWarps = 4;

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
// {lo, hi} -> bf16x2 with lo in bits 0..15
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
// Private suffix data is read exactly once per step: it bypasses L1 and is marked evict-first in L2 so
// that it does not push out the shared prefix, which every step re-reads.
__device__ __forceinline__ uint64_t l2_stream_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(pol));
  return pol;
}
// Asks L2 to fetch one (page, kv head) slab; costs no registers and no shared memory.
template <int D>
__device__ __forceinline__ void l2_prefetch_slab(const void *p) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(p), "r"(kPage * D * 2) : "memory");
}
template <bool STREAM>
__device__ __forceinline__ uint4 ld16(const uint4 *p, uint64_t policy) {
  uint4 v;
  if (STREAM)
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;\n"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(policy));
  else
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// A row of D elements is D / 8 chunks of 16 bytes; NJ = D / 32 chunks per lane of a K row, NH = D / 64 of a V row.
template <int D>
struct PageRegs {
  static constexpr int NJ = D / 32, NH = D / 64;
  uint4 k[2 * NJ];  // k[j]: row gid, chunk tig+4j;  k[NJ+j]: row gid+8, same chunk
  uint4 v[4 * NH];  // v[NH x + half]: token {2tig, 2tig+1, 2tig+8, 2tig+9}[x], chunk gid + 8 half
};

template <bool STREAM, int D>
__device__ __forceinline__ void issue_loads(PageRegs<D> &r, const uint4 *kslab, const uint4 *vslab, int gid, int tig,
                                            uint64_t pol) {
  constexpr int NJ = D / 32, NH = D / 64, ROW = D / 8;
#pragma unroll
  for (int j = 0; j < NJ; ++j) {
    r.k[j] = ld16<STREAM>(kslab + gid * ROW + tig + 4 * j, pol);
    r.k[NJ + j] = ld16<STREAM>(kslab + (gid + 8) * ROW + tig + 4 * j, pol);
  }
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const int tok = 2 * tig + (x & 1) + (x >> 1) * 8;
#pragma unroll
    for (int half = 0; half < NH; ++half) r.v[NH * x + half] = ld16<STREAM>(vslab + tok * ROW + gid + 8 * half, pol);
  }
}

__device__ __forceinline__ uint32_t word(const uint4 &v, int i) {
  return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w;
}

template <int D>
struct State {
  float m0, m1, l0, l1;  // heads 2tig and 2tig+1 (l: this lane's share)
  float o[D / 16][4];    // o[i]: head-dim tile i; [0],[1]: d = D_gid[2i], heads 2tig, 2tig+1; [2],[3]: D_gid[2i+1]
};

// One page: tokens [tok_base, tok_base+16), those at or beyond `hi` masked.
template <int D>
__device__ __forceinline__ void compute_page(State<D> &st, const PageRegs<D> &r, const uint32_t (&qf)[D / 32][4],
                                             float sl2, int tok_base, int hi, int gid, int tig) {
  constexpr int NJ = D / 32, NH = D / 64;
  float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int j = 0; j < NJ; ++j) {
    mma16816(c, r.k[j].x, r.k[NJ + j].x, r.k[j].y, r.k[NJ + j].y, qf[j][0], qf[j][1]);
    mma16816(c, r.k[j].z, r.k[NJ + j].z, r.k[j].w, r.k[NJ + j].w, qf[j][2], qf[j][3]);
  }
  const bool v0 = tok_base + gid < hi, v1 = tok_base + gid + 8 < hi;
  const float s00 = v0 ? c[0] * sl2 : -INFINITY, s01 = v0 ? c[1] * sl2 : -INFINITY;
  const float s10 = v1 ? c[2] * sl2 : -INFINITY, s11 = v1 ? c[3] * sl2 : -INFINITY;
  float mx0 = fmaxf(s00, s10), mx1 = fmaxf(s01, s11);
#pragma unroll
  for (int sh = 4; sh <= 16; sh <<= 1) {
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
  }
  const float mn0 = fmaxf(st.m0, mx0), mn1 = fmaxf(st.m1, mx1);
  const float r0 = mn0 == -INFINITY ? 0.f : mn0, r1 = mn1 == -INFINITY ? 0.f : mn1;
  const float a0 = fast_exp2(st.m0 - r0), a1 = fast_exp2(st.m1 - r1);
  const float p00 = fast_exp2(s00 - r0), p01 = fast_exp2(s01 - r1);
  const float p10 = fast_exp2(s10 - r0), p11 = fast_exp2(s11 - r1);
  st.l0 = st.l0 * a0 + (p00 + p10);
  st.l1 = st.l1 * a1 + (p01 + p11);
  st.m0 = mn0;
  st.m1 = mn1;
#pragma unroll
  for (int i = 0; i < D / 16; ++i) {
    st.o[i][0] *= a0; st.o[i][1] *= a1; st.o[i][2] *= a0; st.o[i][3] *= a1;
  }
  const uint32_t pb0 = transpose8x8(pack_bf16x2(p00, p01));
  const uint32_t pb1 = transpose8x8(pack_bf16x2(p10, p11));
#pragma unroll
  for (int half = 0; half < NH; ++half) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t x0 = word(r.v[0 * NH + half], i), y0 = word(r.v[1 * NH + half], i);
      const uint32_t x1 = word(r.v[2 * NH + half], i), y1 = word(r.v[3 * NH + half], i);
      mma16816(st.o[half * 4 + i], __byte_perm(x0, y0, 0x5410), __byte_perm(x0, y0, 0x7632),
               __byte_perm(x1, y1, 0x5410), __byte_perm(x1, y1, 0x7632), pb0, pb1);
    }
  }
}

template <int MODE, int D>
__device__ __forceinline__ void
attn_mma_body(const Params &p, const __nv_bfloat16 *__restrict__ q, float sl2, float *__restrict__ o_part,
              float *__restrict__ lse_part, int prefetch_pages) {
  constexpr bool STREAM = MODE == kSuffix;  // private suffix data is read exactly once
  const int lane = threadIdx.x & 31, gid = lane >> 2, tig = lane & 3;
  const int nparts_mode = MODE == kPrefix ? p.n_prefix_parts : p.n_parts - p.suffix_part_base;
  const long long n_items = (long long)p.B * p.Hkv * nparts_mode;
  // the order CTAs are launched in may be given (longest first); every CTA index appears once
  const long long cta = MODE == kSuffix && p.suffix_order ? __ldg(p.suffix_order + blockIdx.x) : blockIdx.x;
  const long long item = cta * kWarps + (threadIdx.x >> 5);
  if (item >= n_items) return;
  int b, h, part;
  if (MODE == kSuffix) {  // kv heads of one page are adjacent in the pool: neighbours stream neighbours
    h = (int)(item % p.Hkv);
    part = (int)((item / p.Hkv) % nparts_mode);
    b = (int)(item / ((long long)p.Hkv * nparts_mode));
  } else {  // candidates of a group walk the same pages at the same time
    b = (int)(item % p.B);
    h = (int)((item / p.B) % p.Hkv);
    part = (int)(item / ((long long)p.B * p.Hkv));
  }
  // The item's first two page ids do not depend on the sequence length (only on the part index): their
  // loads, the length's and the queries' are issued together instead of one after the other.  Entries of a
  // page-table row beyond the sequence are read here but never used as page ids.
  int pid_first = 0, pid_second = 0;
  if (MODE == kSuffix) {
    const int first_pg = part * (p.suffix_part_tokens >> 4);
    const int32_t *row_pages = p.suffix_pages + (size_t)b * p.max_sp;
    if (first_pg < p.max_sp) pid_first = __ldg(row_pages + first_pg);
    if (first_pg + 1 < p.max_sp) pid_second = __ldg(row_pages + first_pg + 1);
  }
  uint32_t qf[D / 32][4];
#pragma unroll
  for (int j = 0; j < D / 32; ++j) {
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (gid < p.g) v = __ldg(reinterpret_cast<const uint4 *>(q + ((size_t)b * p.Hq + (size_t)h * p.g + gid) * D) + tig + 4 * j);
    qf[j][0] = v.x; qf[j][1] = v.y; qf[j][2] = v.z; qf[j][3] = v.w;
  }
  const Span sp = resolve_span<MODE>(p, b, part);
  const int g = p.g;
  const size_t row0 = (size_t)b * p.Hq + (size_t)h * g;
  if (sp.lo >= sp.hi) {
    if (lane < g) lse_part[(row0 + lane) * p.n_parts + sp.part] = -INFINITY;
    return;
  }
  State<D> st;
  st.m0 = st.m1 = -INFINITY;
  st.l0 = st.l1 = 0.f;
#pragma unroll
  for (int i = 0; i < D / 16; ++i) st.o[i][0] = st.o[i][1] = st.o[i][2] = st.o[i][3] = 0.f;

  const uint4 *kpool = reinterpret_cast<const uint4 *>(p.k_pool);
  const uint4 *vpool = reinterpret_cast<const uint4 *>(p.v_pool);
  const int pg_first = sp.lo >> 4, pg_end = (sp.hi + 15) >> 4;
  constexpr size_t kSlab = kPage * D * 2 / 16;  // uint4 per (page, kv head)

  // hi_of(page id): a page id outside the pool is replaced by page 0 and fully masked
  auto slab_of = [&](int pid, int &hi_eff) -> size_t {
    hi_eff = sp.hi;
    if ((unsigned)pid >= (unsigned)p.num_pages) {
      latch(p, kDevBadPage);
      pid = 0;
      hi_eff = 0;
    }
    return slab_index(p, pid, h) * kSlab;
  };

  const uint64_t pol = l2_stream_policy();
  PageRegs<D> ra, rb;
  int hi_a, hi_b = 0;
  {
    const size_t s = slab_of(MODE == kSuffix ? pid_first : __ldg(sp.pages + pg_first), hi_a);
    issue_loads<STREAM, D>(ra, kpool + s, vpool + s, gid, tig, pol);
  }
  int pid_next = 0;
  if (pg_first + 1 < pg_end) pid_next = MODE == kSuffix ? pid_second : __ldg(sp.pages + pg_first + 1);
  // The register double buffer covers one page of latency; the stream from HBM is kept kPrefetch pages
  // further ahead by asking L2 for the slabs (lanes 0 and 1, one page each per two-page iteration).
  const int kPrefetch = prefetch_pages;
  auto prefetch_page = [&](int pgi, int pid) {
    if (pgi < pg_end && (unsigned)pid < (unsigned)p.num_pages) {
      const size_t s = slab_index(p, pid, h) * kSlab;
      l2_prefetch_slab<D>(kpool + s);
      l2_prefetch_slab<D>(vpool + s);
    }
  };
  if (STREAM && lane < kPrefetch) {   // kPrefetch <= 32
    const int pgi = pg_first + 2 + lane;
    if (pgi < pg_end) prefetch_page(pgi, __ldg(sp.pages + pgi));
  }
  for (int pg = pg_first; pg < pg_end; pg += 2) {
    const bool has_b = pg + 1 < pg_end;
    int pid_next2 = 0;
    const int pf_pg = pg + 2 + kPrefetch + (lane & 1);
    int pf_pid = -1;
    if (STREAM && pf_pg < pg_end) pf_pid = __ldg(sp.pages + pf_pg);   // used at the end of the iteration
    if (has_b) {
      const size_t s = slab_of(pid_next, hi_b);
      issue_loads<STREAM, D>(rb, kpool + s, vpool + s, gid, tig, pol);
      if (pg + 2 < pg_end) pid_next2 = __ldg(sp.pages + pg + 2);
    }
    compute_page(st, ra, qf, sl2, pg * kPage, hi_a, gid, tig);
    if (has_b) {
      if (pg + 2 < pg_end) {
        const size_t s = slab_of(pid_next2, hi_a);
        issue_loads<STREAM, D>(ra, kpool + s, vpool + s, gid, tig, pol);
        if (pg + 3 < pg_end) pid_next = __ldg(sp.pages + pg + 3);
      }
      compute_page(st, rb, qf, sl2, (pg + 1) * kPage, hi_b, gid, tig);
    }
    if (STREAM && lane < 2) prefetch_page(pf_pg, pf_pid);
  }

  float l0 = st.l0, l1 = st.l1;
#pragma unroll
  for (int sh = 4; sh <= 16; sh <<= 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, sh);
    l1 += __shfl_xor_sync(0xffffffffu, l1, sh);
  }
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int head = 2 * tig + e;
    if (head >= g) continue;
    const float l = e ? l1 : l0, m = e ? st.m1 : st.m0;
    const size_t slot = (row0 + head) * p.n_parts + sp.part;
    if (gid == 0) lse_part[slot] = l > 0.f ? (m + log2f(l)) * kLn2 : -INFINITY;
    if (l > 0.f) {
      const float inv = 1.f / l;
      float *dst = o_part + slot * D + 8 * gid;
#pragma unroll
      for (int half = 0; half < D / 64; ++half) {
        const float(*t)[4] = st.o + half * 4;
        float4 w0 = make_float4(t[0][e] * inv, t[0][e + 2] * inv, t[1][e] * inv, t[1][e + 2] * inv);
        float4 w1 = make_float4(t[2][e] * inv, t[2][e + 2] * inv, t[3][e] * inv, t[3][e + 2] * inv);
        *reinterpret_cast<float4 *>(dst + half * 64) = w0;
        *reinterpret_cast<float4 *>(dst + half * 64 + 4) = w1;
      }
    }
  }
}

template <int MODE, int D>
__global__ void __launch_bounds__(kWarps * 32, 2)
attn_mma_kernel(Params p, const __nv_bfloat16 *__restrict__ q, float sl2, float *__restrict__ o_part,
                float *__restrict__ lse_part, int prefetch_pages) {
  attn_mma_body<MODE, D>(p, q, sl2, o_part, lse_part, prefetch_pages);
  // As the programmatic dependent of the prefix pass the suffix grid starts before that one ends; one thread of the
  // grid waits for the prerequisite grid before it exits, so that this grid - and the merge behind it - cannot
  // complete earlier.  Without a prerequisite the instruction returns at once.
  if (MODE == kSuffix && blockIdx.x == gridDim.x - 1 && threadIdx.x == 0)
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
}

}  // namespace

// L2 prefetch distance of the suffix stream in pages (MC_SUFFIX_PREFETCH, default 2, 0 disables).
static int suffix_prefetch_pages() {
  static int v = -1;
  if (v < 0) {
    const char *e = std::getenv("MC_SUFFIX_PREFETCH");
    v = e && *e ? std::atoi(e) : 2;
    if (v < 0) v = 0;
    if (v > 32) v = 32;
  }
  return v;
}

int mma_items_per_cta() { return kWarps; }

bool mma_supported(const Params &p, int dtype) {
  return dtype == MC_BF16 && (p.d == 128 || p.d == 64) && p.g >= 1 && p.g <= 8;
}

mc_status_t launch_mma(const Params &p, int mode, const void *q, float scale, float *o_part, float *lse_part,
                       cudaStream_t stream, bool beside_previous) {
  const int nparts_mode = mode == kPrefix ? p.n_prefix_parts : p.n_parts - p.suffix_part_base;
  const long long n_items = (long long)p.B * p.Hkv * nparts_mode;
  if (n_items == 0) return MC_OK;
  const unsigned grid = (unsigned)((n_items + kWarps - 1) / kWarps);
  const float sl2 = scale * kLog2e;
  const __nv_bfloat16 *qb = reinterpret_cast<const __nv_bfloat16 *>(q);
  if (mode == kPrefix) {
    if (p.d == 128) attn_mma_kernel<kPrefix, 128><<<grid, kWarps * 32, 0, stream>>>(p, qb, sl2, o_part, lse_part, 0);
    else attn_mma_kernel<kPrefix, 64><<<grid, kWarps * 32, 0, stream>>>(p, qb, sl2, o_part, lse_part, 0);
  } else {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kWarps * 32);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = beside_previous ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, p.d == 128 ? attn_mma_kernel<kSuffix, 128> : attn_mma_kernel<kSuffix, 64>, p, qb, sl2,
                           o_part, lse_part, suffix_prefetch_pages()) != cudaSuccess) {
      count_launch();
      return MC_ERR_CUDA;
    }
  }
  count_launch();
  return check_launch();
}

}  // namespace mc
