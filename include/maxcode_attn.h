/*
 * maxcode_attn.h - C ABI of the shared-prefix grouped-query decode-attention library (B200, sm_100a).
 *
 * Operation.  One decode step for B candidate rollouts organised in G prompt groups.  All candidates of
 * a group share the group's prompt (the "prefix"); each candidate has a private continuation (the
 * "suffix").  This is the workload of the max-reward search of Section 2.2 ("Max-Reward Search": k
 * candidate actions are sampled from one state s_i) with the budgets of Section 3.1 ("Experimental
 * Setup": K = 8 candidates x depth 8; flat sampling with n = 64).  For candidate b (group j), query
 * head hq and its kv head h = hq / (Hq / Hkv):
 *
 *     K    = concat(Kprefix_j[0:P_j, h], Ksuffix_b[0:s_b, h])          (V likewise)
 *     z_t  = scale * <q[b, hq], K_t>
 *     lse  = log sum_t exp(z_t)                  natural logarithm
 *     o    = sum_t exp(z_t - lse) * V_t
 *
 * The library computes this as three passes: a prefix pass (each group's prefix is attended by the
 * stacked queries of all its candidates), a suffix pass (each candidate's private tokens, split into
 * token chunks) and a log-sum-exp merge of the partial results.
 *
 * Memory layout (all DEVICE memory, owned by the caller, borrowed by the layout object):
 *   k_pool, v_pool  [num_pages][Hkv][page_size][d]   elements of `dtype`; 16-byte aligned.  One (page, kv head)
 *                                              slab is page_size*d contiguous elements; page_size is 16 (the
 *                                              layout the kernels walk directly), 32 or 64 tokens.
 *   prefix_pages    int32 [G][max_prefix_pages]   physical page ids of group j's prefix, in token order
 *   prefix_len      int32 [G]                     tokens (the last page may be partially filled)
 *   suffix_pages    int32 [B][max_suffix_pages]   physical page ids of candidate b's suffix
 *   suffix_len      int32 [B]                     tokens; read on the device at every call, advanced
 *                                                 by mc_kv_append
 *   group_offsets   int32 [G+1]                   candidates group_offsets[j] .. group_offsets[j+1]-1
 *                                                 belong to group j (contiguous in b)
 *   q               [B][Hq][d] `dtype`            o  [B][Hq][d] `dtype`        lse  [B][Hq] float
 * Page-table entries beyond a sequence's pages are never dereferenced.  Slots of a page beyond the
 * sequence length may hold any finite values.  A page id outside [0, num_pages) makes the kernels skip
 * that page and latch MC_ERR_INVALID_ARG in the device status word (see mc_get_last_status).
 * With page_size 32 or 64 the kernels still move 16-token blocks (a page is 2 or 4 of them, contiguous per kv head)
 * and read page tables that the layout object derives from the caller's once, at create time: after changing entries
 * of prefix_pages, suffix_pages or an outer level's pages call mc_kv_layout_refresh_tables.  With page_size 16 the
 * caller's tables are read at every call and there is nothing to refresh.
 *
 * Partial results ("parts").  rows = B*Hq, row = b*Hq + hq.  Each row has n_parts slots:
 *   parts [0, n_prefix_parts)            prefix splits of prefix_part_tokens tokens each
 *   parts [n_prefix_parts, n_parts)      suffix chunks of suffix_part_tokens tokens each
 *   o_part   float [rows][n_parts][d]    normalised partial output of that token range
 *   lse_part float [rows][n_parts]       its log-sum-exp; -inf marks an empty part (o_part undefined)
 *
 * Conventions.  All hot calls (append, prefix, suffix, merge, decode) are asynchronous on `stream`
 * (a cudaStream_t passed as void*; NULL is the default stream), allocate nothing and do not
 * synchronise.  Errors detectable on the host are returned immediately; conditions detected on the
 * device are latched in a status word.  A layout handle is not thread-safe; distinct handles are
 * independent.  No entry point throws.
 */
#ifndef MAXCODE_ATTN_H_
#define MAXCODE_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MC_OK = 0,
  MC_ERR_INVALID_ARG = 1,        /* null / misaligned pointer, inconsistent sizes, bad page id, full suffix */
  MC_ERR_UNSUPPORTED = 2,        /* dtype / head_dim / page_size / head ratio outside the supported set */
  MC_ERR_OUT_OF_MEMORY = 3,
  MC_ERR_WORKSPACE_TOO_SMALL = 4,
  MC_ERR_CUDA = 5,               /* a CUDA runtime call failed */
  MC_ERR_TIMEOUT = 6             /* a bounded device-side wait gave up */
} mc_status_t;

/* MC_F32 / MC_BF16: the cache, q and o all have that type.  MC_FP8_E4M3: the cache holds 8-bit floating-point codes
 * (E4M3 of Micikevicius et al., "FP8 Formats for Deep Learning": 1 sign, 4 exponent bits with bias 7, 3 mantissa
 * bits, no infinities, largest magnitude 448) with one float scale per (page, kv head) for K and one for V - a code
 * stands for decode(code) * scale - while q, o, k_new and v_new are bf16.  The paper takes the model and its cache as
 * given; this halves the bytes per cached token (2 * Hkv * d instead of 4 * Hkv * d).  head_dim must be 128 and
 * Hq / Hkv at most 8. */
typedef enum { MC_F32 = 0, MC_BF16 = 1, MC_FP8_E4M3 = 2 } mc_dtype_t;

typedef struct mc_kv_layout mc_kv_layout_t;   /* opaque, owned by the library */

typedef struct {
  int32_t num_groups;            /* G >= 1 */
  int32_t batch;                 /* B >= 1, total candidates */
  int32_t num_q_heads;           /* Hq, a multiple of Hkv */
  int32_t num_kv_heads;          /* Hkv */
  int32_t head_dim;              /* d: 64, 128 or 256 (256: every pass on the plain-ALU kernel; MC_FP8_E4M3, the
                                    tensor-core passes and mc_decode_attn_static: see their own limits) */
  int32_t page_size;             /* tokens per page: 16, 32 or 64 (MC_FP8_E4M3 and mc_decode_attn_static: 16) */
  int32_t num_pages;             /* pages in each pool */
  int32_t max_prefix_pages;      /* row stride of prefix_pages */
  int32_t max_suffix_pages;      /* row stride of suffix_pages; 0: no private tokens at all (scoring whole
                                    sequences): suffix_pages / suffix_len may be NULL, no suffix part slots,
                                    no suffix launch, mc_kv_append returns MC_ERR_INVALID_ARG */
  int32_t dtype;                 /* mc_dtype_t */
  void *k_pool, *v_pool;         /* device */
  const int32_t *group_offsets;  /* device, [G+1] */
  const int32_t *prefix_pages;   /* device, [G][max_prefix_pages] */
  const int32_t *prefix_len;     /* device, [G] */
  const int32_t *suffix_pages;   /* device, [B][max_suffix_pages] */
  int32_t *suffix_len;           /* device, [B]; mc_kv_append increments it */
  float *k_scale, *v_scale;      /* device, [num_pages][Hkv] each; MC_FP8_E4M3 only (else ignored, may be NULL).  Read by
                                    the attention passes; mc_kv_append writes the entry of a page when it writes the
                                    page's first token */
} mc_kv_layout_desc_t;

typedef struct {
  int32_t rows;                  /* B*Hq */
  int32_t n_parts;               /* part slots per row */
  int32_t n_prefix_parts;        /* prefix part slots of all cascade levels (base level first) */
  int32_t prefix_part_tokens;    /* tokens per prefix split of the base level (multiple of 16) */
  int32_t suffix_part_tokens;    /* tokens per suffix chunk (multiple of 16) */
  int32_t head_dim;
  int32_t prefix_ctas;           /* persistent CTAs of the tensor-core prefix pass; 0: that kernel is not used */
} mc_part_geometry_t;

/* Builds the layout object (step 1 of the path, the paged-KV layout): validates the descriptor, fixes
 * the part geometry from the table strides and allocates the handle's small device state (status word).
 * May synchronise the device.  Pointers in `desc` are borrowed and must outlive the handle.
 * Returns MC_ERR_INVALID_ARG / MC_ERR_UNSUPPORTED / MC_ERR_OUT_OF_MEMORY / MC_ERR_CUDA on failure
 * (*out is then NULL). */
mc_status_t mc_kv_layout_create(const mc_kv_layout_desc_t *desc, mc_kv_layout_t **out);

/* An outer level of a prefix cascade: token ranges shared by MORE candidates than the base descriptor's groups
 * (e.g. a system prompt shared by every prompt group, in front of each group's own prefix).  Same pools, another
 * group map: candidates group_offsets[j] .. group_offsets[j+1]-1 (contiguous in b) attend to pages[j][0 : len[j]].
 * All pointers DEVICE memory, borrowed for the life of the handle. */
typedef struct {
  int32_t num_groups;            /* groups at this level, 1 <= num_groups <= B */
  int32_t max_pages;             /* row stride of pages */
  const int32_t *group_offsets;  /* device, [num_groups+1], increasing, last = B */
  const int32_t *pages;          /* device, [num_groups][max_pages] */
  const int32_t *len;            /* device, [num_groups], tokens */
  const int32_t *row_limit;      /* device, [B], or NULL.  Candidate b sees only the first row_limit[b] tokens of its
                                    group at this level (a causal mask when the candidates of a group are the query
                                    positions of one sequence and the level holds that sequence's own tokens).  Must not
                                    decrease from one candidate of a group to the next; values above len are the same as
                                    len, 0 hides the level from that candidate. */
} mc_prefix_level_t;

/* mc_kv_layout_create for a cascade deeper than two levels: every candidate attends to the tokens of each outer
 * level's group it belongs to, to its base-level prefix and to its suffix (the order of concatenation does not
 * change the result).  The prefix pass covers every level, each level writes part slots of its own, the merge
 * combines them all.  n_outer <= 3.  With n_outer = 0 this is mc_kv_layout_create.
 * Scoring / prefill of whole sequences uses the same call: make every (sequence, query position) a candidate, give
 * the base descriptor the shared prompt (its groups then hold all positions of all sequences of a prompt group) and
 * empty suffixes, and add one outer level whose groups are the sequences, whose pages are each sequence's own
 * tokens and whose row_limit is position + 1. */
mc_status_t mc_kv_layout_create_cascade(const mc_kv_layout_desc_t *desc, const mc_prefix_level_t *outer,
                                        int32_t n_outer, mc_kv_layout_t **out);

/* Frees the handle and its device state.  NULL is accepted. */
mc_status_t mc_kv_layout_destroy(mc_kv_layout_t *layout);

/* Debug aid: checks on the device that group_offsets is increasing and ends at B, that lengths fit the
 * table strides, that every referenced page id lies in [0, num_pages) and that no page is referenced
 * twice.  Synchronises `stream`.  `scratch` is device memory of at least num_pages * (page_size / 16) * 4 bytes.
 * With page_size 32 or 64 it first re-derives the layout's tables from the caller's (mc_kv_layout_refresh_tables). */
mc_status_t mc_kv_layout_validate(mc_kv_layout_t *layout, void *scratch, size_t scratch_bytes, void *stream);

/* MC_FP8_E4M3 layouts whose prefix pass runs on the tensor cores keep the prefix levels widened to 16-bit pools of
 * their own (made by mc_kv_layout_create*, which waits for them; 4 * Hkv * d bytes per prefix page slot of the
 * tables): that pass needs 16-bit operands and the prefix does not change while the candidates decode.  After
 * changing prefix pages, their scales, the prefix tables or prefix_len of such a layout, call this to widen them
 * again (asynchronous on `stream`).  On every other layout it does nothing and returns MC_OK. */
mc_status_t mc_kv_layout_refresh_prefix(mc_kv_layout_t *layout, void *stream);

/* page_size 32 or 64: rewrites the layout's own page tables (in 16-token blocks: entry e of a caller's table becomes
 * blocks e * page_size / 16 + 0, 1, ...) from the caller's prefix_pages, suffix_pages and outer-level pages as they
 * are now; one small launch per table, asynchronous on `stream`, order it before the next attention or append call.
 * Needed after the caller changes a table entry (assigning a page to a growing suffix, swapping a prefix); lengths
 * are always read live and need no refresh.  page_size 16: does nothing and returns MC_OK. */
mc_status_t mc_kv_layout_refresh_tables(mc_kv_layout_t *layout, void *stream);

/* Part geometry chosen at create time (needed to size and index o_part / lse_part). */
mc_status_t mc_kv_layout_geometry(const mc_kv_layout_t *layout, mc_part_geometry_t *out);

/* Bytes of device workspace that mc_decode_attn and mc_decode_step_host need (partials + staging). */
size_t mc_workspace_bytes(const mc_kv_layout_t *layout);

/* Appends one token per candidate: writes k_new/v_new [B][Hkv][d] (device, `dtype`) into slot
 * suffix_len[b] % 16 of page suffix_pages[b][suffix_len[b] / 16], then increments suffix_len[b], all on
 * the device.  A candidate whose page row is full is left unchanged and MC_ERR_INVALID_ARG is latched.
 * MC_FP8_E4M3: k_new / v_new are bf16 and are quantised on the way in.  The token that opens a page (slot 0) fixes
 * that page's scales, per kv head and for K and V separately: scale = (2 * max|row|) / 448 (1 for a row of zeros), so
 * later rows up to twice as large still fit and larger values saturate at +-448 * scale; the other 15 tokens of the
 * page use the stored scale.  code = e4m3(x / scale), the quotient rounded once in single precision, the conversion
 * to the nearest code, ties to even.  The cache therefore does not depend on how tokens were grouped into calls. */
mc_status_t mc_kv_append(mc_kv_layout_t *layout, const void *k_new, const void *v_new, void *stream);

/* mc_kv_append with rotary position embedding (the step of the language model's decode layer that precedes the
 * attention; the paper takes the model as given and does not define it - the definition is the published one of
 * Su et al., "RoFormer").  A head's d elements are d/2 complex numbers, element i the real and element i + d/2
 * the imaginary part; the one at index i of a token at position pos is multiplied by exp(j pos theta_i),
 * theta_i = theta_base^(-2 i / d).  pos of candidate b's new token = suffix_len[b] (before the increment) plus
 * pos_offset[b] when pos_offset (device int32 [B]) is given, else plus the prefix lengths of b's groups on every
 * cascade level, read on the device.  The rotated key row is stored in the cache, v_new unchanged; when q
 * (device [B][Hq][d], 16-byte aligned) is not NULL its rows are rotated in place to the same position.  Angles
 * are formed in double precision, the rotation in single precision, results rounded to `dtype`.  Errors as
 * mc_kv_append; theta_base <= 0 is MC_ERR_INVALID_ARG. */
mc_status_t mc_kv_append_rope(mc_kv_layout_t *layout, const void *k_new, const void *v_new, void *q,
                              const int32_t *pos_offset, double theta_base, void *stream);

/* Appends up to n_max tokens per candidate in one call (ingesting a prompt or a candidate's whole continuation
 * before it is scored - the value model of Section 2.3, "Generative Value Function Guided Search", reads every
 * candidate in full - or storing several speculated tokens):
 *   k_new, v_new  device [B][n_max][Hkv][d], of the type mc_kv_append takes
 *   n_new         device int32 [B] or NULL: candidate b gets its first min(max(n_new[b], 0), n_max) tokens; NULL: n_max
 * Token t of candidate b lands at suffix position suffix_len[b] + t; then suffix_len[b] grows by the count, on the
 * device.  A candidate whose tokens do not all fit its page row, or whose row lacks a valid page id for one of them,
 * keeps its length (rows of it may have been written beyond that length) and MC_ERR_INVALID_ARG is latched.
 * theta_base > 0 rotates the keys as mc_kv_append_rope does, token t to position (tokens in front of the candidate's
 * suffix, or pos_offset[b]) + suffix_len[b] + t, and, when q (device [B][n_max][Hq][d]) is given, the query rows of
 * the same tokens in place; theta_base = 0 stores the keys as they are (q and pos_offset must then be NULL).
 * An MC_FP8_E4M3 cache is written as by successive mc_kv_append calls (a page's scales come from the token that
 * opens it, whether that token is part of this call or was stored before); the rotation is not available on it.
 * n_max <= 65535.  Two launches; asynchronous on `stream`. */
mc_status_t mc_kv_append_tokens(mc_kv_layout_t *layout, const void *k_new, const void *v_new, int32_t n_max,
                                const int32_t *n_new, void *q, const int32_t *pos_offset, double theta_base,
                                void *stream);

/* Prefix pass: for every group and kv head, the stacked queries of all the group's candidates attend
 * to the group's prefix; writes parts [0, n_prefix_parts) of every row.  q: device [B][Hq][d]. */
mc_status_t mc_prefix_attn(mc_kv_layout_t *layout, const void *q, float scale,
                           float *o_part, float *lse_part, void *stream);

/* Suffix pass: every candidate attends to its private suffix, chunk by chunk; writes parts
 * [n_prefix_parts, n_parts) of every row.  On a layout without suffix storage (max_suffix_pages = 0) there are
 * no such parts and the call launches nothing. */
mc_status_t mc_suffix_attn(mc_kv_layout_t *layout, const void *q, float scale,
                           float *o_part, float *lse_part, void *stream);

/* Log-sum-exp merge over the n_parts slots of every row:  m = max_i lse_i, w_i = exp(lse_i - m),
 * o = sum_i w_i o_i / sum_i w_i, lse = m + log sum_i w_i.  Parts with lse = -inf are skipped; a row with
 * no non-empty part gets o = 0, lse = -inf.  o: device [B][Hq][d] `dtype`; lse: device [B][Hq] float. */
mc_status_t mc_merge_lse(mc_kv_layout_t *layout, const float *o_part, const float *lse_part,
                         void *o, float *lse, void *stream);

/* The whole step: prefix pass, suffix pass, merge.  `ws` is device memory of at least
 * mc_workspace_bytes(layout) bytes, 256-byte aligned (else MC_ERR_WORKSPACE_TOO_SMALL / INVALID_ARG).
 * On a layout without suffix storage (max_suffix_pages = 0) whose prefix pass yields one part per row (one
 * unsplit level, or two nested unsplit levels), the prefix pass writes o and lse itself: one launch, `ws` unused. */
mc_status_t mc_decode_attn(mc_kv_layout_t *layout, const void *q, float scale,
                           void *o, float *lse, void *ws, size_t ws_bytes, void *stream);

/* One whole decode step with device-resident tensors: appends k_new/v_new (as mc_kv_append) and runs
 * mc_decode_attn.  k_new = v_new = NULL skips the append (then identical to mc_decode_attn).  The suffix pass
 * is scheduled beside the prefix pass (it starts once the prefix pass's CTAs are running); everything is
 * enqueued on `stream` or on streams of the handle that fork from and join it, so the call can be captured
 * into a CUDA graph and replayed: the lengths it depends on are read on the device. */
mc_status_t mc_decode_step(mc_kv_layout_t *layout, const void *k_new, const void *v_new, const void *q,
                           float scale, void *o, float *lse, void *ws, size_t ws_bytes, void *stream);

/* Same step for a caller that keeps its per-step tensors on the HOST: copies q (and, if k_new/v_new are
 * non-NULL, the appended token) host->device into the workspace, appends, runs mc_decode_attn, copies o
 * and lse device->host and synchronises `stream`.  Host pointers should be pinned for the copies to be
 * asynchronous.  The KV pools stay resident on the device. */
mc_status_t mc_decode_step_host(mc_kv_layout_t *layout, const void *k_new_host, const void *v_new_host,
                                const void *q_host, float scale, void *o_host, float *lse_host,
                                void *ws, size_t ws_bytes, void *stream);

/* (No counterpart in the paper: an addition for callers that cannot allocate.)
 * The whole step - prefix pass, suffix pass, merge - without a layout handle, a workspace or any
 * allocation.  It is meant for code that runs where cudaMalloc is off limits: inside a serving loop
 * whose memory was carved up at start-up by another allocator, in a plug-in that is forbidden to touch
 * the device heap, or late in a process whose GPU memory is already fully committed.  The partial results
 * go to a fixed scratch array compiled into the library (mc_static_scratch_bytes() bytes, 16 MiB, resident
 * on every GPU that loads the library until the process exits).  The call itself calls no cudaMalloc /
 * cudaFree and no allocating library routine.
 *   desc        same descriptor as mc_kv_layout_create (all pointers DEVICE memory, borrowed for the call)
 *   q, o, lse   device, as for mc_decode_attn
 *   dev_status  optional device int32: set to 0, then to MC_ERR_INVALID_ARG if a bad page id or length is
 *               met (such pages are skipped).  NULL: the condition is recorded nowhere the caller can read.
 * Limits and rules:
 *   - status(256 B) + rows*n_parts*(d+1)*4 bytes of partials must fit the scratch array, with rows = B*Hq
 *     and n_parts = ceil(max_prefix_tokens/Tp) + ceil(max_suffix_tokens/Ts), Tp and Ts its own fixed rule
 *     (about 8 prefix splits and 16 suffix chunks, 256..4096 tokens); otherwise MC_ERR_WORKSPACE_TOO_SMALL and nothing
 *     is launched.  (Configuration 1 needs about 1.7 MiB; the large benchmark configurations do not fit.)
 *   - The first call on each device looks up the scratch array's device address (the device must be
 *     current).  With CUDA's lazy module loading that look-up is also the moment the driver loads the module
 *     holding the array and sets its 16 MiB aside on that device.  So make one call per device at start-up,
 *     while memory is still to be had and outside any stream capture; if the device cannot spare the
 *     16 MiB any more, that first call returns MC_ERR_CUDA.  Later calls reserve nothing.
 *   - All calls share the one array and it keeps the previous call's contents (the call clears the status
 *     word it uses; every part slot is rewritten).  Two calls whose kernels overlap on the GPU - different
 *     streams, or different threads - race on it: serialise them.
 *   - Asynchronous on `stream`, like the other hot calls.  Both passes run on the warp-level kernels. */
mc_status_t mc_decode_attn_static(const mc_kv_layout_desc_t *desc, const void *q, float scale, void *o,
                                  float *lse, int32_t *dev_status, void *stream);

/* Size in bytes of the scratch array behind mc_decode_attn_static. */
size_t mc_static_scratch_bytes(void);

/* Reads and clears the device status word (synchronises `stream`): MC_OK, or the first latched error. */
mc_status_t mc_get_last_status(mc_kv_layout_t *layout, void *stream);

/* (No counterpart in the paper: a measurement aid.)  Streams `bytes` bytes of DEVICE memory at `buf` (16-byte
 * aligned) through the SMs once with 16-byte read-only loads and stores nothing but, possibly, one word at `sink`
 * (device uint32).  Timed on a buffer several times the L2 size it gives the read-only HBM rate a streaming kernel
 * can reach on this GPU, the ceiling of the suffix pass; a copy-based figure counts reads and writes.
 * Asynchronous on `stream`. */
mc_status_t mc_hbm_read_probe(const void *buf, size_t bytes, uint32_t *sink, void *stream);

/* Kernel launches issued by this library since it was loaded (all handles, all threads). */
uint64_t mc_launch_count(void);

const char *mc_status_string(mc_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* MAXCODE_ATTN_H_ */
