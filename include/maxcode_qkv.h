/*
 * maxcode_qkv.h - C ABI of the fused query/key/value projection + rotary embedding + append (B200, sm_100a).
 *
 * The step of the language model's decode layer that feeds the attention of maxcode_attn.h.  The paper takes the
 * model whose rollouts it samples as given (Section 2.2, "Max-Reward Search", samples candidate actions from an LLM;
 * Section 3.1, "Experimental Setup", names the models) and does not define this step; the definition is the usual
 * one of a grouped-query attention layer.  For the hidden state x[b] of candidate b and a weight matrix W with one
 * row per output feature:
 *
 *     y[b] = W x[b] (+ bias)                     N = (Hq + 2 Hkv) d features, fp32 accumulation
 *     q[b, h] = y[b, h d : (h+1) d]                                   h < Hq
 *     k[b, h] = y[b, (Hq + h) d : (Hq + h + 1) d]                     h < Hkv
 *     v[b, h] = y[b, (Hq + Hkv + h) d : (Hq + Hkv + h + 1) d]         h < Hkv
 *
 * q and k are rotated to the new token's position as mc_kv_append_rope rotates them (Su et al., "RoFormer": element
 * i of a head is the real and element i + d/2 the imaginary part of a complex number that is multiplied by
 * exp(j pos theta_base^(-2 i / d))), in single precision on the fp32 sums, and rounded to bf16 once.  q goes to the
 * caller's buffer; k and v are stored as the candidate's next suffix token exactly where mc_kv_append would store
 * them, and suffix_len[b] grows by one.  One call therefore replaces a GEMM, a rotation kernel and mc_kv_append, and
 * the projected rows never travel through HBM as a [B][N] bf16 matrix.
 *
 * With B candidates (64 to 256 in the paper's search budgets) every weight is used B times: the product streams W
 * once from HBM and is bound by that stream, not by the tensor cores.  It runs as tcgen05 tiles (two heads = one
 * 256-feature tile) fed by TMA on a persistent grid whose CTAs take equal contiguous shares of the whole stream of
 * W, so that every SM pulls on HBM throughout; where a share ends inside a head pair its fp32 partial sums are a
 * "piece", and the pieces of a pair meet, in a fixed order, in the kernel that rotates and appends.
 */
#ifndef MAXCODE_QKV_H_
#define MAXCODE_QKV_H_

#include <stddef.h>
#include <stdint.h>

#include "maxcode_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mc_qkv_plan mc_qkv_plan_t;   /* opaque, owned by the library */

/* Prepares the projection for one layout and one weight matrix.
 *   layout   an MC_BF16 layout with head_dim 128 and suffix storage (MC_ERR_UNSUPPORTED otherwise); borrowed, must
 *            outlive the plan
 *   w_qkv    DEVICE bf16 [(Hq + 2 Hkv) * 128][hidden], row n = the weights of output feature n, 16-byte aligned;
 *            borrowed (the plan keeps a tensor map over it, not a copy): must outlive the plan
 *   bias     DEVICE bf16 [(Hq + 2 Hkv) * 128] or NULL; borrowed
 *   hidden   length of a hidden state, a multiple of 64, at least 64
 * Allocates the plan's device workspace (the fp32 pieces: pieces * rows rounded up to 128 or 256 * features rounded
 * up to 256 * 4 bytes, pieces being the most any head pair has) and may synchronise.  MC_ERR_INVALID_ARG / MC_ERR_UNSUPPORTED / MC_ERR_OUT_OF_MEMORY / MC_ERR_CUDA on
 * failure (*out is then NULL). */
mc_status_t mc_qkv_plan_create(mc_kv_layout_t *layout, const void *w_qkv, const void *bias, int32_t hidden,
                               mc_qkv_plan_t **out);

/* Frees the plan and its workspace.  NULL is accepted. */
mc_status_t mc_qkv_plan_destroy(mc_qkv_plan_t *plan);

/* How the plan shares out the work: `pieces` = the most pieces any head pair is cut into, `ctas` CTAs in the
 * product's grid, `workspace_bytes` of partial sums.  Any pointer may be NULL. */
mc_status_t mc_qkv_plan_geometry(const mc_qkv_plan_t *plan, int32_t *pieces, int32_t *ctas, size_t *workspace_bytes);

/* The step: projects, rotates, writes q and appends k, v.
 *   x           DEVICE bf16 [B][hidden], 16-byte aligned
 *   q_out       DEVICE bf16 [B][Hq][128], 16-byte aligned: the rotated queries, ready for mc_decode_attn
 *   pos_offset  DEVICE int32 [B] or NULL, theta_base: as for mc_kv_append_rope; theta_base = 0 skips the rotation
 *               (pos_offset must then be NULL)
 * Three launches chained as programmatic dependents (a small one that looks up every candidate's slot and rotation
 * and moves its length; the product, which runs beside it; the sum of the product's pieces with bias, rotation and
 * the stores), asynchronous on `stream`, no allocation, no synchronisation.  A plan serves one call at a time (its
 * workspace is per plan): calls on one plan must be ordered on one stream.  A candidate whose page row is full or whose next page id is invalid gets its q
 * but no token, keeps its length, and MC_ERR_INVALID_ARG is latched in the layout's status word (mc_get_last_status);
 * a bounded device-side wait that gives up latches MC_ERR_TIMEOUT. */
mc_status_t mc_qkv_append(mc_qkv_plan_t *plan, const void *x, void *q_out, const int32_t *pos_offset,
                          double theta_base, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* MAXCODE_QKV_H_ */
