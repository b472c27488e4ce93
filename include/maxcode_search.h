/*
 * maxcode_search.h - C ABI of the batched max-reward search bookkeeping (B200, sm_100a).
 *
 * The search loop of the paper keeps, for every trajectory tau = (s_0, ..., s_T) it expands, a handful of scalar
 * quantities.  With f_r(e_t) the categorical reward of step t (Section 2.3, "Categorical Reward Formulation"),
 * f(e_t) the raw reward (the speed-up of a correct candidate, 0 for an incorrect one) and gamma the discount:
 *
 *     u_t   = max_{k <= t} gamma^(k-1) f_r(e_k)                       best discounted reward so far   (Section 2.3)
 *     v*_t  = max(u_t / gamma, max_{k >= t} gamma^(k-t) f_r(e_k))      value target                    (Section 2.3)
 *     lab_t = f_r(max_{k >= t} gamma^(k-t) f(e_k))                     cross-entropy label             (Section 2.3)
 *     G     = max_{t in [1,T]} gamma^(t-1) f_r(e_t)                    trajectory return               (Section 2.1)
 *     tau*  = argmax_i G(tau_i)                                        max-reward inference operator   (Section 2.1)
 *     V(q | s, u) = softmax(W_v h)_q,  E = sum_q q V(q)                value head and its mean         (Section 2.3)
 *
 * These entry points compute them for N trajectories at once.  Steps are 1-based in the formulas and 0-based in
 * memory.  Per-step arrays are step-major: element (t, n) lies at index t*N + n, so that consecutive trajectories
 * are consecutive in memory.  All pointers are DEVICE memory owned by the caller; every call is asynchronous on
 * `stream` (a cudaStream_t passed as void*), allocates nothing and does not synchronise.  Arithmetic is fp32.
 */
#ifndef MAXCODE_SEARCH_H_
#define MAXCODE_SEARCH_H_

#include <stddef.h>
#include <stdint.h>

#include "maxcode_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Rewards, best-so-far, value targets, labels and returns of N trajectories of at most T steps.
 *   speedup_pct  float [T][N]   speed-up of step t's candidate in percent (100 = as fast as the original)
 *   correct      uint8 [T][N]   non-zero: the candidate passed its tests
 *   len          int32 [N]      steps of trajectory n (1..T; values outside are clamped to [0, T]); NULL: all have T
 *   s1 < s2 < s3                class boundaries in percent, all above 100; 0 < gamma <= 1
 * Outputs (any may be NULL to skip it), for t < len[n]; entries with t >= len[n] are written as 0:
 *   reward       uint8 [T][N]   f_r(e_t) in 0..4
 *   best_so_far  float [T][N]   u_t
 *   value_target float [T][N]   v*_t
 *   label        uint8 [T][N]   lab_t in 0..4
 *   traj_return  float [N]      G (0 for an empty trajectory)
 * Returns MC_ERR_INVALID_ARG for null inputs, N < 1, T < 1, unordered boundaries or gamma outside (0, 1]. */
mc_status_t mc_search_returns(const float *speedup_pct, const uint8_t *correct, const int32_t *len, int32_t N, int32_t T,
                              float s1, float s2, float s3, float gamma, uint8_t *reward, float *best_so_far,
                              float *value_target, uint8_t *label, float *traj_return, void *stream);

/* Value head: logits float [N][5] (the classification head's output for the five reward classes) ->
 * prob float [N][5] (softmax; may be NULL) and expected float [N] (sum_q q * prob[q]). */
mc_status_t mc_search_value_head(const float *logits, int32_t N, float *prob, float *expected, void *stream);

/* For every group j (entries group_offsets[j] .. group_offsets[j+1]-1 of `values`, int32 [P+1], increasing) the index
 * of its largest value, the first one among equals, -1 for an empty group: best int32 [P].  With values = traj_return
 * this is tau*, with values = expected the state the guided search expands next.  NaN values are never selected. */
mc_status_t mc_search_group_argmax(const float *values, const int32_t *group_offsets, int32_t P, int32_t *best,
                                   void *stream);

/* mc_search_value_head and both uses of mc_search_group_argmax as ONE launch over groups (Section 2.3, "Generative
 * Value Function Guided Search": the state with the highest mean value is expanded; Section 2.1: tau* has the highest
 * return).  For every group j = entries group_offsets[j] .. group_offsets[j+1]-1:
 *   logits        float [N][5]  ->  prob float [N][5] (may be NULL), expected float [N] (may be NULL)
 *   best_expected int32 [P]     index of the group's largest mean (may be NULL)
 *   traj_return   float [N]     ->  best_return int32 [P]: index of the group's largest return (both NULL or both given)
 * Ties go to the smaller index, NaN is never selected, an empty group gives -1.  Entries outside every group are
 * not visited (their prob / expected are not written).  group_offsets int32 [P+1], increasing. */
mc_status_t mc_search_select(const float *logits, const float *traj_return, const int32_t *group_offsets, int32_t P,
                             float *prob, float *expected, int32_t *best_return, int32_t *best_expected, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* MAXCODE_SEARCH_H_ */
