"""CPU oracle for shared-prefix grouped-query decode attention.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain definition that the CUDA library is checked against.  It is imported only
by tests, by the smoke check and by the benchmark's CPU-baseline leg; the library itself never calls it
and there is no CPU fallback.  It shares no code with the CUDA path.

What it computes.  The paper (Section 2.2, "Max-Reward Search"; Section 3.1, "Experimental Setup") fixes
only the workload shape: k candidates are sampled from one state, so they share one prompt.  The
operation itself is textbook scaled-dot-product attention of ONE query per candidate and query head
over that candidate's whole key/value history, which is the group's shared prefix followed by the
candidate's private suffix:

    K = concat(Kprefix[group(b)][:, h], Ksuffix[b][:, h])      n rows of d,  h = kv_head_of(hq)
    z_t = scale * sum_c q[b, hq, c] * K[t, c]
    lse = log sum_t exp(z_t)                                   natural log
    o   = sum_t exp(z_t - lse) * V[t]

All arithmetic is float64 on the unpaged, concatenated K/V.  The only numerical device is subtracting
max_t z_t before exponentiating (the definition of a stable softmax); there is no blocking, no online
update and no splitting in `attend`.  `merge_partials` is the definition of the log-sum-exp merge and
is the oracle for the library's merge step alone.

Pins (tests/test_oracle_pins.py): pure-Python brute force over every index on tiny inputs, closed
forms (one key; two keys; identical keys; constant V; dominant key), invariants (weights sum to one;
any split + merge equals the monolithic result; token / candidate permutations; key shift; MHA
expansion of the GQA map), a hand-computed fixture (tests/golden/two_key_softmax.txt) and PyTorch's
float64 scaled_dot_product_attention as a library special case.
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np


def attend(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float) -> Tuple[np.ndarray, float]:
    """Attention of one query over n key/value rows.

    q [d], K [n][d], V [n][dv]  ->  (o [dv] float64, lse float64).
    n == 0 gives o = 0 and lse = -inf (an empty history contributes nothing).
    """
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    n = K.shape[0]
    if n == 0:
        return np.zeros(V.shape[1] if V.ndim == 2 else q.shape[0], dtype=np.float64), -np.inf
    z = scale * (K @ q)                 # z_t = scale * <q, K_t>
    m = z.max()
    p = np.exp(z - m)                   # unnormalised weights, max one
    l = p.sum()
    o = (p @ V) / l                     # sum_t p_t V_t / sum_t p_t
    lse = m + np.log(l)
    return o, float(lse)


def attention_weights(q: np.ndarray, K: np.ndarray, scale: float) -> np.ndarray:
    """The softmax weights exp(z_t - lse) themselves, [n] float64."""
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    z = scale * (K @ q)
    m = z.max()
    p = np.exp(z - m)
    return p / p.sum()


def merge_partials(o_parts: np.ndarray, lse_parts: np.ndarray) -> Tuple[np.ndarray, float]:
    """Log-sum-exp merge of partial attention results over disjoint token sets.

    o_parts [n_parts][d], lse_parts [n_parts]  ->  (o [d], lse).
    m = max_i lse_i; w_i = exp(lse_i - m); o = sum_i w_i o_i / sum_i w_i; lse = m + log sum_i w_i.
    Parts with lse = -inf carry no tokens and are skipped; if every part is empty, o = 0, lse = -inf.
    """
    o_parts = np.asarray(o_parts, dtype=np.float64)
    lse_parts = np.asarray(lse_parts, dtype=np.float64)
    keep = lse_parts != -np.inf
    if not keep.any():
        return np.zeros(o_parts.shape[1], dtype=np.float64), -np.inf
    lp = lse_parts[keep]
    op = o_parts[keep]
    m = lp.max()
    w = np.exp(lp - m)
    s = w.sum()
    return (w @ op) / s, float(m + np.log(s))


def contiguous_kv_head(hq: int, Hq: int, Hkv: int) -> int:
    """Query heads [h*g, (h+1)*g) read kv head h, g = Hq / Hkv."""
    return hq // (Hq // Hkv)


def decode_attention(q: np.ndarray,
                     k_prefix: Sequence[np.ndarray], v_prefix: Sequence[np.ndarray],
                     k_suffix: Sequence[np.ndarray], v_suffix: Sequence[np.ndarray],
                     group_offsets: Sequence[int], scale: float,
                     kv_head_of: Optional[Callable[[int, int, int], int]] = None,
                     rows: Optional[Sequence[Tuple[int, int]]] = None,
                     ) -> Tuple[np.ndarray, np.ndarray]:
    """One decode step for every candidate b and query head hq.

    q          [B][Hq][d]
    k_prefix   per group j:      [P_j][Hkv][d]       (v_prefix likewise)
    k_suffix   per candidate b:  [s_b][Hkv][d]       (v_suffix likewise)
    group_offsets [G+1]: candidates group_offsets[j] .. group_offsets[j+1]-1 belong to group j.
    rows: optional list of (b, hq) to compute; others are left as NaN.
    Returns o [B][Hq][d] float64, lse [B][Hq] float64.
    """
    if kv_head_of is None:
        kv_head_of = contiguous_kv_head
    q = np.asarray(q)
    B, Hq, d = q.shape
    Hkv = (k_prefix[0] if len(k_prefix) else k_suffix[0]).shape[1]
    o = np.full((B, Hq, d), np.nan, dtype=np.float64)
    lse = np.full((B, Hq), np.nan, dtype=np.float64)
    group_of = np.zeros(B, dtype=np.int64)
    for j in range(len(group_offsets) - 1):
        group_of[group_offsets[j]:group_offsets[j + 1]] = j
    todo = rows if rows is not None else [(b, hq) for b in range(B) for hq in range(Hq)]
    for (b, hq) in todo:
        j = int(group_of[b])
        h = kv_head_of(hq, Hq, Hkv)
        K = np.concatenate([k_prefix[j][:, h, :], k_suffix[b][:, h, :]], axis=0).astype(np.float64)
        V = np.concatenate([v_prefix[j][:, h, :], v_suffix[b][:, h, :]], axis=0).astype(np.float64)
        o[b, hq], lse[b, hq] = attend(q[b, hq], K, V, scale)
    return o, lse


def token_range_partial(q_row: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float,
                        lo: int, hi: int) -> Tuple[np.ndarray, float]:
    """Partial result (o, lse) of one query over tokens [lo, hi) of its history: attention restricted to
    that slice.  This is what a prefix split or a suffix chunk must emit before the merge."""
    lo = max(0, lo)
    hi = max(lo, min(hi, K.shape[0]))
    return attend(q_row, K[lo:hi], V[lo:hi], scale)


def decode_attention_cascade(q: np.ndarray,
                             levels: Sequence[Tuple[Sequence[np.ndarray], Sequence[np.ndarray], Sequence[int]]],
                             k_suffix: Sequence[np.ndarray], v_suffix: Sequence[np.ndarray], scale: float,
                             kv_head_of: Optional[Callable[[int, int, int], int]] = None,
                             rows: Optional[Sequence[Tuple[int, int]]] = None) -> Tuple[np.ndarray, np.ndarray]:
    """One decode step when the shared history is a cascade of levels (a prefix tree deeper than two).

    levels: list of (k_list, v_list, group_offsets), outermost first; level i gives every candidate of its
    group j the rows k_list[j] [len][Hkv][d].  Candidate b's history is the concatenation of its group's rows at
    every level followed by its private suffix; the result is attention over that whole history (the order of
    concatenation does not matter).  With a single level this is `decode_attention`.
    """
    if kv_head_of is None:
        kv_head_of = contiguous_kv_head
    q = np.asarray(q)
    B, Hq, d = q.shape
    Hkv = k_suffix[0].shape[1]
    group_of = []
    for (_, _, go) in levels:
        g_of = np.zeros(B, dtype=np.int64)
        for j in range(len(go) - 1):
            g_of[go[j]:go[j + 1]] = j
        group_of.append(g_of)
    o = np.full((B, Hq, d), np.nan, dtype=np.float64)
    lse = np.full((B, Hq), np.nan, dtype=np.float64)
    todo = rows if rows is not None else [(b, hq) for b in range(B) for hq in range(Hq)]
    for (b, hq) in todo:
        h = kv_head_of(hq, Hq, Hkv)
        ks = [lv[0][int(group_of[i][b])][:, h, :] for i, lv in enumerate(levels)] + [k_suffix[b][:, h, :]]
        vs = [lv[1][int(group_of[i][b])][:, h, :] for i, lv in enumerate(levels)] + [v_suffix[b][:, h, :]]
        K = np.concatenate(ks, axis=0).astype(np.float64)
        V = np.concatenate(vs, axis=0).astype(np.float64)
        o[b, hq], lse[b, hq] = attend(q[b, hq], K, V, scale)
    return o, lse


def scoring_attention(q: Sequence[np.ndarray],
                      k_prefix: Sequence[np.ndarray], v_prefix: Sequence[np.ndarray],
                      k_seq: Sequence[np.ndarray], v_seq: Sequence[np.ndarray],
                      group_offsets: Sequence[int], scale: float,
                      kv_head_of: Optional[Callable[[int, int, int], int]] = None
                      ) -> Tuple[List[np.ndarray], List[np.ndarray]]:
    """Causal attention of whole sequences behind a shared prompt (scoring / prefill of candidates).

    Sequence b (in prompt group j) has n_b tokens with keys/values k_seq[b], v_seq[b] [n_b][Hkv][d] and one query
    per token, q[b] [n_b][Hq][d].  The query at position i attends to the group's whole prompt and to the
    sequence's own tokens 0..i (itself included):  K = concat(Kprefix_j, Kseq_b[0 : i+1]),  o = softmax(scale q K^T) V.
    This is `attend` applied row by row, nothing else.  Returns per sequence (o [n_b][Hq][d], lse [n_b][Hq]).
    """
    if kv_head_of is None:
        kv_head_of = contiguous_kv_head
    outs, lses = [], []
    for b in range(len(k_seq)):
        j = 0
        while not (group_offsets[j] <= b < group_offsets[j + 1]):
            j += 1
        n_b, Hq, d = np.asarray(q[b]).shape
        Hkv = k_seq[b].shape[1]
        o = np.zeros((n_b, Hq, d), dtype=np.float64)
        lse = np.zeros((n_b, Hq), dtype=np.float64)
        for i in range(n_b):
            for hq in range(Hq):
                h = kv_head_of(hq, Hq, Hkv)
                K = np.concatenate([k_prefix[j][:, h, :], k_seq[b][:i + 1, h, :]], axis=0).astype(np.float64)
                V = np.concatenate([v_prefix[j][:, h, :], v_seq[b][:i + 1, h, :]], axis=0).astype(np.float64)
                o[i, hq], lse[i, hq] = attend(q[b][i, hq], K, V, scale)
        outs.append(o)
        lses.append(lse)
    return outs, lses
