"""CPU oracle for the max-reward search bookkeeping (test infrastructure, not a product path).

Plain fp64 restatements of the quantities the paper defines around its search loop; every function is the printed
definition written out with explicit loops (no scans, no recurrences), so that it can be checked against the paper
by eye.  Only `tests/`, the smoke check and the benchmark's CPU leg may import this module.

Notation follows the paper: a trajectory has steps t = 1..T with execution feedback e_t; f_r(e) is the categorical
reward; gamma in (0, 1] the discount; u_t the best discounted reward so far; v*_t the value target.
"""
from __future__ import annotations

from typing import Sequence, Tuple

import numpy as np


def categorical_reward(speedup_pct: float, correct: bool, s1: float, s2: float, s3: float) -> int:
    """f_r(e) of the "Categorical Reward Formulation" (Section 2.3): 0 if the speed-up is at most 100 % or the code
    is incorrect; 1, 2, 3 for the half-open-on-the-left intervals (100, s1], (s1, s2], (s2, s3]; 4 above s3.
    Speed-ups and thresholds are in percent, 100 < s1 < s2 < s3."""
    if not correct or speedup_pct <= 100.0:
        return 0
    if speedup_pct <= s1:
        return 1
    if speedup_pct <= s2:
        return 2
    if speedup_pct <= s3:
        return 3
    return 4


def raw_reward(speedup_pct: float, correct: bool) -> float:
    """f(e): the speed-up itself for a correct candidate, nothing for an incorrect one (reading: Section 2 says f
    returns higher values for better performance and that an incorrect candidate falls in the lowest class)."""
    return float(speedup_pct) if correct else 0.0


def best_so_far(r: Sequence[float], gamma: float) -> np.ndarray:
    """u_t = max_{k <= t} gamma^(k-1) r_k for t = 1..T (Section 2.3, data collection step 2)."""
    T = len(r)
    u = np.zeros(T, dtype=np.float64)
    for t in range(1, T + 1):
        u[t - 1] = max(gamma ** (k - 1) * float(r[k - 1]) for k in range(1, t + 1))
    return u


def future_best(r: Sequence[float], gamma: float) -> np.ndarray:
    """max_{k >= t} gamma^(k-t) r_k for t = 1..T: the best discounted reward still to come, step t included."""
    T = len(r)
    m = np.zeros(T, dtype=np.float64)
    for t in range(1, T + 1):
        m[t - 1] = max(gamma ** (k - t) * float(r[k - 1]) for k in range(t, T + 1))
    return m


def value_targets(r: Sequence[float], gamma: float) -> np.ndarray:
    """v*_t = max(u_t / gamma, max_{k >= t} gamma^(k-t) r_k) (Section 2.3, as printed)."""
    u, m = best_so_far(r, gamma), future_best(r, gamma)
    return np.maximum(u / gamma, m)


def trajectory_return(r: Sequence[float], gamma: float) -> float:
    """G(tau) = max_{t in [1, T]} gamma^(t-1) r_t (Section 2.1, the max-reward inference operator's objective)."""
    return max(gamma ** (t - 1) * float(r[t - 1]) for t in range(1, len(r) + 1))


def future_labels(speedup_pct: Sequence[float], correct: Sequence[bool], gamma: float, s1: float, s2: float,
                  s3: float) -> Tuple[np.ndarray, np.ndarray]:
    """Training label of the value model at every step: v* = f_r(max_{k >= t} gamma^(k-t) r_k) with r_k = f(e_k) the
    raw reward (Section 2.3, below the cross-entropy loss).  Returns (label[T] int, the discounted maximum[T])."""
    raw = [raw_reward(s, c) for s, c in zip(speedup_pct, correct)]
    m = future_best(raw, gamma)
    lab = np.array([categorical_reward(x, True, s1, s2, s3) for x in m], dtype=np.int64)
    return lab, m


def value_head(logits: Sequence[float]) -> Tuple[np.ndarray, float]:
    """V(q | s, u) = softmax(logits) over the five reward classes (Section 2.3) and its mean sum_q q V(q), the
    "expected estimated value" the guided search ranks states by."""
    z = np.asarray(logits, dtype=np.float64)
    e = np.exp(z - z.max())
    p = e / e.sum()
    return p, float(sum(q * p[q] for q in range(len(p))))


def group_argmax(values: Sequence[float], group_offsets: Sequence[int]) -> np.ndarray:
    """Index (within the whole array) of the largest value of every group; the first one among equals; -1 for an
    empty group.  With values = G(tau_i) this is tau* of Section 2.1, with values = expected value the state chosen
    for expansion in the guided search."""
    out = np.full(len(group_offsets) - 1, -1, dtype=np.int64)
    for j in range(len(group_offsets) - 1):
        best = None
        for i in range(group_offsets[j], group_offsets[j + 1]):
            if best is None or float(values[i]) > float(values[best]):
                best = i
        out[j] = -1 if best is None else best
    return out
