"""CPU oracle for the query/key/value projection of a decode step, taken together with the rotary embedding and the
append that follow it (test infrastructure, not a product path; only `tests/`, the smoke check and the benchmark's CPU
leg may import it).

The paper does not define this step: it belongs to the language model whose decode step the attention serves, and
the paper takes that model as given.  The definition is the usual one of a grouped-query attention layer: for the
hidden state x[b] (one row per candidate) and a weight matrix W with one row per output feature,

    y[b] = W x[b] (+ bias)         N = (Hq + 2 Hkv) d output features
    q[b, h]  = y[b, h d : (h+1) d]                              h < Hq
    k[b, h]  = y[b, (Hq + h) d : (Hq + h + 1) d]                h < Hkv
    v[b, h]  = y[b, (Hq + Hkv + h) d : (Hq + Hkv + h + 1) d]    h < Hkv

after which q and k are rotated to the new token's position (oracle/rope.py) and k, v become the token the
candidate's suffix grows by.  Everything is fp64; the product is numpy's matmul on fp64 operands.
"""
from __future__ import annotations

from typing import Optional, Tuple

import numpy as np

from . import rope


def project(x: np.ndarray, w: np.ndarray, bias: Optional[np.ndarray] = None) -> np.ndarray:
    """y[B][N] = x[B][hidden] W^T (+ bias), W[N][hidden]."""
    y = np.asarray(x, dtype=np.float64) @ np.asarray(w, dtype=np.float64).T
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)[None, :]
    return y


def split_heads(y: np.ndarray, Hq: int, Hkv: int, d: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """y[B][(Hq + 2 Hkv) d] -> q[B][Hq][d], k[B][Hkv][d], v[B][Hkv][d]: query heads first, then key heads, then value
    heads, each head d consecutive features."""
    B = y.shape[0]
    assert y.shape[1] == (Hq + 2 * Hkv) * d
    q = y[:, :Hq * d].reshape(B, Hq, d)
    k = y[:, Hq * d:(Hq + Hkv) * d].reshape(B, Hkv, d)
    v = y[:, (Hq + Hkv) * d:].reshape(B, Hkv, d)
    return q, k, v


def qkv_step(x: np.ndarray, w: np.ndarray, bias: Optional[np.ndarray], pos: np.ndarray, base: float,
             Hq: int, Hkv: int, d: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """The projection followed by the rotation of q and k to position pos[b] (base <= 0: no rotation).  Returns
    q[B][Hq][d], k[B][Hkv][d], v[B][Hkv][d] in fp64: the query of the decode step and the token to append."""
    q, k, v = split_heads(project(x, w, bias), Hq, Hkv, d)
    if base > 0:
        q, k = rope.rope_rows(q, pos, base), rope.rope_rows(k, pos, base)
    return q, k, v.copy()


def abs_dot(x: np.ndarray, w: np.ndarray) -> np.ndarray:
    """sum_i |x[b, i]| |W[n, i]| for every (b, n): the quantity a forward error bound of the product scales with."""
    return np.abs(np.asarray(x, dtype=np.float64)) @ np.abs(np.asarray(w, dtype=np.float64)).T
