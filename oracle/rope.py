"""CPU oracle for the rotary position embedding applied to the appended key and the query of a decode step (test
infrastructure, not a product path; only `tests/`, the smoke check and the benchmark's CPU leg may import it).

The paper does not define this step: it belongs to the language model whose decode step the attention serves.  The
definition is the published one (rotary position embedding, Su et al., "RoFormer"): the d elements of a head are d/2
complex numbers, and the one at index i of a token at position `pos` is multiplied by exp(j * pos * theta_i) with
theta_i = base^(-2 i / d).  Pairing: element i is the real part and element i + d/2 the imaginary part ("rotate-half"
layout).  Everything is fp64; the product is written out with explicit real arithmetic.
"""
from __future__ import annotations

import math

import numpy as np


def rope_angles(pos: int, d: int, base: float) -> np.ndarray:
    """pos * theta_i for i = 0 .. d/2 - 1, theta_i = base^(-2 i / d)."""
    return np.array([pos * base ** (-2.0 * i / d) for i in range(d // 2)], dtype=np.float64)


def rope_rotate(x: np.ndarray, pos: int, base: float) -> np.ndarray:
    """Rotates one head row x[d] (any float dtype, computed in fp64) to position `pos`."""
    d = x.shape[-1]
    assert d % 2 == 0 and x.ndim == 1
    h = d // 2
    out = np.zeros(d, dtype=np.float64)
    for i in range(h):
        a = pos * base ** (-2.0 * i / d)
        re, im = float(x[i]), float(x[i + h])
        out[i] = re * math.cos(a) - im * math.sin(a)
        out[i + h] = re * math.sin(a) + im * math.cos(a)
    return out


def rope_rows(x: np.ndarray, pos: np.ndarray, base: float) -> np.ndarray:
    """x[B][H][d], pos[B]: every head row of candidate b rotated to position pos[b]."""
    B, H, _ = x.shape
    out = np.zeros(x.shape, dtype=np.float64)
    for b in range(B):
        for h in range(H):
            out[b, h] = rope_rotate(x[b, h], int(pos[b]), base)
    return out
