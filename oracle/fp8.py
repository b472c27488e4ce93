"""CPU oracle for the 8-bit floating-point (e4m3) KV cache with one scale per (page, kv head).  TEST INFRASTRUCTURE
ONLY: imported by tests, the smoke check and the benchmark's CPU leg; the library never calls it and shares no code
with it.

The paper takes the language model and its cache as given and defines none of this.  What is restated here is the
published format: the "E4M3" 8-bit floating-point encoding of Micikevicius et al., "FP8 Formats for Deep Learning"
(Section 3, Table 1) - one sign bit, four exponent bits with bias 7, three mantissa bits, no infinities, the single
NaN pattern S.1111.111, largest finite magnitude 448 - written out from that definition, value by value, in float64.

    code = s eeee mmm
    e = 0            value = (-1)^s * 2^-6 * (m / 8)                  subnormal (m = 0: zero)
    0 < e, not NaN   value = (-1)^s * 2^(e - 7) * (1 + m / 8)
    e = 15, m = 7    NaN

Encoding rounds to the nearest representable value, ties to the value whose mantissa code is even, and saturates:
every magnitude above 448 (and either infinity) becomes +-448; NaN becomes the NaN pattern.

A cache page holds 16 tokens.  For each (page, kv head) the cache stores 16 x d codes of K, 16 x d codes of V and
one float32 scale for each; the value a code stands for is decode(code) * scale.

Readings (nothing of this is fixed by the paper or by the format):
  * When is a page's scale fixed?  By the token that opens the page (slot 0), before the later rows are known:
    scale = 2 * max|row| / 448 for that token's row of the kv head (K and V separately), so a row twice as large as
    the first still fits; larger values saturate.  A first row of zeros gives scale 1.  The scale never changes
    afterwards, so the stored cache does not depend on how tokens were grouped into append calls.
  * Where is the quotient rounded?  x / scale is formed in float32 (one correctly rounded division) and that
    float32 number is encoded; the scale itself is (2 * amax) / 448 with the product exact and one correctly
    rounded float32 division.  The device takes the same decisions in the same precision, so codes and scales are
    compared bit for bit.
  * Attention over such a cache is attention over the values the codes stand for (float64 decode * float64(scale)):
    `dequantise` + oracle.attention.

Pins (tests/test_oracle_fp8_pins.py): the printed extremes of the format (448, 2^-6, 2^-9), all 256 codes against
torch.float8_e4m3fn as a library special case, encode(decode(c)) = c for every finite code, nearest-value brute force
over all 254 finite values on random and on exactly-halfway inputs, hand-listed ties, saturation, monotonicity and
symmetry, the error bound 2^-4 relative (2^-10 absolute below 2^-6), and the scale rule's guarantee that the opening
row never saturates.
"""
from __future__ import annotations

from typing import Tuple

import numpy as np

E4M3_MAX = 448.0
NAN_CODE = 0x7F
PAGE = 16
HEADROOM = 2.0


def e4m3_decode(code) -> np.ndarray:
    """uint8 codes -> float64 values, by the format's definition."""
    c = np.asarray(code, dtype=np.uint8).astype(np.int64)
    s = (c >> 7) & 1
    e = (c >> 3) & 0xF
    m = c & 0x7
    sub = 2.0 ** -6 * (m / 8.0)
    nor = 2.0 ** (e - 7.0) * (1.0 + m / 8.0)
    v = np.where(e == 0, sub, nor)
    v = np.where((e == 15) & (m == 7), np.nan, v)
    return np.where(s == 1, -v, v)


def e4m3_encode(x) -> np.ndarray:
    """float32 values -> uint8 codes: nearest representable value, ties to the even mantissa code, magnitudes above
    448 saturate to 448, NaN -> the NaN pattern.  The input is taken as float32 (that is the precision in which the
    decision is defined); the arithmetic below is exact in float64."""
    x = np.asarray(x, dtype=np.float32).astype(np.float64)
    nan = np.isnan(x)
    sign = np.where(np.signbit(x), 0x80, 0)
    a = np.minimum(np.abs(np.where(nan, 0.0, x)), E4M3_MAX)             # saturation of the input ...
    # the binade of a: representable values are spaced 2^(E - 3) apart, E = floor(log2 a) but at least -6
    # (frexp gives a = f * 2^k with 0.5 <= f < 1, so floor(log2 a) = k - 1, exactly)
    E = np.maximum(np.frexp(a)[1] - 1, -6)
    q = np.exp2(E - 3.0)
    n = np.rint(a / q)                                                   # round half to even; a / q is exact
    r = np.minimum(n * q, E4M3_MAX)                                      # ... and of the rounded value
    # code of the representable value r (n is even exactly when its mantissa code is even)
    Er = np.maximum(np.frexp(r)[1] - 1, -6)
    normal = r >= 2.0 ** -6
    code_sub = np.rint(r / 2.0 ** -9)                                    # subnormal: e = 0, m = r / 2^-9
    code_nor = (Er + 7) * 8 + np.rint((r / np.exp2(Er.astype(np.float64)) - 1.0) * 8.0)
    code = np.where(normal, code_nor, code_sub).astype(np.int64)
    return np.where(nan, NAN_CODE, sign | code).astype(np.uint8)


def page_scale(first_row) -> np.float32:
    """Scale of a (page, kv head) from the row of the token that opens the page: (2 * max|row|) / 448 in float32,
    1 when the row is all zeros."""
    amax = np.float32(np.max(np.abs(np.asarray(first_row, dtype=np.float32)))) if np.size(first_row) else np.float32(0)
    if not amax > 0:
        return np.float32(1.0)
    return np.float32(np.float32(amax * np.float32(HEADROOM)) / np.float32(E4M3_MAX))


def quantise_rows(rows, scale) -> np.ndarray:
    """rows [n][d] float32, one float32 scale -> codes [n][d]: encode(float32(row / scale))."""
    rows = np.asarray(rows, dtype=np.float32)
    return e4m3_encode(rows / np.float32(scale))


def dequantise(codes, scale) -> np.ndarray:
    """The values the codes stand for, float64."""
    return e4m3_decode(codes) * np.float64(np.float32(scale))


def quantise_sequence(tokens) -> Tuple[np.ndarray, np.ndarray]:
    """A whole sequence that starts on a page boundary, tokens [n][Hkv][d] float32 -> (codes [n][Hkv][d] uint8,
    scales [ceil(n / 16)][Hkv] float32): every page's scale from its first token's row, every row divided by its
    page's scale and encoded."""
    tokens = np.asarray(tokens, dtype=np.float32)
    n, Hkv, d = tokens.shape
    n_pages = (n + PAGE - 1) // PAGE
    codes = np.zeros((n, Hkv, d), dtype=np.uint8)
    scales = np.ones((n_pages, Hkv), dtype=np.float32)
    for pg in range(n_pages):
        lo, hi = pg * PAGE, min(n, (pg + 1) * PAGE)
        for h in range(Hkv):
            scales[pg, h] = page_scale(tokens[lo, h])
            codes[lo:hi, h] = quantise_rows(tokens[lo:hi, h], scales[pg, h])
    return codes, scales


def dequantise_sequence(codes, scales) -> np.ndarray:
    """(codes [n][Hkv][d], scales [pages][Hkv]) -> values [n][Hkv][d] float64."""
    codes = np.asarray(codes, dtype=np.uint8)
    n = codes.shape[0]
    per_token = np.asarray(scales, dtype=np.float32)[np.arange(n) // PAGE]          # [n][Hkv]
    return e4m3_decode(codes) * per_token[:, :, None].astype(np.float64)
