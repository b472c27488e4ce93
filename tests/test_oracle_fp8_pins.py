"""Pins of the e4m3 KV-cache oracle (oracle/fp8.py) against things other than itself: the extremes the format's
definition prints (Micikevicius et al., "FP8 Formats for Deep Learning", Table 1: largest normal 448, smallest normal
2^-6, smallest subnormal 2^-9, NaN S.1111.111, no infinities), PyTorch's float8_e4m3fn as a library special case,
brute force over all finite values, hand-listed ties, and the guarantees of the page-scale rule."""
import math

import numpy as np
import pytest
import torch

from oracle import attention as orc
from oracle import fp8


def finite_codes():
    c = np.arange(256, dtype=np.uint8)
    return c[(c & 0x7F) != 0x7F]


def test_printed_extremes_of_the_format():
    d = fp8.e4m3_decode
    assert d(0b0_1111_110) == 448.0 and d(0b1_1111_110) == -448.0
    assert d(0b0_0001_000) == 2.0 ** -6
    assert d(0b0_0000_001) == 2.0 ** -9
    assert d(0b0_0000_111) == 0.875 * 2.0 ** -6          # largest subnormal
    assert d(0b0_0111_000) == 1.0 and d(0b0_0111_001) == 1.125 and d(0b0_1000_100) == 3.0
    assert d(0) == 0.0 and d(0x80) == 0.0 and math.copysign(1.0, float(d(0x80))) == -1.0
    assert np.isnan(d(0x7F)) and np.isnan(d(0xFF))
    assert np.isfinite(d(finite_codes())).all() and len(finite_codes()) == 254      # no infinities


def test_every_code_decodes_as_the_library_type_does():
    c = np.arange(256, dtype=np.uint8)
    lib = torch.from_numpy(c.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    ours = fp8.e4m3_decode(c)
    assert np.array_equal(np.isnan(lib), np.isnan(ours))
    ok = ~np.isnan(lib)
    assert np.array_equal(lib[ok], ours[ok]) and np.array_equal(np.signbit(lib[ok]), np.signbit(ours[ok]))


def test_finite_codes_survive_a_round_trip():
    c = finite_codes()
    assert np.array_equal(fp8.e4m3_encode(fp8.e4m3_decode(c).astype(np.float32)), c)


def nearest_by_brute_force(x):
    """Nearest of the 254 finite values by search; on a tie the value whose code is even; beyond +-448 that end."""
    c = finite_codes()
    vals = fp8.e4m3_decode(c)
    out = []
    for v in np.asarray(x, dtype=np.float64):
        dist = np.abs(vals - v)
        best = np.flatnonzero(dist == dist.min())
        best = [i for i in best if np.signbit(vals[i]) == np.signbit(v)] or list(best)      # +-0 by the sign of x
        if len(best) > 1:
            best = [i for i in best if c[i] % 2 == 0]
        out.append(c[best[0]])
    return np.array(out, dtype=np.uint8)


def test_encoding_is_the_nearest_value_with_ties_to_even():
    rng = np.random.default_rng(3)
    x = (rng.normal(size=3000) * np.exp(rng.uniform(-9, 6.5, size=3000))).astype(np.float32)
    assert np.array_equal(fp8.e4m3_encode(x), nearest_by_brute_force(x))
    # every midpoint between neighbouring values (exactly representable in float32), both signs
    vals = np.sort(fp8.e4m3_decode(finite_codes()[finite_codes() < 0x80]))
    mid = ((vals[:-1] + vals[1:]) / 2).astype(np.float32)
    for m in (mid, -mid):
        assert np.array_equal(fp8.e4m3_encode(m), nearest_by_brute_force(m))


def test_hand_listed_ties_and_saturation():
    e = lambda v: int(fp8.e4m3_encode(np.float32(v)))
    assert e(1.0625) == 0b0_0111_000           # between 1 (m = 0) and 1.125 (m = 1): the even one
    assert e(1.1875) == 0b0_0111_010           # between 1.125 (m = 1) and 1.25 (m = 2)
    assert e(2.0 ** -10) == 0                  # half the smallest subnormal: zero is even
    assert e(3 * 2.0 ** -10) == 2              # between 2^-9 (m = 1) and 2^-8 (m = 2)
    assert e(15 * 2.0 ** -10) == 0b0_0001_000  # between the largest subnormal (m = 7) and 2^-6 (e = 1, m = 0)
    assert e(448) == e(449) == e(464) == e(480) == e(1e30) == e(np.inf) == 0x7E
    assert e(-1e30) == e(-np.inf) == 0xFE
    assert e(np.nan) == 0x7F
    assert e(0.0) == 0 and e(-0.0) == 0x80


def test_encoding_agrees_with_the_library_cast_inside_the_finite_range():
    rng = np.random.default_rng(4)
    x = (rng.normal(size=200000) * np.exp(rng.uniform(-12, 6, size=200000))).astype(np.float32)
    x = x[np.abs(x) <= 448.0]
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(fp8.e4m3_encode(x), lib)


def test_encoding_is_monotone_odd_and_within_half_a_step():
    x = np.sort(np.random.default_rng(5).uniform(-500, 500, size=20000).astype(np.float32))
    v = fp8.e4m3_decode(fp8.e4m3_encode(x))
    assert (np.diff(v) >= 0).all()
    assert np.array_equal(fp8.e4m3_decode(fp8.e4m3_encode(-x)), -v)
    inside = np.abs(x) <= 448
    err = np.abs(v - x.astype(np.float64))[inside]
    bound = np.maximum(np.abs(x[inside].astype(np.float64)) * 2.0 ** -4, 2.0 ** -10)
    assert (err <= bound).all()


def test_page_scale_rule():
    rng = np.random.default_rng(6)
    for _ in range(50):
        row = rng.normal(size=128).astype(np.float32) * np.float32(rng.uniform(1e-3, 50))
        s = fp8.page_scale(row)
        assert s.dtype == np.float32 and s == np.float32(np.float32(2 * np.abs(row).max()) / np.float32(448))
        codes = fp8.quantise_rows(row[None], s)[0]
        # the opening row uses half the range: |value / scale| <= 224 (+ rounding), nothing saturates
        assert (codes & 0x7F).max() <= int(fp8.e4m3_encode(np.float32(224.5)))
        back = fp8.dequantise(codes, s)
        assert np.abs(back - row).max() <= np.abs(row).max() * 2.0 ** -4
        # a later row up to twice as large still fits, a larger one saturates at +-448 * scale
        assert np.abs(fp8.dequantise(fp8.quantise_rows(2 * row[None], s), s)).max() <= 448 * float(s) * (1 + 1e-7)
        big = fp8.dequantise(fp8.quantise_rows(5 * row[None], s), s)[0]
        assert np.abs(big).max() == pytest.approx(448 * float(s))
    assert fp8.page_scale(np.zeros(64, dtype=np.float32)) == np.float32(1)


def test_sequence_quantisation_is_page_by_page_and_independent_of_batching():
    rng = np.random.default_rng(7)
    tok = rng.normal(size=(41, 2, 8)).astype(np.float32)
    tok[17] *= 9                                             # a row far above its page's opening row: saturates
    codes, scales = fp8.quantise_sequence(tok)
    assert codes.shape == (41, 2, 8) and scales.shape == (3, 2)
    for pg in range(3):
        for h in range(2):
            assert scales[pg, h] == fp8.page_scale(tok[16 * pg, h])
            assert np.array_equal(codes[16 * pg:16 * pg + 16, h], fp8.quantise_rows(tok[16 * pg:16 * pg + 16, h], scales[pg, h]))
    # token by token (what successive one-token appends do) gives the same cache
    for t in range(41):
        for h in range(2):
            assert np.array_equal(codes[t, h], fp8.quantise_rows(tok[t:t + 1, h], scales[t // 16, h])[0])
    vals = fp8.dequantise_sequence(codes, scales)
    assert np.array_equal(vals[20, 1], fp8.e4m3_decode(codes[20, 1]) * np.float64(scales[1, 1]))
    assert np.abs(vals[17]).max() == pytest.approx(448 * float(scales[1].max()), rel=0.5)     # clipped, not 9 x


def test_attention_over_the_cache_is_attention_over_the_decoded_values():
    rng = np.random.default_rng(8)
    K, V = rng.normal(size=(50, 1, 16)).astype(np.float32), rng.normal(size=(50, 1, 16)).astype(np.float32)
    q = rng.normal(size=16)
    (kc, ks), (vc, vs) = fp8.quantise_sequence(K), fp8.quantise_sequence(V)
    Kd, Vd = fp8.dequantise_sequence(kc, ks)[:, 0], fp8.dequantise_sequence(vc, vs)[:, 0]
    o, lse = orc.attend(q, Kd, Vd, 0.25)
    # the same through the format's definition, value by value, without the helpers
    z = np.array([0.25 * sum(q[c] * float(fp8.e4m3_decode(kc[t, 0, c])) * float(ks[t // 16, 0]) for c in range(16))
                  for t in range(50)])
    w = np.exp(z - z.max())
    assert lse == pytest.approx(z.max() + math.log(w.sum()), abs=1e-12)
    o2 = sum(w[t] / w.sum() * fp8.e4m3_decode(vc[t, 0]) * float(vs[t // 16, 0]) for t in range(50))
    assert np.abs(o - o2).max() <= 1e-12
    # quantisation error of the inputs is what the format allows (relative 2^-4 per element that fits its page's
    # range, plus half a subnormal step), not more; elements beyond the range sit at its end
    per_tok = ks[np.arange(50) // 16, 0][:, None].astype(np.float64)
    fits = np.abs(K[:, 0]) <= 448 * per_tok
    assert (np.abs(Kd - K[:, 0])[fits] <= (np.abs(K[:, 0]) * 2.0 ** -4 + 2.0 ** -10 * per_tok)[fits] * (1 + 1e-6)).all()
    assert np.allclose(np.abs(Kd)[~fits], np.broadcast_to(448 * per_tok, Kd.shape)[~fits])
