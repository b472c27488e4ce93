"""Pins of the rotary-embedding oracle against what the mathematics fixes: complex multiplication, the closed form for
d = 2, isometry, the relative-position property that motivates the construction, and composition of rotations."""
import cmath
import math

import numpy as np

from oracle import rope


def _row(seed, d):
    return np.random.default_rng(seed).standard_normal(d)


def test_is_multiplication_of_complex_pairs():
    d, base, pos = 16, 10000.0, 37
    x = _row(0, d)
    y = rope.rope_rotate(x, pos, base)
    for i in range(d // 2):
        z = complex(x[i], x[i + d // 2]) * cmath.exp(1j * pos * base ** (-2.0 * i / d))
        assert abs(y[i] - z.real) < 1e-12 and abs(y[i + d // 2] - z.imag) < 1e-12


def test_closed_form_d2_and_quarter_turn():
    # d = 2: one pair, theta_0 = 1, so position p rotates the plane by p radians
    y = rope.rope_rotate(np.array([1.0, 0.0]), 3, 10000.0)
    assert np.allclose(y, [math.cos(3.0), math.sin(3.0)], atol=1e-15)
    # base 1 makes every theta_i = 1; a row (a, b | c, d) at angle pi/2 ... use an angle through the position unit:
    # with base = 1 and pos = 1 every pair turns by exactly 1 radian
    x = np.array([2.0, -1.0, 0.5, 4.0])      # pairs (2, 0.5) and (-1, 4)
    y = rope.rope_rotate(x, 1, 1.0)
    c, s = math.cos(1.0), math.sin(1.0)
    assert np.allclose(y, [2 * c - 0.5 * s, -1 * c - 4 * s, 2 * s + 0.5 * c, -1 * s + 4 * c], atol=1e-15)


def test_position_zero_is_identity_and_norm_is_kept():
    x = _row(1, 128)
    assert np.array_equal(rope.rope_rotate(x, 0, 10000.0), x)
    for pos in (1, 17, 4095, 70000):
        y = rope.rope_rotate(x, pos, 10000.0)
        assert abs(np.linalg.norm(y) - np.linalg.norm(x)) < 1e-10
        h = 64
        for i in (0, 5, 63):   # each pair keeps its own length
            assert abs(math.hypot(y[i], y[i + h]) - math.hypot(x[i], x[i + h])) < 1e-10


def test_scores_depend_on_the_position_difference_only():
    d, base = 64, 10000.0
    q, k = _row(2, d), _row(3, d)
    ref = float(rope.rope_rotate(q, 9, base) @ k)          # query 9 positions after the key
    for n in (0, 1, 100, 5000):
        s = float(rope.rope_rotate(q, n + 9, base) @ rope.rope_rotate(k, n, base))
        assert abs(s - ref) < 1e-8
    # and a different distance gives a different score (the property is not vacuous)
    assert abs(float(rope.rope_rotate(q, 10, base) @ k) - ref) > 1e-3


def test_rotations_compose():
    x = _row(4, 32)
    a = rope.rope_rotate(rope.rope_rotate(x, 11, 500.0), 31, 500.0)
    assert np.allclose(a, rope.rope_rotate(x, 42, 500.0), atol=1e-12)


def test_angles_and_rows():
    ang = rope.rope_angles(7, 8, 10000.0)
    assert np.allclose(ang, [7.0, 0.7, 0.07, 0.007], rtol=1e-12)     # base^(-2i/8) = 10^-i
    x = np.random.default_rng(5).standard_normal((3, 2, 8))
    pos = np.array([0, 4, 9])
    y = rope.rope_rows(x, pos, 10000.0)
    assert np.array_equal(y[0], x[0])
    assert np.allclose(y[2, 1], rope.rope_rotate(x[2, 1], 9, 10000.0))
    # a planted mistake (the transposed rotation) is told apart
    wrong = rope.rope_rotate(x[1, 0], -4, 10000.0)
    assert not np.allclose(y[1, 0], wrong)
