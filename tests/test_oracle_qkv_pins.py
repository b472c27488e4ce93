"""Pins of the projection oracle (oracle/qkv.py) against things other than itself: explicit loops with exact
summation, unit vectors and selector matrices whose result can be read off, a library linear layer, linearity, and
the head order written out by hand."""
import math

import numpy as np
import torch

from oracle import qkv
from oracle import rope


def test_product_is_the_sum_written_out():
    rng = np.random.default_rng(0)
    x, w, b = rng.standard_normal((3, 7)), rng.standard_normal((12, 7)), rng.standard_normal(12)
    y = qkv.project(x, w, b)
    for r in range(3):
        for n in range(12):
            ref = math.fsum(float(x[r, i]) * float(w[n, i]) for i in range(7)) + float(b[n])
            assert abs(y[r, n] - ref) <= 1e-13
    # a transposed weight matrix or a bias added per row instead of per feature would not survive these shapes
    assert y.shape == (3, 12)
    assert np.allclose(qkv.project(x, w), y - b[None, :], atol=1e-13)


def test_unit_inputs_read_off_columns_and_rows():
    rng = np.random.default_rng(1)
    w = rng.standard_normal((8, 5))
    for i in range(5):                       # x = e_i picks column i of W: y[n] = W[n, i]
        e = np.zeros((1, 5))
        e[0, i] = 1.0
        assert np.array_equal(qkv.project(e, w)[0], w[:, i])
    x = rng.standard_normal((4, 5))          # W = a selector: feature n copies input n
    sel = np.eye(5)[[4, 0, 2]]
    assert np.array_equal(qkv.project(x, sel), x[:, [4, 0, 2]])


def test_agrees_with_a_library_linear_layer():
    rng = np.random.default_rng(2)
    x, w, b = rng.standard_normal((6, 33)), rng.standard_normal((20, 33)), rng.standard_normal(20)
    lib = torch.nn.functional.linear(torch.from_numpy(x), torch.from_numpy(w), torch.from_numpy(b)).numpy()
    assert np.abs(qkv.project(x, w, b) - lib).max() <= 1e-12


def test_linearity():
    rng = np.random.default_rng(3)
    x1, x2, w = rng.standard_normal((2, 9)), rng.standard_normal((2, 9)), rng.standard_normal((6, 9))
    assert np.allclose(qkv.project(2.5 * x1 - x2, w), 2.5 * qkv.project(x1, w) - qkv.project(x2, w), atol=1e-12)


def test_head_order_by_hand():
    Hq, Hkv, d = 4, 2, 2
    y = np.arange(2 * (Hq + 2 * Hkv) * d, dtype=np.float64).reshape(2, -1)      # features 0..15 and 16..31
    q, k, v = qkv.split_heads(y, Hq, Hkv, d)
    assert q.shape == (2, 4, 2) and k.shape == (2, 2, 2) and v.shape == (2, 2, 2)
    assert q[0].tolist() == [[0, 1], [2, 3], [4, 5], [6, 7]]
    assert k[0].tolist() == [[8, 9], [10, 11]]
    assert v[0].tolist() == [[12, 13], [14, 15]]
    assert q[1, 3].tolist() == [22, 23] and k[1, 0].tolist() == [24, 25] and v[1, 1].tolist() == [30, 31]


def test_step_rotates_queries_and_keys_but_not_values():
    rng = np.random.default_rng(4)
    Hq, Hkv, d, hidden, B = 4, 2, 8, 16, 3
    x, w = rng.standard_normal((B, hidden)), rng.standard_normal(((Hq + 2 * Hkv) * d, hidden))
    bias = rng.standard_normal((Hq + 2 * Hkv) * d)
    pos = np.array([0, 5, 1234])
    q, k, v = qkv.qkv_step(x, w, bias, pos, 10000.0, Hq, Hkv, d)
    y = x @ w.T + bias
    # position 0 leaves q and k as projected
    assert np.allclose(q[0].ravel(), y[0, :Hq * d], atol=1e-13) and np.allclose(k[0].ravel(), y[0, Hq * d:(Hq + Hkv) * d], atol=1e-13)
    # the values never turn
    assert np.allclose(v.reshape(B, -1), y[:, (Hq + Hkv) * d:], atol=1e-13)
    # a rotated pair, by the closed form: (re, im) -> (re cos a - im sin a, re sin a + im cos a), a = pos * base^(-2i/d)
    b, h, i = 2, 1, 3
    re, im = y[b, (Hq + h) * d + i], y[b, (Hq + h) * d + i + d // 2]
    a = 1234 * 10000.0 ** (-2.0 * i / d)
    assert abs(k[b, h, i] - (re * math.cos(a) - im * math.sin(a))) <= 1e-10
    assert abs(k[b, h, i + d // 2] - (re * math.sin(a) + im * math.cos(a))) <= 1e-10
    # rotation keeps each head's norm; the scores it exists for depend on the distance of positions only
    assert np.allclose(np.linalg.norm(q, axis=-1), np.linalg.norm(y[:, :Hq * d].reshape(B, Hq, d), axis=-1), atol=1e-10)
    q2, k2, _ = qkv.qkv_step(x, w, bias, pos + 77, 10000.0, Hq, Hkv, d)
    assert abs(float(q[1, 0] @ k[2, 0]) - float(q2[1, 0] @ k2[2, 0])) <= 1e-9
    # no rotation asked for
    q0, k0, _ = qkv.qkv_step(x, w, bias, pos, 0.0, Hq, Hkv, d)
    assert np.allclose(q0.reshape(B, -1), y[:, :Hq * d], atol=1e-13)
    assert np.array_equal(rope.rope_rows(q0, pos, 10000.0), q)


def test_abs_dot_bounds_the_product():
    rng = np.random.default_rng(5)
    x, w = rng.standard_normal((4, 50)), rng.standard_normal((9, 50))
    a = qkv.abs_dot(x, w)
    assert (a >= np.abs(qkv.project(x, w)) - 1e-12).all()
    assert abs(a[2, 3] - math.fsum(abs(float(x[2, i])) * abs(float(w[3, i])) for i in range(50))) <= 1e-12
