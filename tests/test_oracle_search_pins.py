"""Pins of the search-bookkeeping oracle (oracle/search.py) against what the paper's formulas and plain mathematics
fix: a hand-computed fixture, closed forms for gamma = 1, library routines, invariants and brute force."""
import math
import os

import numpy as np
import pytest

from oracle import search as orc

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "max_reward_bookkeeping.txt")
SPEEDUP = [110.0, 400.0, 350.0, 90.0]
CORRECT = [True, False, True, True]
S = (120.0, 200.0, 300.0)


def golden_rows():
    rows = []
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            v = [float(x) for x in line.split()]
            rows.append((v[0], v[1:5], v[5:9], v[9:13], v[13], v[14:18]))
    return rows


@pytest.mark.parametrize("row", golden_rows())
def test_hand_computed_fixture(row):
    gamma, r, u, v, G, labels = row
    got_r = [orc.categorical_reward(s, c, *S) for s, c in zip(SPEEDUP, CORRECT)]
    assert got_r == [int(x) for x in r]
    np.testing.assert_allclose(orc.best_so_far(got_r, gamma), u, rtol=0, atol=1e-15)
    np.testing.assert_allclose(orc.value_targets(got_r, gamma), v, rtol=0, atol=1e-15)
    assert orc.trajectory_return(got_r, gamma) == G
    lab, _ = orc.future_labels(SPEEDUP, CORRECT, gamma, *S)
    assert lab.tolist() == [int(x) for x in labels]


def test_value_head_fixture_and_properties():
    p, ev = orc.value_head([0.0, math.log(2.0), 0.0, math.log(4.0), 0.0])
    np.testing.assert_allclose(p, np.array([1, 2, 1, 4, 1]) / 9.0, atol=1e-15)
    assert abs(ev - 20.0 / 9.0) < 1e-15
    rng = np.random.default_rng(0)
    for _ in range(20):
        z = rng.normal(size=5) * 5
        p, ev = orc.value_head(z)
        assert abs(p.sum() - 1.0) < 1e-14 and (p >= 0).all()
        p2, ev2 = orc.value_head(z + 123.0)                    # shift invariance
        np.testing.assert_allclose(p, p2, atol=1e-13)
        assert 0.0 <= ev <= 4.0
    p, ev = orc.value_head([-1e3, -1e3, 1e3, -1e3, -1e3])     # one dominant class
    assert abs(ev - 2.0) < 1e-12
    p, ev = orc.value_head([7.0] * 5)                          # uniform: mean of 0..4
    assert abs(ev - 2.0) < 1e-14


def test_bin_edges_are_closed_on_the_right():
    s1, s2, s3 = S
    f = lambda x, c=True: orc.categorical_reward(x, c, s1, s2, s3)
    assert [f(100.0), f(np.nextafter(100.0, 200.0)), f(s1), f(np.nextafter(s1, 1e9)), f(s2), f(np.nextafter(s2, 1e9)),
            f(s3), f(np.nextafter(s3, 1e9)), f(1e9), f(0.0), f(-5.0)] == [0, 1, 1, 2, 2, 3, 3, 4, 4, 0, 0]
    assert f(1e9, False) == 0 and f(150.0, False) == 0


def test_gamma_one_closed_forms_and_library_routines():
    rng = np.random.default_rng(1)
    for _ in range(50):
        T = int(rng.integers(1, 12))
        r = rng.integers(0, 5, size=T)
        u = orc.best_so_far(r, 1.0)
        np.testing.assert_array_equal(u, np.maximum.accumulate(r))                     # running maximum
        m = orc.future_best(r, 1.0)
        np.testing.assert_array_equal(m, np.maximum.accumulate(r[::-1])[::-1])         # reversed running maximum
        np.testing.assert_array_equal(orc.value_targets(r, 1.0), np.full(T, r.max()))  # max(before, after) = overall max
        assert orc.trajectory_return(r, 1.0) == r.max() == u[-1]


def test_discount_invariants():
    rng = np.random.default_rng(2)
    for _ in range(50):
        T = int(rng.integers(1, 12))
        r = rng.integers(0, 5, size=T).astype(float)
        g = float(rng.uniform(0.3, 1.0))
        u, m, v = orc.best_so_far(r, g), orc.future_best(r, g), orc.value_targets(r, g)
        assert (np.diff(u) >= 0).all() and u[0] == r[0]                 # best so far never decreases
        assert abs(u[-1] - orc.trajectory_return(r, g)) < 1e-15          # G = the last best-so-far
        for t in range(T - 1):                                           # one-step recurrences of the definitions
            assert abs(m[t] - max(r[t], g * m[t + 1])) < 1e-12
            assert abs(u[t + 1] - max(u[t], g ** (t + 1) * r[t + 1])) < 1e-12
        assert m[-1] == r[-1]
        assert (v >= m - 1e-15).all() and (v >= u / g - 1e-15).all()
        np.testing.assert_allclose(orc.best_so_far(3.0 * r, g), 3.0 * u, rtol=1e-14)   # positive homogeneity
        # a discounted maximum equals the plain maximum of explicitly discounted copies
        for t in range(T):
            assert abs(m[t] - np.max(r[t:] * g ** np.arange(T - t))) < 1e-12


def test_labels_with_gamma_one_are_the_largest_future_class():
    """f_r is monotone in the speed-up, so binning the largest future raw reward gives the largest future class."""
    rng = np.random.default_rng(3)
    for _ in range(50):
        T = int(rng.integers(1, 10))
        sp = rng.uniform(50, 400, size=T)
        ok = rng.random(T) < 0.7
        lab, _ = orc.future_labels(sp, ok, 1.0, *S)
        r = np.array([orc.categorical_reward(s, c, *S) for s, c in zip(sp, ok)])
        np.testing.assert_array_equal(lab, np.maximum.accumulate(r[::-1])[::-1])


def test_group_argmax_against_numpy_and_ties():
    rng = np.random.default_rng(4)
    vals = rng.normal(size=40)
    go = [0, 7, 7, 19, 40]
    got = orc.group_argmax(vals, go)
    assert got[1] == -1
    for j in (0, 2, 3):
        assert got[j] == go[j] + int(np.argmax(vals[go[j]:go[j + 1]]))
    assert orc.group_argmax([1.0, 3.0, 3.0, 2.0], [0, 4]).tolist() == [1]      # first among equals
