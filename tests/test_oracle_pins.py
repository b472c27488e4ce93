"""Pins for the CPU oracle: everything here is checked against mathematics, not against the oracle itself.

Brute force (pure-Python loops over every index, no numpy arithmetic), closed forms, invariants, a
hand-computed fixture and PyTorch's float64 scaled_dot_product_attention as a library special case.
"""
import math
import os

import numpy as np
import pytest

from oracle import attention as orc

HERE = os.path.dirname(os.path.abspath(__file__))


# ---------------------------------------------------------------------------------------------------
# brute force: explicit loops, direct sum of exponentials without max subtraction (small |z| only)
# ---------------------------------------------------------------------------------------------------
def brute_force_decode(q, k_prefix, v_prefix, k_suffix, v_suffix, group_offsets, scale):
    B, Hq, d = len(q), len(q[0]), len(q[0][0])
    Hkv = len(k_prefix[0][0]) if len(k_prefix[0]) else len(k_suffix[0][0])
    g = Hq // Hkv
    out_o = [[[0.0] * d for _ in range(Hq)] for _ in range(B)]
    out_lse = [[0.0] * Hq for _ in range(B)]
    for b in range(B):
        j = None
        for jj in range(len(group_offsets) - 1):
            if group_offsets[jj] <= b < group_offsets[jj + 1]:
                j = jj
        for hq in range(Hq):
            h = hq // g
            keys, vals = [], []
            for t in range(len(k_prefix[j])):
                keys.append(k_prefix[j][t][h])
                vals.append(v_prefix[j][t][h])
            for t in range(len(k_suffix[b])):
                keys.append(k_suffix[b][t][h])
                vals.append(v_suffix[b][t][h])
            e = []
            for t in range(len(keys)):
                dot = math.fsum(q[b][hq][c] * keys[t][c] for c in range(d))
                e.append(math.exp(scale * dot))
            denom = math.fsum(e)
            out_lse[b][hq] = math.log(denom)
            for c in range(d):
                out_o[b][hq][c] = math.fsum(e[t] * vals[t][c] for t in range(len(keys))) / denom
    return out_o, out_lse


def _tiny_problem(seed, G=2, C=2, Hq=4, Hkv=2, d=6, P=(5, 9), S=(0, 3, 7, 1)):
    rng = np.random.default_rng(seed)
    B = G * C
    q = rng.normal(size=(B, Hq, d))
    kp = [rng.normal(size=(P[j], Hkv, d)) for j in range(G)]
    vp = [rng.normal(size=(P[j], Hkv, d)) for j in range(G)]
    ks = [rng.normal(size=(S[b], Hkv, d)) for b in range(B)]
    vs = [rng.normal(size=(S[b], Hkv, d)) for b in range(B)]
    go = [j * C for j in range(G + 1)]
    return q, kp, vp, ks, vs, go


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_brute_force_tiny(seed):
    q, kp, vp, ks, vs, go = _tiny_problem(seed)
    scale = 0.37
    o, lse = orc.decode_attention(q, kp, vp, ks, vs, go, scale)
    bo, blse = brute_force_decode(q.tolist(), [x.tolist() for x in kp], [x.tolist() for x in vp],
                                  [x.tolist() for x in ks], [x.tolist() for x in vs], go, scale)
    np.testing.assert_allclose(o, np.array(bo), rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, np.array(blse), rtol=0, atol=1e-12)


def test_brute_force_unequal_groups_and_mqa():
    # groups of unequal size (3 and 1 candidates), a single kv head
    rng = np.random.default_rng(7)
    Hq, Hkv, d = 3, 1, 4
    q = rng.normal(size=(4, Hq, d))
    kp = [rng.normal(size=(4, Hkv, d)), rng.normal(size=(2, Hkv, d))]
    vp = [rng.normal(size=(4, Hkv, d)), rng.normal(size=(2, Hkv, d))]
    ks = [rng.normal(size=(n, Hkv, d)) for n in (2, 0, 5, 1)]
    vs = [rng.normal(size=(n, Hkv, d)) for n in (2, 0, 5, 1)]
    go = [0, 3, 4]
    o, lse = orc.decode_attention(q, kp, vp, ks, vs, go, 0.5)
    bo, blse = brute_force_decode(q.tolist(), [x.tolist() for x in kp], [x.tolist() for x in vp],
                                  [x.tolist() for x in ks], [x.tolist() for x in vs], go, 0.5)
    np.testing.assert_allclose(o, np.array(bo), atol=1e-12)
    np.testing.assert_allclose(lse, np.array(blse), atol=1e-12)


# ---------------------------------------------------------------------------------------------------
# hand-computed fixture
# ---------------------------------------------------------------------------------------------------
def test_golden_two_key_fixture():
    rows = {}
    with open(os.path.join(HERE, "golden", "two_key_softmax.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            c, lse, o0, o1 = line.split()
            rows[int(c)] = (float(lse), float(o0), float(o1))
    K = np.array([[1.0, 5.0], [0.0, -2.0]])
    V = np.array([[4.0, 8.0], [0.0, -4.0]])
    o, lse = orc.attend(np.array([math.log(3.0), 0.0]), K, V, 1.0)
    assert abs(lse - rows[1][0]) < 1e-14 and np.allclose(o, rows[1][1:], atol=1e-14)
    o, lse = orc.attend(np.array([math.log(3.0) / 2, 0.0]), K, V, 2.0)
    assert abs(lse - rows[2][0]) < 1e-14 and np.allclose(o, rows[2][1:], atol=1e-14)
    K3 = np.array([[math.log(2.0), 0, 0], [0, math.log(3.0), 0], [0, 0, math.log(5.0)]])
    V3 = np.array([[10.0, 0.0], [0.0, 10.0], [10.0, 10.0]])
    o, lse = orc.attend(np.ones(3), K3, V3, 1.0)
    assert abs(lse - rows[3][0]) < 1e-14 and np.allclose(o, rows[3][1:], atol=1e-13)


# ---------------------------------------------------------------------------------------------------
# closed forms
# ---------------------------------------------------------------------------------------------------
def test_single_key_returns_its_value_row():
    rng = np.random.default_rng(0)
    q, k, v = rng.normal(size=8), rng.normal(size=(1, 8)), rng.normal(size=(1, 8))
    o, lse = orc.attend(q, k, v, 0.25)
    np.testing.assert_allclose(o, v[0], atol=1e-15)
    assert abs(lse - 0.25 * float(q @ k[0])) < 1e-14


def test_identical_keys_give_mean_of_v():
    rng = np.random.default_rng(1)
    n, d = 37, 8
    q, k = rng.normal(size=d), rng.normal(size=d)
    K = np.tile(k, (n, 1))
    V = rng.normal(size=(n, d))
    o, lse = orc.attend(q, K, V, 0.3)
    np.testing.assert_allclose(o, V.mean(axis=0), atol=1e-14)
    assert abs(lse - (math.log(n) + 0.3 * float(q @ k))) < 1e-13
    # q = 0 is the same closed form with z = 0
    o, lse = orc.attend(np.zeros(d), rng.normal(size=(n, d)), V, 0.3)
    np.testing.assert_allclose(o, V.mean(axis=0), atol=1e-14)
    assert abs(lse - math.log(n)) < 1e-14
    # scale -> 0 likewise
    o, _ = orc.attend(q, rng.normal(size=(n, d)), V, 0.0)
    np.testing.assert_allclose(o, V.mean(axis=0), atol=1e-14)


def test_two_keys_sigmoid_mix():
    rng = np.random.default_rng(2)
    q, K, V = rng.normal(size=5), rng.normal(size=(2, 5)), rng.normal(size=(2, 5))
    z = 0.7 * (K @ q)
    s = 1.0 / (1.0 + math.exp(-(z[0] - z[1])))
    o, _ = orc.attend(q, K, V, 0.7)
    np.testing.assert_allclose(o, s * V[0] + (1 - s) * V[1], atol=1e-14)


def test_dominant_key_and_large_scores_are_stable():
    rng = np.random.default_rng(3)
    d, n = 4, 20
    q = np.array([1.0, 0, 0, 0])
    K = rng.normal(size=(n, d)) * 0.1
    K[11, 0] = 1000.0                      # z = 1000 would overflow a naive exp
    V = rng.normal(size=(n, d))
    o, lse = orc.attend(q, K, V, 1.0)
    np.testing.assert_allclose(o, V[11], atol=1e-20)
    assert abs(lse - 1000.0) < 1e-9
    # hugely negative scores must not underflow to 0/0
    o, lse = orc.attend(q, -1000.0 - 1000.0 * np.abs(rng.normal(size=(n, d))), V, 1.0)
    assert np.isfinite(o).all() and np.isfinite(lse)


def test_constant_v_is_returned_for_any_keys():
    rng = np.random.default_rng(4)
    v = rng.normal(size=6)
    o, _ = orc.attend(rng.normal(size=6), rng.normal(size=(50, 6)) * 3, np.tile(v, (50, 1)), 1.0)
    np.testing.assert_allclose(o, v, atol=1e-14)


def test_empty_history():
    o, lse = orc.attend(np.ones(4), np.zeros((0, 4)), np.zeros((0, 4)), 1.0)
    assert lse == -np.inf and (o == 0).all()
    o, lse = orc.merge_partials(np.ones((3, 4)), np.full(3, -np.inf))
    assert lse == -np.inf and (o == 0).all()


# ---------------------------------------------------------------------------------------------------
# invariants
# ---------------------------------------------------------------------------------------------------
def test_weights_sum_to_one_and_reproduce_o():
    rng = np.random.default_rng(5)
    q, K, V = rng.normal(size=16), rng.normal(size=(300, 16)) * 2, rng.normal(size=(300, 16))
    w = orc.attention_weights(q, K, 0.25)
    assert abs(w.sum() - 1.0) < 1e-12 and (w >= 0).all()
    o, lse = orc.attend(q, K, V, 0.25)
    np.testing.assert_allclose(o, w @ V, atol=1e-13)
    # exp(z_t - lse) are the weights
    np.testing.assert_allclose(np.exp(0.25 * (K @ q) - lse), w, atol=1e-14)


@pytest.mark.parametrize("cuts", [[0], [1], [13], [40], [0, 0, 17], [5, 5, 20, 39], list(range(0, 41, 3))])
def test_split_plus_merge_equals_monolithic(cuts):
    rng = np.random.default_rng(6)
    n, d = 40, 8
    q, K, V = rng.normal(size=d), rng.normal(size=(n, d)) * 3, rng.normal(size=(n, d))
    o, lse = orc.attend(q, K, V, 0.5)
    edges = [0] + sorted(cuts) + [n]
    parts = [orc.token_range_partial(q, K, V, 0.5, edges[i], edges[i + 1]) for i in range(len(edges) - 1)]
    om, lm = orc.merge_partials(np.stack([p[0] for p in parts]), np.array([p[1] for p in parts]))
    np.testing.assert_allclose(om, o, atol=1e-13)
    assert abs(lm - lse) < 1e-13


def test_merge_against_direct_weighted_sum():
    # merge written out directly: o = sum_i exp(lse_i) o_i / sum_i exp(lse_i) for small lse
    rng = np.random.default_rng(8)
    op, lp = rng.normal(size=(5, 3)), rng.normal(size=5)
    lp[2] = -np.inf
    w = [math.exp(x) if x != -np.inf else 0.0 for x in lp]
    expect = sum(w[i] * op[i] for i in range(5)) / sum(w)
    o, lse = orc.merge_partials(op, lp)
    np.testing.assert_allclose(o, expect, atol=1e-14)
    assert abs(lse - math.log(sum(w))) < 1e-14
    # a NaN-filled o row of an empty part must not leak
    op[2] = np.nan
    o2, _ = orc.merge_partials(op, lp)
    np.testing.assert_allclose(o2, expect, atol=1e-14)


def test_token_permutation_and_key_shift():
    rng = np.random.default_rng(9)
    n, d = 64, 8
    q, K, V = rng.normal(size=d), rng.normal(size=(n, d)), rng.normal(size=(n, d))
    o, lse = orc.attend(q, K, V, 0.4)
    perm = rng.permutation(n)
    o2, lse2 = orc.attend(q, K[perm], V[perm], 0.4)
    np.testing.assert_allclose(o2, o, atol=1e-14)
    assert abs(lse2 - lse) < 1e-13
    u = rng.normal(size=d)
    o3, lse3 = orc.attend(q, K + u, V, 0.4)
    np.testing.assert_allclose(o3, o, atol=1e-13)
    assert abs(lse3 - (lse + 0.4 * float(q @ u))) < 1e-12


def test_candidate_permutation_and_group_isolation():
    q, kp, vp, ks, vs, go = _tiny_problem(11)
    o, lse = orc.decode_attention(q, kp, vp, ks, vs, go, 0.5)
    # swap the two candidates of group 1 (b = 2, 3)
    perm = [0, 1, 3, 2]
    o2, lse2 = orc.decode_attention(q[perm], kp, vp, [ks[i] for i in perm], [vs[i] for i in perm], go, 0.5)
    np.testing.assert_allclose(o2, o[perm], atol=1e-14)
    np.testing.assert_allclose(lse2, lse[perm], atol=1e-14)
    # changing group 0's prefix must not change group 1's candidates, and must change group 0's
    kp2 = [kp[0] + 1.0, kp[1]]
    o3, _ = orc.decode_attention(q, kp2, vp, ks, vs, go, 0.5)
    np.testing.assert_allclose(o3[2:], o[2:], atol=0)
    assert np.abs(o3[:2] - o[:2]).max() > 1e-3
    # changing candidate 1's suffix changes only candidate 1
    vs2 = list(vs)
    vs2[1] = vs[1] + 1.0
    o4, _ = orc.decode_attention(q, kp, vp, ks, vs2, go, 0.5)
    np.testing.assert_allclose(o4[[0, 2, 3]], o[[0, 2, 3]], atol=0)
    assert np.abs(o4[1] - o[1]).max() > 1e-3


def test_gqa_equals_mha_with_replicated_heads():
    q, kp, vp, ks, vs, go = _tiny_problem(12, Hq=6, Hkv=3)
    g = 2
    o, lse = orc.decode_attention(q, kp, vp, ks, vs, go, 0.5)
    rep = lambda xs: [np.repeat(x, g, axis=1) for x in xs]          # kv head h -> heads h*g .. h*g+g-1
    o2, lse2 = orc.decode_attention(q, rep(kp), rep(vp), rep(ks), rep(vs), go, 0.5)
    np.testing.assert_allclose(o2, o, atol=1e-15)
    np.testing.assert_allclose(lse2, lse, atol=1e-15)
    # the interleaved map (hq % Hkv) is a different function: the oracle must not silently equal it
    o3, _ = orc.decode_attention(q, kp, vp, ks, vs, go, 0.5, kv_head_of=lambda hq, Hq, Hkv: hq % Hkv)
    assert np.abs(o3 - o).max() > 1e-3


def test_rows_subset_matches_full():
    q, kp, vp, ks, vs, go = _tiny_problem(13)
    o, lse = orc.decode_attention(q, kp, vp, ks, vs, go, 0.5)
    o2, lse2 = orc.decode_attention(q, kp, vp, ks, vs, go, 0.5, rows=[(1, 2), (3, 0)])
    np.testing.assert_array_equal(o2[1, 2], o[1, 2])
    np.testing.assert_array_equal(o2[3, 0], o[3, 0])
    assert np.isnan(o2[0, 0]).all() and lse2[3, 0] == lse[3, 0]


# ---------------------------------------------------------------------------------------------------
# library special case: float64 scaled_dot_product_attention on the concatenated, head-repeated K/V
# ---------------------------------------------------------------------------------------------------
def test_matches_torch_sdpa_float64():
    torch = pytest.importorskip("torch")
    q, kp, vp, ks, vs, go = _tiny_problem(14, G=1, C=3, Hq=4, Hkv=2, d=8, P=(11,), S=(0, 4, 9))
    scale = 1.0 / math.sqrt(8)
    o, _ = orc.decode_attention(q, kp, vp, ks, vs, go, scale)
    for b in range(3):
        K = np.concatenate([kp[0], ks[b]], axis=0)          # [n][Hkv][d]
        V = np.concatenate([vp[0], vs[b]], axis=0)
        Kt = torch.from_numpy(np.repeat(K, 2, axis=1)).permute(1, 0, 2)[None]   # [1][Hq][n][d]
        Vt = torch.from_numpy(np.repeat(V, 2, axis=1)).permute(1, 0, 2)[None]
        Qt = torch.from_numpy(q[b])[None, :, None, :]                            # [1][Hq][1][d]
        ref = torch.nn.functional.scaled_dot_product_attention(Qt, Kt, Vt, scale=scale)[0, :, 0].numpy()
        np.testing.assert_allclose(o[b], ref, atol=1e-12)


# ---------------------------------------------------------------------------------------------------
# cascade (prefix tree deeper than two levels): reduces to the two-level function by concatenation
# ---------------------------------------------------------------------------------------------------
def test_cascade_equals_two_level_with_concatenated_prefixes():
    q, kp, vp, ks, vs, go = _tiny_problem(21, G=2, C=2)
    rng = np.random.default_rng(22)
    Hkv, d = kp[0].shape[1], kp[0].shape[2]
    root_k, root_v = rng.normal(size=(7, Hkv, d)), rng.normal(size=(7, Hkv, d))      # shared by all 4 candidates
    o, lse = orc.decode_attention_cascade(q, [([root_k], [root_v], [0, 4]), (kp, vp, go)], ks, vs, 0.4)
    kp2 = [np.concatenate([root_k, k], axis=0) for k in kp]
    vp2 = [np.concatenate([root_v, v], axis=0) for v in vp]
    o2, lse2 = orc.decode_attention(q, kp2, vp2, ks, vs, go, 0.4)
    np.testing.assert_allclose(o, o2, atol=1e-14)
    np.testing.assert_allclose(lse, lse2, atol=1e-13)
    # a single level is the two-level function itself, and the level order is irrelevant
    o3, lse3 = orc.decode_attention_cascade(q, [(kp, vp, go)], ks, vs, 0.4)
    o4, lse4 = orc.decode_attention(q, kp, vp, ks, vs, go, 0.4)
    np.testing.assert_array_equal(o3, o4)
    o5, _ = orc.decode_attention_cascade(q, [(kp, vp, go), ([root_k], [root_v], [0, 4])], ks, vs, 0.4)
    np.testing.assert_allclose(o5, o, atol=1e-14)
    # an outer level whose groups cut across differently: 3 + 1 candidates
    mid_k = [rng.normal(size=(3, Hkv, d)), rng.normal(size=(5, Hkv, d))]
    mid_v = [rng.normal(size=(3, Hkv, d)), rng.normal(size=(5, Hkv, d))]
    o6, lse6 = orc.decode_attention_cascade(q, [(mid_k, mid_v, [0, 3, 4]), (kp, vp, go)], ks, vs, 0.4)
    bo, blse = brute_force_decode(
        q.tolist(), [np.concatenate([mid_k[0 if b < 3 else 1], kp[b // 2]], axis=0).tolist() for b in range(4)],
        [np.concatenate([mid_v[0 if b < 3 else 1], vp[b // 2]], axis=0).tolist() for b in range(4)],
        [x.tolist() for x in ks], [x.tolist() for x in vs], [0, 1, 2, 3, 4], 0.4)
    np.testing.assert_allclose(o6, np.array(bo), atol=1e-12)
    np.testing.assert_allclose(lse6, np.array(blse), atol=1e-12)


# ------------------------------------------------------------------------------------------------------------
# scoring (causal attention of whole sequences behind a shared prompt)
# ------------------------------------------------------------------------------------------------------------
def _scoring_case(seed=0, G=2, C=2, Hq=4, Hkv=2, d=8):
    rng = np.random.default_rng(seed)
    go = [0, C, 2 * C][:G + 1]
    kp = [rng.normal(size=(int(rng.integers(3, 9)), Hkv, d)) for _ in range(G)]
    vp = [rng.normal(size=k.shape) for k in kp]
    ks = [rng.normal(size=(int(rng.integers(1, 7)), Hkv, d)) for _ in range(G * C)]
    vs = [rng.normal(size=k.shape) for k in ks]
    q = [rng.normal(size=(k.shape[0], Hq, d)) for k in ks]
    return q, kp, vp, ks, vs, go


def test_scoring_last_position_is_the_decode_step():
    """The query at a sequence's last position sees the prompt and the whole sequence: exactly one decode step."""
    q, kp, vp, ks, vs, go = _scoring_case(1)
    o, lse = orc.scoring_attention(q, kp, vp, ks, vs, go, 0.3)
    q_last = np.stack([qb[-1] for qb in q])
    o_ref, lse_ref = orc.decode_attention(q_last, kp, vp, ks, vs, go, 0.3)
    for b in range(len(ks)):
        np.testing.assert_allclose(o[b][-1], o_ref[b], atol=1e-14)
        np.testing.assert_allclose(lse[b][-1], lse_ref[b], atol=1e-14)


def test_scoring_is_causal_and_positions_are_decode_steps_of_truncated_sequences():
    q, kp, vp, ks, vs, go = _scoring_case(2)
    o, lse = orc.scoring_attention(q, kp, vp, ks, vs, go, 0.5)
    # changing the tokens after position i changes nothing at or before i
    ks2 = [k.copy() for k in ks]
    vs2 = [v.copy() for v in vs]
    for b in range(len(ks)):
        ks2[b][2:] += 7.0
        vs2[b][2:] -= 3.0
    o2, lse2 = orc.scoring_attention(q, kp, vp, ks2, vs2, go, 0.5)
    for b in range(len(ks)):
        np.testing.assert_array_equal(o[b][:2], o2[b][:2])
        np.testing.assert_array_equal(lse[b][:2], lse2[b][:2])
        if ks[b].shape[0] > 2:
            assert np.abs(o[b][2:] - o2[b][2:]).max() > 1e-3
    # position i of sequence b = a decode step of the sequence cut after token i
    b, i = 1, min(1, ks[1].shape[0] - 1)
    cut_k = [k[:i + 1] if n == b else k for n, k in enumerate(ks)]
    cut_v = [v[:i + 1] if n == b else v for n, v in enumerate(vs)]
    qq = np.stack([q[n][min(i, q[n].shape[0] - 1)] if n == b else q[n][-1] for n in range(len(ks))])
    o_ref, lse_ref = orc.decode_attention(qq, kp, vp, cut_k, cut_v, go, 0.5)
    np.testing.assert_allclose(o[b][i], o_ref[b], atol=1e-14)
    np.testing.assert_allclose(lse[b][i], lse_ref[b], atol=1e-14)


def test_scoring_without_prompt_is_library_causal_attention():
    """With an empty prompt and MHA heads it is plain causal self-attention: torch's float64 routine."""
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(3)
    n, H, d = 6, 2, 4
    k, v, q = (rng.normal(size=(n, H, d)) for _ in range(3))
    o, _ = orc.scoring_attention([q], [np.zeros((0, H, d))], [np.zeros((0, H, d))], [k], [v], [0, 1], 0.7)
    t = lambda a: torch.from_numpy(np.transpose(a, (1, 0, 2))[None].copy())       # [1][H][n][d]
    ref = torch.nn.functional.scaled_dot_product_attention(t(q), t(k), t(v), is_causal=True, scale=0.7)
    np.testing.assert_allclose(o[0], np.transpose(ref[0].numpy(), (1, 0, 2)), atol=1e-12)
