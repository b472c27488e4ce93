"""GPU parity of the search bookkeeping (through the C ABI) against the fp64 oracle, element by element.
Integer outputs (reward classes, argmax indices) are compared exactly; labels exactly except where the fp64
discounted maximum lies within 1e-3 percent of a class boundary (fp32 and fp64 may then fall on either side);
floating-point outputs within 1e-5 relative (fp32 products of at most 32 factors)."""
import numpy as np
import pytest
import torch

from oracle import search as orc
from paper_2601_05475_b200 import binding as mc
from paper_2601_05475_b200 import workload as wl

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

S = wl.SEARCH_THRESHOLDS


def run_returns(batch, gamma, use_len=True, outputs=("reward", "u", "v", "label", "G")):
    N, T = batch["N"], batch["T"]
    dev = lambda a: torch.from_numpy(a).cuda()
    sp, ok, ln = dev(batch["speedup"]), dev(batch["correct"]), dev(batch["len"])
    out = {
        "reward": torch.full((T, N), 77, dtype=torch.uint8, device="cuda"),
        "u": torch.full((T, N), float("nan"), device="cuda"),
        "v": torch.full((T, N), float("nan"), device="cuda"),
        "label": torch.full((T, N), 77, dtype=torch.uint8, device="cuda"),
        "G": torch.full((N,), float("nan"), device="cuda"),
    }
    arg = lambda k: out[k] if k in outputs else None
    mc.mc_search_returns(sp, ok, ln if use_len else None, N, T, S[0], S[1], S[2], gamma, arg("reward"), arg("u"),
                         arg("v"), arg("label"), arg("G"))
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def check_returns(batch, gamma, got, use_len=True, outputs=("reward", "u", "v", "label", "G")):
    N, T = batch["N"], batch["T"]
    for n in range(N):
        L = int(batch["len"][n]) if use_len else T
        sp = batch["speedup"][:L, n].astype(np.float64)
        ok = batch["correct"][:L, n] != 0
        r = [orc.categorical_reward(s, c, *S) for s, c in zip(sp, ok)]
        if "reward" in outputs:
            assert got["reward"][:L, n].tolist() == r
            assert (got["reward"][L:, n] == 0).all()
        if "u" in outputs:
            np.testing.assert_allclose(got["u"][:L, n], orc.best_so_far(r, gamma), rtol=1e-5, atol=1e-7)
            assert (got["u"][L:, n] == 0).all()
        if "v" in outputs:
            np.testing.assert_allclose(got["v"][:L, n], orc.value_targets(r, gamma), rtol=1e-5, atol=1e-7)
            assert (got["v"][L:, n] == 0).all()
        if "label" in outputs:
            lab, m = orc.future_labels(sp, ok, gamma, *S)
            edges = np.array([100.0, *S])
            clear = np.abs(m[:, None] - edges[None, :]).min(axis=1) > 1e-3
            assert (got["label"][:L, n][clear] == lab[clear]).all()
            assert (np.abs(got["label"][:L, n] - lab) <= 1).all()
            assert (got["label"][L:, n] == 0).all()
        if "G" in outputs:
            ref = orc.trajectory_return(r, gamma) if L else 0.0
            assert abs(got["G"][n] - ref) <= 1e-5 * max(1.0, ref)


@pytest.mark.parametrize("T,gamma", [(8, 1.0), (8, 0.9), (5, 0.5), (13, 0.97), (27, 0.8), (40, 0.95)])
def test_returns_match_oracle(T, gamma):
    """T = 8 is the paper's depth; 13 / 27 / 40 take the 16-step, the 32-step and the any-length kernel; 300
    trajectories span two thread blocks with a ragged tail."""
    for problems in (60, 61):     # 300 trajectories (a multiple of 4: four per thread when T <= 8) and 305 (one per thread)
        batch = wl.draw_search_batch(problems=problems, K=5, T=T, seed=T)
        got = run_returns(batch, gamma)
        check_returns(batch, gamma, got)


def test_returns_without_lengths_and_with_skipped_outputs():
    batch = wl.draw_search_batch(problems=20, K=8, T=8, seed=3)
    got = run_returns(batch, 0.9, use_len=False)
    check_returns(batch, 0.9, got, use_len=False)
    batch = wl.draw_search_batch(problems=10, K=8, T=40, seed=4)
    got = run_returns(batch, 0.9, outputs=("v", "G"))          # value targets without the best-so-far array
    check_returns(batch, 0.9, got, outputs=("v", "G"))
    assert (got["reward"] == 77).all() and np.isnan(got["u"]).all()   # skipped outputs are not touched


def test_fixture_of_the_hand_computed_example():
    batch = {"N": 1, "T": 4, "speedup": np.array([[110.0], [400.0], [350.0], [90.0]], dtype=np.float32),
             "correct": np.array([[1], [0], [1], [1]], dtype=np.uint8), "len": np.array([4], dtype=np.int32)}
    got = run_returns(batch, 0.5)
    assert got["reward"][:, 0].tolist() == [1, 0, 4, 0]
    assert got["u"][:, 0].tolist() == [1, 1, 1, 1] and got["v"][:, 0].tolist() == [2, 2, 4, 2]
    assert got["label"][:, 0].tolist() == [1, 2, 4, 0] and got["G"][0] == 1


def test_value_head_and_selection_match_oracle():
    batch = wl.draw_search_batch(problems=70, K=8, T=8, seed=5)
    N, P = batch["N"], batch["P"]
    logits = torch.from_numpy(batch["logits"]).cuda()
    prob = torch.empty((N, 5), device="cuda")
    ev = torch.empty((N,), device="cuda")
    mc.mc_search_value_head(logits, N, prob, ev)
    go = torch.from_numpy(batch["group_offsets"]).cuda()
    best = torch.full((P,), -9, dtype=torch.int32, device="cuda")
    mc.mc_search_group_argmax(ev, go, P, best)
    torch.cuda.synchronize()
    prob, ev_h, best = prob.cpu().numpy(), ev.cpu().numpy(), best.cpu().numpy()
    ref_ev = np.zeros(N)
    for n in range(N):
        p, e = orc.value_head(batch["logits"][n].astype(np.float64))
        np.testing.assert_allclose(prob[n], p, rtol=1e-5, atol=1e-7)
        assert abs(ev_h[n] - e) <= 1e-5
        ref_ev[n] = e
    # the selection is decided in fp32 on the device: exact against the oracle's argmax of the device's own values,
    # and a valid choice (within rounding of the best) against the fp64 values
    assert best.tolist() == orc.group_argmax(ev_h, batch["group_offsets"]).tolist()
    ref_best = orc.group_argmax(ref_ev, batch["group_offsets"])
    for j in range(P):
        assert ref_ev[best[j]] >= ref_ev[ref_best[j]] - 2e-5


def test_fused_selection_matches_oracle_and_the_separate_calls():
    """mc_search_select: value head, selection by mean value and selection by return in one launch."""
    batch = wl.draw_search_batch(problems=70, K=8, T=8, seed=6)
    N, P = batch["N"], batch["P"]
    rng = np.random.default_rng(2)
    G_np = (rng.integers(0, 5, size=N) * 0.9 ** rng.integers(0, 8, size=N)).astype(np.float32)             # many ties
    go_np = batch["group_offsets"].copy()
    go_np[3] = go_np[2]                                        # an empty group
    logits, G, go = (torch.from_numpy(a).cuda() for a in (batch["logits"], G_np, go_np))
    prob = torch.full((N, 5), -7.0, device="cuda")
    ev = torch.full((N,), -7.0, device="cuda")
    best_g, best_e = (torch.full((P,), -9, dtype=torch.int32, device="cuda") for _ in range(2))
    mc.mc_search_select(logits, G, go, P, prob, ev, best_g, best_e)
    torch.cuda.synchronize()
    prob, ev_h = prob.cpu().numpy(), ev.cpu().numpy()
    inside = np.zeros(N, dtype=bool)
    for j in range(P):
        inside[go_np[j]:go_np[j + 1]] = True
    for n in range(N):
        if inside[n]:
            p, e = orc.value_head(batch["logits"][n].astype(np.float64))
            np.testing.assert_allclose(prob[n], p, rtol=1e-5, atol=1e-7)
            assert abs(ev_h[n] - e) <= 1e-5
        else:                                                  # entries outside every group are not visited
            assert ev_h[n] == -7.0
    assert best_g.cpu().tolist() == orc.group_argmax(G_np, go_np).tolist()           # exact: the inputs are given
    assert best_e.cpu().tolist() == orc.group_argmax(np.where(inside, ev_h, np.nan), go_np).tolist()
    assert best_g.cpu().tolist()[2] == -1
    # the separate calls give the same
    ev2 = torch.empty((N,), device="cuda")
    b2 = torch.empty((P,), dtype=torch.int32, device="cuda")
    mc.mc_search_value_head(logits, N, None, ev2)
    mc.mc_search_group_argmax(ev2, go, P, b2)
    torch.cuda.synchronize()
    assert torch.equal(b2, best_e) and torch.equal(ev2[torch.from_numpy(inside).cuda()], ev[torch.from_numpy(inside).cuda()])
    # only the selection, nothing stored; and the host checks
    best_only = torch.full((P,), -9, dtype=torch.int32, device="cuda")
    mc.mc_search_select(logits, None, go, P, None, None, None, best_only)
    torch.cuda.synchronize()
    assert torch.equal(best_only, best_e)
    with pytest.raises(mc.McError):
        mc.mc_search_select(logits, G, go, P, None, ev, None, best_only)            # a return array without its output
    only_g = torch.full((P,), -9, dtype=torch.int32, device="cuda")
    mc.mc_search_select(logits, G, go, P, None, None, only_g, None)                  # only tau*
    torch.cuda.synchronize()
    assert torch.equal(only_g, best_g)
    with pytest.raises(mc.McError):
        mc.mc_search_select(logits, None, go, P)                                     # nothing asked for


def test_group_argmax_edge_cases():
    vals = torch.tensor([1.0, 3.0, 3.0, 2.0, float("nan"), -1.0, float("-inf")] + [0.5] * 70 + [9.0], device="cuda")
    go = torch.tensor([0, 4, 4, 6, 7, 78], dtype=torch.int32, device="cuda")
    best = torch.full((5,), -9, dtype=torch.int32, device="cuda")
    mc.mc_search_group_argmax(vals, go, 5, best)
    torch.cuda.synchronize()
    # ties -> first; empty -> -1; NaN never selected; a lone -inf is still an entry; a group longer than a warp
    assert best.cpu().tolist() == [1, -1, 5, 6, 77]


def test_search_host_errors():
    x = torch.zeros(8, device="cuda")
    c = torch.zeros(8, dtype=torch.uint8, device="cuda")
    L = mc.lib()
    assert L.mc_search_returns(None, c.data_ptr(), None, 8, 1, 120.0, 200.0, 300.0, 1.0, *([None] * 5), None) == mc.MC_ERR_INVALID_ARG
    assert L.mc_search_returns(x.data_ptr(), c.data_ptr(), None, 8, 1, 200.0, 120.0, 300.0, 1.0, *([None] * 5), None) == mc.MC_ERR_INVALID_ARG
    assert L.mc_search_returns(x.data_ptr(), c.data_ptr(), None, 8, 1, 120.0, 200.0, 300.0, 1.5, *([None] * 5), None) == mc.MC_ERR_INVALID_ARG
    assert L.mc_search_returns(x.data_ptr(), c.data_ptr(), None, 0, 1, 120.0, 200.0, 300.0, 1.0, *([None] * 5), None) == mc.MC_ERR_INVALID_ARG
    assert L.mc_search_value_head(None, 4, None, x.data_ptr(), None) == mc.MC_ERR_INVALID_ARG
    assert L.mc_search_group_argmax(x.data_ptr(), None, 1, None, None) == mc.MC_ERR_INVALID_ARG
