"""Full-size configurations in the launch configuration the benchmark times: sampled output rows against
the CPU oracle (each row's whole history is copied back through the page tables and attended in fp64),
plus properties that hold at any size."""
import numpy as np
import pytest
import torch

from oracle import attention as orc
from paper_2601_05475_b200 import binding as mc
from paper_2601_05475_b200 import workload as wl
from paper_2601_05475_b200.harness import device_append, device_q, logical_rows, make_device_problem

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)


def check_rows(dp, q, o, lse, rows):
    cfg = dp.cfg
    errs, lerrs = [], []
    for (b, hq) in rows:
        K, V = logical_rows(dp, b, hq // cfg.g)
        o_ref, lse_ref = orc.attend(q[b, hq].float().cpu().numpy(), K, V, cfg.scale)
        errs.append(np.abs(o[b, hq].float().cpu().numpy().astype(np.float64) - o_ref))
        lerrs.append(abs(float(lse[b, hq]) - lse_ref))
    errs = np.stack(errs)
    assert errs.max() <= 2e-2 and errs.mean() <= 2e-3, (errs.max(), errs.mean())
    assert np.max(lerrs) <= 1e-3, np.max(lerrs)           # np.max propagates a NaN, the builtin may not


def sample_rows(cfg, n, seed):
    rng = np.random.default_rng(seed)
    rows = [(int(rng.integers(cfg.B)), int(rng.integers(cfg.Hq))) for _ in range(n)]
    return rows + [(0, 0), (cfg.B - 1, cfg.Hq - 1)]


@pytest.mark.parametrize("name,n_rows,steps", [("cfg2", 24, 32), ("cfg3", 24, 0), ("cfg4", 10, 64)])
def test_full_size_sampled_rows(name, n_rows, steps):
    """The configuration as the benchmark runs it: one decode step, then the whole append sweep (32 consecutive
    steps for configuration 2, 64 for configuration 4) through mc_decode_step, with sampled rows checked against
    the oracle on the first steps, around the step that opens a new page for every candidate, and on the last."""
    cfg = wl.CONFIGS[name]
    dp = make_device_problem(cfg, headroom_tokens=steps + 1)
    q = device_q(cfg, 0)
    o, lse = dp.decode(q)
    torch.cuda.synchronize()
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    check_rows(dp, q, o, lse, sample_rows(cfg, n_rows, 1))
    len0 = dp.suffix_len.clone()
    for step in range(1, steps + 1):
        k_new, v_new = device_append(cfg, step)
        q = device_q(cfg, step)
        mc.mc_decode_step(dp.layout, k_new, v_new, q, cfg.scale, dp.o, dp.lse, dp.ws_ptr, dp.ws_bytes)
        if step not in (1, 2, 15, 16, 17, steps):
            continue
        torch.cuda.synchronize()
        assert torch.equal(dp.suffix_len, len0 + step)
        assert torch.isfinite(dp.o.float()).all() and torch.isfinite(dp.lse).all()
        rows = sample_rows(cfg, 6, 10 + step)
        check_rows(dp, q, dp.o, dp.lse, rows)
        # the appended token is the last row of each sampled candidate's history
        b, hq = rows[0]
        K, V = logical_rows(dp, b, hq // cfg.g)
        np.testing.assert_array_equal(K[-1], k_new[b, hq // cfg.g].float().cpu().numpy())
        np.testing.assert_array_equal(V[-1], v_new[b, hq // cfg.g].float().cpu().numpy())
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    dp.close()


def test_full_size_properties_cfg2():
    """Any-size properties: constant V gives that constant; candidates of one group with identical queries
    and empty suffixes give identical outputs; lse grows by log 2 when the history is duplicated."""
    cfg = wl.CONFIGS["cfg2"]
    dp = make_device_problem(cfg)
    q = device_q(cfg, 0)
    dp.v_pool.fill_(0.5)
    o, _ = dp.decode(q)
    torch.cuda.synchronize()
    assert (o.float() - 0.5).abs().max().item() <= 4e-3
    dp.suffix_len.zero_()
    q[:] = q[0:1]
    o, lse = dp.decode(q)
    torch.cuda.synchronize()
    assert torch.equal(o[0], o[17]) and torch.equal(lse[0], lse[63])
    dp.close()


def test_full_size_cascade_cfg3_with_a_root_prompt():
    """Configuration 3 with a 4096-token prompt shared by all 256 candidates in front of the group prefixes
    (stacked query tile of 1024 rows per kv head at the root level)."""
    cfg = wl.CONFIGS["cfg3"]
    dp = make_device_problem(cfg, outer=[([0, cfg.B], [4096])])
    assert dp.geom.n_prefix_parts >= 2
    q = device_q(cfg, 0)
    o, lse = dp.decode(q)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    check_rows(dp, q, o, lse, sample_rows(cfg, 16, 3))
    dp.close()


def test_merge_waits_for_a_prefix_pass_that_outlasts_the_suffix_pass(monkeypatch):
    """The suffix pass starts while the prefix pass is still running; the merge must not.  A long prefix on few
    CTAs against suffixes of at most one page: the fused call equals the three passes run one after another."""
    monkeypatch.setenv("MC_PREFIX_CTAS", "8")
    cfg = wl.Config("long_prefix", "bf16", G=4, C=16, Hq=32, Hkv=8, d=128, prefix=("fixed", 32768),
                    suffix=("uniform", 0, 16))
    dp = make_device_problem(cfg, headroom_tokens=4)
    q = device_q(cfg, 0)
    g = dp.geom
    assert g.prefix_ctas == 8
    lse_off = (g.rows * g.n_parts * g.head_dim * 4 + 255) // 256 * 256
    o_part, lse_part = dp.ws_ptr, dp.ws_ptr + lse_off
    o_ref, lse_ref = torch.empty_like(dp.o), torch.empty_like(dp.lse)
    mc.mc_prefix_attn(dp.layout, q, cfg.scale, o_part, lse_part)
    mc.mc_suffix_attn(dp.layout, q, cfg.scale, o_part, lse_part)
    mc.mc_merge_lse(dp.layout, o_part, lse_part, o_ref, lse_ref)
    torch.cuda.synchronize()
    check_rows(dp, q, o_ref, lse_ref, sample_rows(cfg, 4, 5))
    for _ in range(5):
        dp.ws.zero_()   # a merge that ran early would find empty prefix parts
        dp.o.zero_()
        dp.lse.zero_()
        o, lse = dp.decode(q)
        torch.cuda.synchronize()
        assert torch.equal(o, o_ref) and torch.equal(lse, lse_ref)
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    dp.close()


def test_search_bookkeeping_at_bench_size_sampled_rows():
    """2^20 trajectories x 8 steps, the launch configuration bench.py times; 300 sampled trajectories and every
    problem's selection are checked against the oracle."""
    from oracle import search as sorc
    b = wl.draw_search_batch(problems=1 << 17, K=8, T=8, seed=0)
    N, T, P = b["N"], b["T"], b["P"]
    dev = lambda a: torch.from_numpy(a).cuda()
    r = torch.empty((T, N), dtype=torch.uint8, device="cuda")
    lab = torch.empty_like(r)
    u, v = torch.empty((T, N), device="cuda"), torch.empty((T, N), device="cuda")
    G = torch.empty(N, device="cuda")
    best = torch.empty(P, dtype=torch.int32, device="cuda")
    s1, s2, s3 = wl.SEARCH_THRESHOLDS
    mc.mc_search_returns(dev(b["speedup"]), dev(b["correct"]), dev(b["len"]), N, T, s1, s2, s3, 0.95, r, u, v, lab, G)
    mc.mc_search_group_argmax(G, dev(b["group_offsets"]), P, best)
    torch.cuda.synchronize()
    r, u, v, lab, G, best = (x.cpu().numpy() for x in (r, u, v, lab, G, best))
    rng = np.random.default_rng(0)
    for n in [0, N - 1] + [int(x) for x in rng.integers(N, size=300)]:
        L = int(b["len"][n])
        sp, ok = b["speedup"][:L, n].astype(np.float64), b["correct"][:L, n] != 0
        rr = [sorc.categorical_reward(s, c, s1, s2, s3) for s, c in zip(sp, ok)]
        assert r[:L, n].tolist() == rr
        np.testing.assert_allclose(u[:L, n], sorc.best_so_far(rr, 0.95), rtol=1e-5)
        np.testing.assert_allclose(v[:L, n], sorc.value_targets(rr, 0.95), rtol=1e-5)
        l_ref, m = sorc.future_labels(sp, ok, 0.95, s1, s2, s3)
        clear = np.abs(m[:, None] - np.array([100.0, s1, s2, s3])[None, :]).min(axis=1) > 1e-3
        assert (lab[:L, n][clear] == l_ref[clear]).all()
        assert abs(G[n] - sorc.trajectory_return(rr, 0.95)) <= 1e-5
    assert best.tolist() == sorc.group_argmax(G, b["group_offsets"]).tolist()   # fp32 values, exact decision


def test_scoring_at_bench_size_sampled_rows():
    """32 sequences x 512 tokens behind 4096-token prompts (the configuration bench.py times): 48 sampled
    (sequence, position, head) rows, among them first and last positions, against the oracle's row-by-row definition."""
    from paper_2601_05475_b200.harness import ScoringDeviceProblem, to_device
    scfg = wl.Config("scoring", "bf16", 4, 8, 32, 8, 128, ("fixed", 4096), ("fixed", (0,)), permute_pages=True)
    seq_len = [512] * scfg.B
    hp = wl.make_scoring_host_problem(scfg, [4096] * scfg.G, seq_len)
    q = wl.draw_scoring_q(scfg, seq_len)
    dp = ScoringDeviceProblem(hp)
    assert dp.geom.prefix_ctas > 0
    o, lse = dp.score(to_device(scfg, np.concatenate(q, axis=0)))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    o, lse = o.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
    rng = np.random.default_rng(0)
    rows = [(0, 0, 0), (31, 511, 31), (5, 127, 3), (5, 128, 3)] + \
           [(int(rng.integers(32)), int(rng.integers(512)), int(rng.integers(32))) for _ in range(44)]
    errs = []
    for (b, i, hq) in rows:
        j, h = b // scfg.C, hq // scfg.g
        K = np.concatenate([hp.k_prefix[j][:, h], hp.k_seq[b][:i + 1, h]], axis=0)
        V = np.concatenate([hp.v_prefix[j][:, h], hp.v_seq[b][:i + 1, h]], axis=0)
        o_ref, lse_ref = orc.attend(q[b][i, hq], K, V, scfg.scale)
        v = int(hp.seq_offsets[b]) + i
        errs.append(np.abs(o[v, hq] - o_ref))
        assert abs(lse[v, hq] - lse_ref) <= 1e-3
    errs = np.concatenate(errs)
    assert errs.max() <= 2e-2 and errs.mean() <= 2e-3
    dp.close()
