"""Scoring / prefill of whole sequences behind a shared prompt (every token a query, causal inside the sequence),
run through the cascade layout with per-candidate row limits, against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import attention as orc
from paper_2601_05475_b200 import binding as mc
from paper_2601_05475_b200 import workload as wl
from paper_2601_05475_b200.harness import ScoringDeviceProblem, to_device

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

CASES = {
    # bf16, tcgen05 kernel: g = 4 -> 32 positions per 128-row tile; sequences longer than a tile, ragged prompts,
    # a one-token and an empty sequence
    "bf16": (wl.Config("score", "bf16", 2, 3, 16, 4, 128, ("fixed", 0), ("fixed", (0,)), permute_pages=True, seed=11),
             [300, 77], [70, 1, 40, 0, 133, 33]),
    # g = 8, a prompt shorter than a page and sequences that end inside a K/V tile
    "bf16-g8": (wl.Config("score8", "bf16", 1, 2, 16, 2, 128, ("fixed", 0), ("fixed", (0,)), seed=12), [9], [150, 260]),
    # fp32: the plain-ALU kernels honour the limits too
    "f32": (wl.Config("scoref", "f32", 2, 2, 4, 2, 64, ("fixed", 0), ("fixed", (0,)), seed=13), [40, 17], [20, 5, 33, 18]),
}


@pytest.mark.parametrize("suffix_storage", [False, True, "one-row-tile-items"])
@pytest.mark.parametrize("name", list(CASES))
def test_scoring_matches_oracle(name, suffix_storage, monkeypatch):
    """suffix_storage True also runs the two levels as separate items (MC_PREFIX_CHAIN=0) instead of chained ones.
    suffix_storage False: a layout without private tokens (no suffix part slot, no suffix launch); True: a decode
    layout whose suffixes happen to be empty (the suffix pass runs and reports empty parts)."""
    cfg, prefix_len, seq_len = CASES[name]
    hp = wl.make_scoring_host_problem(cfg, prefix_len, seq_len)
    q = wl.draw_scoring_q(cfg, seq_len)
    if suffix_storage == "one-row-tile-items":      # the prefix kernel that gives each 128-row tile an item of its own
        monkeypatch.setenv("MC_PREFIX_PAIRS", "0")
        suffix_storage = False
    if suffix_storage:
        monkeypatch.setenv("MC_PREFIX_CHAIN", "0")
    dp = ScoringDeviceProblem(hp, suffix_storage=suffix_storage)
    assert dp.geom.n_parts == dp.geom.n_prefix_parts + (1 if suffix_storage else 0)
    assert (dp.geom.prefix_ctas > 0) == (cfg.dtype == "bf16")      # bf16 cases run on the tcgen05 kernel
    scratch = torch.empty(hp.k_pool.shape[0], dtype=torch.int32, device="cuda")
    assert mc.mc_kv_layout_validate(dp.layout, scratch, scratch.numel() * 4) == mc.MC_OK
    o, lse = dp.score(to_device(cfg, np.concatenate(q, axis=0)))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    o_ref, lse_ref = orc.scoring_attention(q, hp.k_prefix, hp.v_prefix, hp.k_seq, hp.v_seq,
                                           [0, cfg.C, 2 * cfg.C][:cfg.G + 1], cfg.scale)
    o_ref, lse_ref = np.concatenate(o_ref, axis=0), np.concatenate(lse_ref, axis=0)
    err = np.abs(o.float().cpu().numpy().astype(np.float64) - o_ref)
    tol = (1e-5, 1e-5) if cfg.dtype == "f32" else (2e-2, 2e-3)
    assert err.max() <= tol[0] and err.mean() <= tol[1], (err.max(), err.mean())
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 1e-3
    if not suffix_storage:       # nowhere to append
        kv = to_device(cfg, np.zeros((dp.n_virtual, cfg.Hkv, cfg.d), dtype=np.float32))
        with pytest.raises(mc.McError):
            mc.mc_kv_append(dp.layout, kv, kv)
    dp.close()


@pytest.mark.parametrize("n_spec", [1, 4])
def test_multi_token_decode_step(n_spec):
    """A decode step that checks several speculated tokens per candidate at once: the last n_spec tokens of every
    sequence are queries, each seeing the prompt and its sequence up to itself (n_spec = 1 is the ordinary step)."""
    cfg = wl.Config("spec", "bf16", 2, 4, 16, 4, 128, ("fixed", 0), ("fixed", (0,)), permute_pages=True, seed=21)
    prefix_len, seq_len = [200, 50], [90, 3, 40, 17, 64, 1, 130, 33]
    hp = wl.make_scoring_host_problem(cfg, prefix_len, seq_len, last_queries=n_spec)
    q_all = wl.draw_scoring_q(cfg, seq_len)
    q = [x[-n_spec:] for x in q_all]
    dp = ScoringDeviceProblem(hp)
    o, lse = dp.score(to_device(cfg, np.concatenate(q, axis=0)))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    o_ref, lse_ref = orc.scoring_attention(q_all, hp.k_prefix, hp.v_prefix, hp.k_seq, hp.v_seq, [0, 4, 8], cfg.scale)
    o_ref = np.concatenate([x[-n_spec:] for x in o_ref], axis=0)
    lse_ref = np.concatenate([x[-n_spec:] for x in lse_ref], axis=0)
    err = np.abs(o.float().cpu().numpy().astype(np.float64) - o_ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 1e-3
    dp.close()


def test_decreasing_row_limits_are_reported_by_validate():
    cfg, prefix_len, seq_len = CASES["f32"]
    hp = wl.make_scoring_host_problem(cfg, prefix_len, seq_len)
    hp.row_limit[3] = 1          # positions 1, 2, 3, 1, ... inside the first sequence
    dp = ScoringDeviceProblem(hp)
    scratch = torch.empty(hp.k_pool.shape[0], dtype=torch.int32, device="cuda")
    assert mc.mc_kv_layout_validate(dp.layout, scratch, scratch.numel() * 4) == mc.MC_ERR_INVALID_ARG
    dp.close()


@pytest.mark.parametrize("direct", ["1", "0"])
def test_prefix_only_layout_single_level(direct, monkeypatch):
    """A plain two-level layout without suffix storage: the prefix pass is the whole step and (direct = 1) writes the
    final output itself, or (direct = 0) one part per row that the merge turns into the output."""
    from paper_2601_05475_b200.harness import DeviceProblem
    monkeypatch.setenv("MC_PREFIX_DIRECT", direct)
    monkeypatch.setenv("MC_PREFIX_PART_TOKENS", "4096")      # one split: one part per row
    cfg = wl.Config("ponly", "bf16", 3, 5, 16, 4, 128, ("loguniform", 1, 700), ("fixed", (0,)), permute_pages=True, seed=31)
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    d = dp.desc
    d.max_suffix_pages, d.suffix_pages, d.suffix_len = 0, 0, 0
    layout = mc.mc_kv_layout_create(d)
    geom = mc.mc_kv_layout_geometry(layout)
    assert geom.n_parts == geom.n_prefix_parts == 1 and geom.prefix_ctas > 0
    q = wl.draw_q(cfg, 0)
    o = torch.full((cfg.B, cfg.Hq, cfg.d), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((cfg.B, cfg.Hq), float("nan"), dtype=torch.float32, device="cuda")
    launches = mc.mc_launch_count()
    mc.mc_decode_attn(layout, to_device(cfg, q), cfg.scale, o, lse, dp.ws_ptr, dp.ws_bytes)
    torch.cuda.synchronize()
    assert mc.mc_launch_count() - launches == (1 if direct == "1" else 2)
    assert mc.mc_get_last_status(layout) == mc.MC_OK
    o_ref, lse_ref = orc.decode_attention(q, hp.k_prefix, hp.v_prefix, hp.k_suffix, hp.v_suffix,
                                          hp.tables.group_offsets.tolist(), cfg.scale)
    err = np.abs(o.float().cpu().numpy().astype(np.float64) - o_ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 1e-3
    mc.mc_kv_layout_destroy(layout)
    dp.close()
