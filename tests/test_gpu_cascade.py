"""Prefix cascades deeper than two levels (a prompt shared by every group in front of each group's own prefix,
and a middle level whose groups cut across the base groups) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import attention as orc
from paper_2601_05475_b200 import binding as mc
from paper_2601_05475_b200 import workload as wl
from paper_2601_05475_b200.harness import DeviceProblem, to_device

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)


def oracle_cascade(hp, q, scale=None):
    levels = [(lv.k, lv.v, lv.group_offsets.tolist()) for lv in hp.outer]
    levels.append((hp.k_prefix, hp.v_prefix, hp.tables.group_offsets.tolist()))
    return orc.decode_attention_cascade(q, levels, hp.k_suffix, hp.v_suffix, hp.cfg.scale if scale is None else scale)


def check(cfg, o, lse, o_ref, lse_ref):
    err = np.abs(o.float().cpu().numpy().astype(np.float64) - o_ref)
    tol = (1e-5, 1e-5) if cfg.dtype == "f32" else (2e-2, 2e-3)
    assert err.max() <= tol[0] and err.mean() <= tol[1], (err.max(), err.mean())
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 1e-3


CASES = {
    # bf16, tensor-core levels: 4 groups x 8 candidates; a 700-token root shared by all 32; a middle level 24 + 8
    "bf16-3-levels": (wl.Config("casc", "bf16", 4, 8, 32, 8, 128, ("loguniform", 100, 900), ("uniform", 0, 300),
                                permute_pages=True, seed=7),
                      [([0, 32], [700]), ([0, 24, 32], [333, 130])]),
    # fp32 (plain-ALU kernels), one outer level
    "f32-2-levels": (wl.Config("cascf", "f32", 2, 3, 4, 2, 64, ("fixed", 70), ("uniform", 0, 50), seed=8),
                     [([0, 6], [45])]),
    # outer level with an empty group
    "bf16-empty-outer-group": (wl.Config("casce", "bf16", 2, 4, 16, 4, 128, ("fixed", 129), ("uniform", 0, 40),
                                         seed=9), [([0, 4, 8], [0, 260])]),
}


@pytest.mark.parametrize("chain", ["1", "0"])
@pytest.mark.parametrize("name", list(CASES))
def test_cascade_matches_oracle(name, chain, monkeypatch):
    """chain: two nested single-split levels run as one item per row tile (the default) or as separate items."""
    monkeypatch.setenv("MC_PREFIX_CHAIN", chain)
    cfg, outer = CASES[name]
    hp = wl.make_host_problem(cfg)
    for i, (go, lens) in enumerate(outer):
        wl.add_outer_level(hp, go, lens, i)
    dp = DeviceProblem.from_host(hp)
    scratch = torch.empty(hp.tables.num_pages, dtype=torch.int32, device="cuda")
    assert mc.mc_kv_layout_validate(dp.layout, scratch, scratch.numel() * 4) == mc.MC_OK
    q = wl.draw_q(cfg, 0)
    o, lse = dp.decode(to_device(cfg, q))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    check(cfg, o, lse, *oracle_cascade(hp, q))
    # appends still work and the outer levels stay in the result
    k_new, v_new = wl.draw_append(cfg, 1)
    q = wl.draw_q(cfg, 1)
    mc.mc_decode_step(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new), to_device(cfg, q), cfg.scale, dp.o,
                      dp.lse, dp.ws_ptr, dp.ws_bytes)
    torch.cuda.synchronize()
    hp.append(k_new, v_new)
    check(cfg, dp.o, dp.lse, *oracle_cascade(hp, q))
    dp.close()


def test_cascade_rejects_bad_level_descriptions():
    cfg, outer = CASES["f32-2-levels"]
    hp = wl.make_host_problem(cfg)
    wl.add_outer_level(hp, *outer[0])
    dp = DeviceProblem.from_host(hp)
    lv = mc.PrefixLevel()
    lv.num_groups, lv.max_pages = 1, 0
    h = mc.c_void_p()
    arr = (mc.PrefixLevel * 1)(lv)
    assert mc.lib().mc_kv_layout_create_cascade(mc.byref(dp.desc), arr, 1, mc.byref(h)) == mc.MC_ERR_INVALID_ARG
    assert mc.lib().mc_kv_layout_create_cascade(mc.byref(dp.desc), arr, 4, mc.byref(h)) == mc.MC_ERR_INVALID_ARG
    assert mc.lib().mc_kv_layout_create_cascade(mc.byref(dp.desc), None, 1, mc.byref(h)) == mc.MC_ERR_INVALID_ARG
    dp.close()


@pytest.mark.parametrize("chain", ["1", "0"])
def test_row_limits_on_the_coarser_level(chain, monkeypatch):
    """An outer level whose candidates see only a per-candidate number of its tokens, in front of unsplit base
    prefixes with the same group boundaries: the two levels run chained (one item per row tile, the limit applied to
    the coarser level's token range) or apart; every row is the plain attention over what it may see."""
    monkeypatch.setenv("MC_PREFIX_CHAIN", chain)
    monkeypatch.setenv("MC_PREFIX_PART_TOKENS", "4096")      # one split per level
    cfg = wl.Config("casl", "bf16", 2, 4, 16, 4, 128, ("fixed", 129), ("uniform", 0, 40), seed=19)
    hp = wl.make_host_problem(cfg)
    wl.add_outer_level(hp, [0, 4, 8], [200, 260], 0)
    dp = DeviceProblem.from_host(hp)
    limit = np.array([10, 10, 150, 200, 0, 33, 260, 300], dtype=np.int32)     # non-decreasing inside a group
    limit_dev = torch.from_numpy(limit).cuda()
    go, ln, pg = dp.outer_tensors[0]
    lv = mc.PrefixLevel()
    lv.num_groups, lv.max_pages = 2, pg.shape[1]
    lv.group_offsets, lv.len, lv.pages, lv.row_limit = go.data_ptr(), ln.data_ptr(), pg.data_ptr(), limit_dev.data_ptr()
    layout = mc.mc_kv_layout_create_cascade(dp.desc, [lv])
    geom = mc.mc_kv_layout_geometry(layout)
    assert geom.n_prefix_parts == 2 and geom.prefix_ctas > 0
    ws = torch.empty(mc.mc_workspace_bytes(layout) + 256, dtype=torch.uint8, device="cuda")
    ws_ptr = (ws.data_ptr() + 255) // 256 * 256
    q = wl.draw_q(cfg, 0)
    mc.mc_decode_attn(layout, to_device(cfg, q), cfg.scale, dp.o, dp.lse, ws_ptr, mc.mc_workspace_bytes(layout))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(layout) == mc.MC_OK
    g = cfg.Hq // cfg.Hkv
    o_ref = np.zeros((cfg.B, cfg.Hq, cfg.d))
    lse_ref = np.zeros((cfg.B, cfg.Hq))
    for b in range(cfg.B):
        j = b // cfg.C
        n = min(int(limit[b]), hp.outer[0].k[j].shape[0])
        for hq in range(cfg.Hq):
            h = hq // g
            K = np.concatenate([hp.outer[0].k[j][:n, h], hp.k_prefix[j][:, h], hp.k_suffix[b][:, h]], axis=0)
            V = np.concatenate([hp.outer[0].v[j][:n, h], hp.v_prefix[j][:, h], hp.v_suffix[b][:, h]], axis=0)
            o_ref[b, hq], lse_ref[b, hq] = orc.attend(q[b, hq], K, V, cfg.scale)
    check(cfg, dp.o, dp.lse, o_ref, lse_ref)
    mc.mc_kv_layout_destroy(layout)
    dp.close()
