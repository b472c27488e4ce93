"""GPU parity: the CUDA library (through its C ABI) against the fp64 CPU oracle, element by element, on the
same seeded inputs.  Tolerances: fp32 max-abs 1e-5; bf16 max-abs 2e-2 and mean-abs 2e-3; lse 1e-3 per row."""
import os

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


def check_close(cfg, o_gpu, lse_gpu, o_ref, lse_ref, rows=None):
    o = o_gpu.float().cpu().numpy().astype(np.float64)
    lse = lse_gpu.cpu().numpy().astype(np.float64)
    if rows is not None:
        idx = tuple(np.array(rows).T)
        o, lse, o_ref, lse_ref = o[idx], lse[idx], o_ref[idx], lse_ref[idx]
    err = np.abs(o - o_ref)
    assert np.isfinite(o).all()
    if cfg.dtype == "f32":
        assert err.max() <= 1e-5, err.max()
    else:
        assert err.max() <= 2e-2, err.max()
        assert err.mean() <= 2e-3, err.mean()
    assert not np.isnan(lse).any()
    empty = np.isneginf(lse_ref)                       # rows without any token: -inf on both sides
    assert np.array_equal(np.isneginf(lse), empty)
    lerr = np.abs(lse[~empty] - lse_ref[~empty])
    assert lerr.size == 0 or lerr.max() <= 1e-3, lerr.max()
    return err.max(), err.mean()


def oracle_full(hp, q, rows=None):
    return orc.decode_attention(q, hp.k_prefix, hp.v_prefix, hp.k_suffix, hp.v_suffix,
                                hp.tables.group_offsets.tolist(), hp.cfg.scale, rows=rows)


def run_decode(hp, q_np):
    dp = DeviceProblem.from_host(hp)
    q = to_device(hp.cfg, q_np)
    o, lse = dp.decode(q)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    return dp, o, lse


SMALL = {
    "cfg0": wl.CONFIGS["cfg0"],
    "cfg1": wl.CONFIGS["cfg1"],
    "cfg2s": wl.scaled_down(wl.CONFIGS["cfg2"], "cfg2s", C=8, prefix=("fixed", 1040), suffix=("uniform", 0, 600),
                            append_steps=4),
    "cfg3s": wl.scaled_down(wl.CONFIGS["cfg3"], "cfg3s", G=3, C=4, prefix=("loguniform", 90, 1500),
                            suffix=("uniform", 0, 700)),
    "cfg3sp": wl.scaled_down(wl.CONFIGS["cfg3"], "cfg3sp", G=3, C=4, prefix=("loguniform", 90, 1500),
                             suffix=("uniform", 0, 700), permute_pages=True),
    "cfg4s": wl.scaled_down(wl.CONFIGS["cfg4"], "cfg4s", G=2, C=3, prefix=("fixed", 512),
                            suffix=("uniform", 1000, 2100), append_steps=2),
}


@pytest.mark.parametrize("name", list(SMALL))
def test_decode_matches_oracle(name):
    cfg = SMALL[name]
    hp = wl.make_host_problem(cfg)
    q = wl.draw_q(cfg, 0)
    dp, o, lse = run_decode(hp, q)
    o_ref, lse_ref = oracle_full(hp, q)
    check_close(cfg, o, lse, o_ref, lse_ref)
    dp.close()


@pytest.mark.parametrize("name", ["cfg2s", "cfg4s"])
def test_append_sweep_matches_oracle_every_step(name):
    cfg = SMALL[name]
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    for step in range(1, cfg.append_steps + 1):
        k_new, v_new = wl.draw_append(cfg, step)
        q = wl.draw_q(cfg, step)
        if step % 2:                      # alternate the two ways of taking a step
            mc.mc_kv_append(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new))
            o, lse = dp.decode(to_device(cfg, q))
        else:
            mc.mc_decode_step(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new), to_device(cfg, q), cfg.scale,
                              dp.o, dp.lse, dp.ws_ptr, dp.ws_bytes)
            o, lse = dp.o, dp.lse
        hp.append(k_new, v_new)
        torch.cuda.synchronize()
        check_close(cfg, o, lse, *oracle_full(hp, q))
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), hp.suffix_len)
    # one more append than the head-room allows: rows that are full are refused and reported
    for _ in range(wl.PAGE + 1):
        mc.mc_kv_append(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new))
    assert mc.mc_get_last_status(dp.layout) == mc.MC_ERR_INVALID_ARG
    dp.close()


def test_appends_that_open_new_chunks(monkeypatch):
    """Suffixes that end exactly on a chunk boundary: the appended token opens a chunk that had no tokens when
    the layout (and the suffix pass's serving order) was made, and later appends fill it."""
    monkeypatch.setenv("MC_SUFFIX_PART_TOKENS", "32")
    cfg = wl.scaled_down(wl.CONFIGS["cfg2"], "boundary", C=6, prefix=("fixed", 200),
                         suffix=("fixed", (0, 32, 64, 31, 96, 33)), append_steps=3)
    hp = wl.make_host_problem(cfg, headroom_tokens=40)
    dp = DeviceProblem.from_host(hp)
    assert dp.geom.suffix_part_tokens == 32
    for step in range(1, 36):
        k_new, v_new = wl.draw_append(cfg, step)
        q = wl.draw_q(cfg, step)
        mc.mc_decode_step(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new), to_device(cfg, q), cfg.scale,
                          dp.o, dp.lse, dp.ws_ptr, dp.ws_bytes)
        hp.append(k_new, v_new)
        if step in (1, 2, 17, 33, 35):
            torch.cuda.synchronize()
            check_close(cfg, dp.o, dp.lse, *oracle_full(hp, q))
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    dp.close()


def test_many_consecutive_steps_stay_correct():
    """240 decode steps in a row on one layout (appends cross page, tile and chunk boundaries many times; every
    barrier of the persistent prefix kernel goes through hundreds of phases); the oracle checks a step now and then
    and the status word stays clean."""
    cfg = wl.scaled_down(wl.CONFIGS["cfg2"], "soak", C=16, prefix=("fixed", 777), suffix=("uniform", 0, 300),
                         append_steps=240)
    hp = wl.make_host_problem(cfg, headroom_tokens=250)
    dp = DeviceProblem.from_host(hp)
    assert dp.geom.prefix_ctas > 0
    for step in range(1, 241):
        k_new, v_new = wl.draw_append(cfg, step)
        q = wl.draw_q(cfg, step)
        mc.mc_decode_step(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new), to_device(cfg, q), cfg.scale,
                          dp.o, dp.lse, dp.ws_ptr, dp.ws_bytes)
        hp.append(k_new, v_new)
        if step % 60 == 0 or step in (1, 17, 239):
            torch.cuda.synchronize()
            rows = [(b, hq) for b in (0, 7, 15) for hq in (0, 31, 63)]
            o_ref, lse_ref = oracle_full(hp, q, rows=rows)
            check_close(cfg, dp.o, dp.lse, o_ref, lse_ref, rows=rows)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    assert torch.isfinite(dp.o.float()).all()
    dp.close()


def test_layouts_can_be_created_and_destroyed_repeatedly():
    cfg = SMALL["cfg3s"]
    hp = wl.make_host_problem(cfg)
    q = to_device(cfg, wl.draw_q(cfg, 0))
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for _ in range(40):
        dp = DeviceProblem.from_host(hp)
        dp.decode(q)
        torch.cuda.synchronize()
        dp.close()
        del dp
    torch.cuda.empty_cache()
    assert free0 - torch.cuda.mem_get_info()[0] < (64 << 20)      # nothing of the 40 handles is left behind


def test_parts_match_oracle_on_their_token_ranges():
    cfg = SMALL["cfg2s"]
    hp = wl.make_host_problem(cfg)
    q = wl.draw_q(cfg, 0)
    dp = DeviceProblem.from_host(hp)
    o_part, lse_part = dp.new_parts()
    qd = to_device(cfg, q)
    mc.mc_prefix_attn(dp.layout, qd, cfg.scale, o_part, lse_part)
    mc.mc_suffix_attn(dp.layout, qd, cfg.scale, o_part, lse_part)
    torch.cuda.synchronize()
    g = dp.geom
    op, lp = o_part.cpu().numpy().astype(np.float64), lse_part.cpu().numpy().astype(np.float64)
    assert not np.isnan(lp).any()                      # every part slot was written
    rng = np.random.default_rng(0)
    for _ in range(40):
        b, hq = int(rng.integers(cfg.B)), int(rng.integers(cfg.Hq))
        h, row = hq // cfg.g, b * cfg.Hq + hq
        for part in range(g.n_parts):
            if part < g.n_prefix_parts:
                K, V = hp.k_prefix[0][:, h], hp.v_prefix[0][:, h]
                T = g.prefix_part_tokens              # part k = tokens [kT, (k+1)T)
                idx = np.arange(part * T, min((part + 1) * T, K.shape[0]))
            else:
                K, V = hp.k_suffix[b][:, h], hp.v_suffix[b][:, h]
                lo = (part - g.n_prefix_parts) * g.suffix_part_tokens
                idx = np.arange(lo, min(lo + g.suffix_part_tokens, K.shape[0]))
            if len(idx):
                o_ref, lse_ref = orc.attend(q[b, hq], K[idx], V[idx], cfg.scale)
            else:
                o_ref, lse_ref = np.zeros(cfg.d), -np.inf
            if lse_ref == -np.inf:
                assert lp[row, part] == -np.inf
            else:
                assert abs(lp[row, part] - lse_ref) <= 1e-3
                assert np.abs(op[row, part] - o_ref).max() <= 2e-2
    # merging the GPU's partials with the oracle's merge reproduces the oracle's full result
    o_ref, lse_ref = oracle_full(hp, q, rows=[(1, 3)])
    om, lm = orc.merge_partials(op[1 * cfg.Hq + 3], lp[1 * cfg.Hq + 3])
    assert np.abs(om - o_ref[1, 3]).max() <= 2e-2 and abs(lm - lse_ref[1, 3]) <= 1e-3
    dp.close()


@pytest.mark.parametrize("name", ["cfg0", "cfg1"])
def test_merge_alone_against_oracle_merge(name):
    cfg = SMALL[name]
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    g = dp.geom
    rng = np.random.default_rng(5)
    op = rng.normal(size=(g.rows, g.n_parts, g.head_dim)).astype(np.float32)
    lp = (rng.normal(size=(g.rows, g.n_parts)) * 4).astype(np.float32)
    lp[rng.random(size=lp.shape) < 0.3] = -np.inf
    lp[0, :] = -np.inf                                  # a row with no tokens at all
    lp[1, 1:] = -np.inf                                 # a row with exactly one part
    lp[2, 0] = 80.0                                     # one dominant part
    op[np.isneginf(lp)] = np.nan                        # empty parts carry garbage that must not leak
    mc.mc_merge_lse(dp.layout, torch.from_numpy(op).cuda(), torch.from_numpy(lp).cuda(), dp.o, dp.lse)
    torch.cuda.synchronize()
    o, lse = dp.o.float().cpu().numpy().reshape(g.rows, -1), dp.lse.cpu().numpy().reshape(-1)
    tol = 1e-5 if cfg.dtype == "f32" else 2e-2
    for r in range(g.rows):
        o_ref, lse_ref = orc.merge_partials(op[r], lp[r])
        if lse_ref == -np.inf:
            assert lse[r] == -np.inf and (o[r] == 0).all()
        else:
            assert abs(lse[r] - lse_ref) <= 1e-3 * max(1.0, abs(lse_ref) / 50) and np.abs(o[r] - o_ref).max() <= tol
    dp.close()


EDGE = [
    # name, dtype, G, C, Hq, Hkv, d, prefix lengths, suffix lengths
    ("all-suffix-empty", "bf16", 1, 3, 8, 2, 128, [33], [0, 0, 0]),
    ("prefix-one-token", "bf16", 1, 2, 8, 1, 128, [1], [0, 5]),
    ("chunk-boundaries", "bf16", 1, 6, 16, 2, 128, [256], [15, 16, 17, 255, 256, 257]),
    ("mha-g1", "bf16", 1, 2, 4, 4, 128, [70], [40, 300]),
    ("g2", "bf16", 2, 2, 4, 2, 128, [100, 17], [3, 0, 290, 31]),
    ("g16-falls-back", "bf16", 1, 2, 16, 1, 128, [50], [10, 90]),
    ("d64-bf16", "bf16", 1, 2, 8, 2, 64, [50], [10, 90]),
    ("f32-d128", "f32", 2, 2, 4, 2, 128, [40, 300], [0, 1, 16, 700]),
    ("single-candidate", "bf16", 1, 1, 8, 1, 128, [512], [513]),
    ("empty-prefix", "bf16", 1, 2, 8, 2, 128, [0], [20, 0]),
]


@pytest.mark.parametrize("case", EDGE, ids=[c[0] for c in EDGE])
def test_edge_shapes(case):
    name, dtype, G, C, Hq, Hkv, d, pl, sl = case
    cfg = wl.Config(name, dtype, G, C, Hq, Hkv, d, ("fixed", 0), ("fixed", tuple(sl)), permute_pages=True, seed=3)
    hp = wl.make_host_problem(cfg, prefix_len=np.array(pl, dtype=np.int32), suffix_len=np.array(sl, dtype=np.int32))
    q = wl.draw_q(cfg, 0)
    dp, o, lse = run_decode(hp, q)
    o_ref, lse_ref = oracle_full(hp, q)
    check_close(cfg, o, lse, o_ref, lse_ref)
    if name == "empty-prefix":                          # candidate 1 has no tokens at all
        assert torch.isneginf(lse[1]).all() and (o[1] == 0).all()
    dp.close()


def test_rising_scores_force_accumulator_rescale():
    """Keys whose scores grow by far more than 2^8 from one 128-token tile to the next: the tensor-core prefix
    pass must rescale its running accumulator (and the other paths their online softmax) and still match."""
    cfg = wl.Config("rising", "bf16", 1, 16, 64, 8, 128, ("fixed", 0), ("fixed", tuple([40] * 16)), permute_pages=True,
                    seed=5)
    hp = wl.make_host_problem(cfg, prefix_len=np.array([1100], dtype=np.int32))
    # scale the logical keys tile by tile (x1, x6, x1, x14, ...) and rebuild the paged image from them
    mult = np.ones(1100, dtype=np.float32)
    for t, f in enumerate([1, 6, 1, 14, 3, 20, 2, 9, 1]):
        mult[t * 128:(t + 1) * 128] = f
    hp.k_prefix[0] = wl._round_to_dtype(cfg, hp.k_prefix[0] * mult[:, None, None])
    wl._scatter(hp.k_pool, hp.tables.prefix_pages[0], hp.k_prefix[0], cfg)
    q = wl.draw_q(cfg, 0)
    dp, o, lse = run_decode(hp, q)
    check_close(cfg, o, lse, *oracle_full(hp, q))
    dp.close()


@pytest.mark.parametrize("scale", [-0.09, 0.0, 0.5])
def test_other_scales(scale):
    """Negative scale (the row extremum is then a minimum), zero scale (uniform weights) and a large one."""
    cfg = SMALL["cfg2s"]
    hp = wl.make_host_problem(cfg)
    q = wl.draw_q(cfg, 0)
    dp = DeviceProblem.from_host(hp)
    o, lse = dp.decode(to_device(cfg, q), scale=scale)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    o_ref, lse_ref = orc.decode_attention(q, hp.k_prefix, hp.v_prefix, hp.k_suffix, hp.v_suffix,
                                          hp.tables.group_offsets.tolist(), scale)
    check_close(cfg, o, lse, o_ref, lse_ref)
    dp.close()


@pytest.mark.parametrize("pairs", ["1", "0"])
@pytest.mark.parametrize("root", [0, 300])
def test_several_row_tiles_and_several_prefix_splits(monkeypatch, root, pairs):
    """44 candidates x 8 heads per kv head = 352 stacked rows (three 128-row tiles, the last partly filled) over a
    ragged 613-token prefix cut into three splits, every row checked; `root` > 0 puts a prompt shared by all
    candidates in front (a two-level cascade whose levels have different splits).  pairs = 1: the row-pair prefix
    kernel (the second pair of row tiles has one tile only); pairs = 0: one row tile per item."""
    monkeypatch.setenv("MC_PREFIX_PART_TOKENS", "256")
    monkeypatch.setenv("MC_PREFIX_PAIRS", pairs)
    cfg = wl.Config("tiles", "bf16", 1, 44, 64, 8, 128, ("fixed", 613), ("uniform", 0, 90), permute_pages=True, seed=11)
    hp = wl.make_host_problem(cfg)
    if root:
        wl.add_outer_level(hp, [0, cfg.B], [root], 0)
    dp = DeviceProblem.from_host(hp)
    assert dp.geom.prefix_ctas > 0 and dp.geom.prefix_part_tokens == 256 and dp.geom.n_prefix_parts >= 3 + (2 if root else 0)
    q = wl.draw_q(cfg, 0)
    o, lse = dp.decode(to_device(cfg, q))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    if root:
        levels = [(lv.k, lv.v, lv.group_offsets.tolist()) for lv in hp.outer]
        levels.append((hp.k_prefix, hp.v_prefix, hp.tables.group_offsets.tolist()))
        ref = orc.decode_attention_cascade(q, levels, hp.k_suffix, hp.v_suffix, cfg.scale)
    else:
        ref = oracle_full(hp, q)
    check_close(cfg, o, lse, *ref)
    dp.close()


@pytest.mark.parametrize("g", [4, 8, 1])
def test_bf16_head_dim_64_on_the_warp_level_tensor_path(g):
    """bf16 with d = 64 runs both passes on the warp-level MMA kernel (the tcgen05 and TMA-fed kernels are d = 128
    only): ragged prefixes, permuted pages, suffixes over several chunks, appends."""
    cfg = wl.Config("d64", "bf16", 3, 4, 2 * g, 2, 64, ("loguniform", 90, 1500), ("uniform", 0, 700), permute_pages=True,
                    append_steps=2, seed=21)
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    assert dp.geom.prefix_ctas == 0
    for step in range(3):
        q = wl.draw_q(cfg, step)
        if step:
            k_new, v_new = wl.draw_append(cfg, step)
            mc.mc_kv_append(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new))
            hp.append(k_new, v_new)
        o, lse = dp.decode(to_device(cfg, q))
        torch.cuda.synchronize()
        assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
        check_close(cfg, o, lse, *oracle_full(hp, q))
    dp.close()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_head_dim_256(dtype):
    """d = 256 runs on the plain-ALU kernel (the tensor-core kernels are built around 128-wide heads): ragged
    prefixes, permuted pages, several chunks, appends (plain and rotary), an outer cascade level."""
    from oracle import rope
    cfg = wl.Config("d256", dtype, 2, 3, 4, 2, 256, ("loguniform", 40, 700), ("uniform", 0, 500), permute_pages=True,
                    append_steps=3, seed=22)
    hp = wl.make_host_problem(cfg)
    wl.add_outer_level(hp, [0, cfg.B], [130])
    dp = DeviceProblem.from_host(hp)
    assert dp.geom.prefix_ctas == 0 and dp.geom.head_dim == 256

    def reference(q):
        levels = [(lv.k, lv.v, lv.group_offsets.tolist()) for lv in hp.outer]
        levels.append((hp.k_prefix, hp.v_prefix, hp.tables.group_offsets.tolist()))
        return orc.decode_attention_cascade(q, levels, hp.k_suffix, hp.v_suffix, cfg.scale)

    for step in range(4):
        q = wl.draw_q(cfg, step)
        if step in (1, 2):
            k_new, v_new = wl.draw_append(cfg, step)
            mc.mc_kv_append(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new))
            hp.append(k_new, v_new)
        if step == 3:          # a rotated key: the cache must hold what the rotation's definition gives
            k_new, v_new = wl.draw_append(cfg, step)
            pos = [130 + int(hp.prefix_len[b // cfg.C]) + int(hp.suffix_len[b]) for b in range(cfg.B)]
            mc.mc_kv_append_rope(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new), None, None, 10000.0)
            k_rot = np.stack([np.stack([rope.rope_rotate(k_new[b, h], pos[b], 10000.0) for h in range(cfg.Hkv)])
                              for b in range(cfg.B)])
            torch.cuda.synchronize()
            s_new = hp.suffix_len.copy()
            got = np.stack([dp.k_pool[int(hp.tables.suffix_pages[b, s_new[b] // 16]), :, s_new[b] % 16].float().cpu().numpy()
                            for b in range(cfg.B)])
            tol = (2.0 ** -8 if dtype == "bf16" else 2.0 ** -20) * np.abs(k_rot).max() * 2 + 1e-6
            assert np.abs(got - k_rot).max() <= tol
            hp.append(got.astype(np.float32), v_new)      # attention is checked on the rows the cache holds
        o, lse = dp.decode(to_device(cfg, q))
        torch.cuda.synchronize()
        assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
        check_close(cfg, o, lse, *reference(q))
    dp.close()


def test_unequal_group_sizes():
    cfg = wl.Config("unequal", "bf16", 2, 2, 8, 2, 128, ("fixed", 0), ("fixed", (5, 40, 0, 100)), seed=4)
    hp = wl.make_host_problem(cfg, prefix_len=np.array([64, 200], dtype=np.int32))
    hp.tables.group_offsets = np.array([0, 3, 4], dtype=np.int32)        # 3 candidates, then 1
    q = wl.draw_q(cfg, 0)
    dp, o, lse = run_decode(hp, q)
    check_close(cfg, o, lse, *oracle_full(hp, q))
    dp.close()


def test_forced_alu_path_matches_oracle(monkeypatch):
    """The plain-ALU split-KV kernels (no tensor cores) on a bf16 configuration."""
    monkeypatch.setenv("MC_FORCE_FMA", "1")
    cfg = SMALL["cfg2s"]
    hp = wl.make_host_problem(cfg)
    q = wl.draw_q(cfg, 0)
    dp, o, lse = run_decode(hp, q)
    check_close(cfg, o, lse, *oracle_full(hp, q))
    dp.close()


@pytest.mark.parametrize("name", ["cfg2s", "cfg3sp", "cfg4s"])
def test_warp_level_suffix_kernel_matches_oracle(monkeypatch, name):
    """The suffix pass on the register-fed warp-level kernel (the default is the TMA-fed one)."""
    monkeypatch.setenv("MC_SUFFIX_TMA", "0")
    cfg = SMALL[name]
    hp = wl.make_host_problem(cfg)
    q = wl.draw_q(cfg, 0)
    dp, o, lse = run_decode(hp, q)
    check_close(cfg, o, lse, *oracle_full(hp, q))
    dp.close()


@pytest.mark.parametrize("env", [{"MC_PDL": "0"}, {"MC_PREFIX_TC": "0"}, {"MC_SUFFIX_ORDER": "0"},
                                 {"MC_PREFIX_TC": "0", "MC_SUFFIX_TMA": "0"}, {"MC_PREFIX_CTAS": "3"}])
@pytest.mark.parametrize("name", ["cfg2s", "cfg3sp"])
def test_alternative_schedules_match_oracle(monkeypatch, env, name):
    """The same step on the library's other schedules: two streams instead of a programmatic dependent launch, the
    warp-level prefix pass, suffix items in plain order, both warp-level passes, a prefix grid of three CTAs (several
    items per CTA).  A decode step and an append step each."""
    for k, v in env.items():
        monkeypatch.setenv(k, v)
    cfg = SMALL[name]
    hp = wl.make_host_problem(cfg, headroom_tokens=4)
    q = wl.draw_q(cfg, 0)
    dp, o, lse = run_decode(hp, q)
    check_close(cfg, o, lse, *oracle_full(hp, q))
    k_new, v_new = wl.draw_append(cfg, 1)
    q = wl.draw_q(cfg, 1)
    mc.mc_decode_step(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new), to_device(cfg, q), cfg.scale, dp.o,
                      dp.lse, dp.ws_ptr, dp.ws_bytes)
    torch.cuda.synchronize()
    hp.append(k_new, v_new)
    check_close(cfg, dp.o, dp.lse, *oracle_full(hp, q))
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    dp.close()


@pytest.mark.parametrize("ts", [1024, 4096])
def test_long_suffix_chunks(monkeypatch, ts):
    """Chunks of more than 64 pages: the suffix kernel reloads its page-id registers on the way."""
    monkeypatch.setenv("MC_SUFFIX_PART_TOKENS", str(ts))
    cfg = SMALL["cfg4s"]
    hp = wl.make_host_problem(cfg)
    q = wl.draw_q(cfg, 0)
    dp, o, lse = run_decode(hp, q)
    assert dp.geom.suffix_part_tokens == ts
    check_close(cfg, o, lse, *oracle_full(hp, q))
    dp.close()


@pytest.mark.parametrize("tp,ts", [(16, 16), (64, 48), (4096, 4096)])
def test_result_does_not_depend_on_part_geometry(monkeypatch, tp, ts):
    monkeypatch.setenv("MC_PREFIX_PART_TOKENS", str(tp))
    monkeypatch.setenv("MC_SUFFIX_PART_TOKENS", str(ts))
    cfg = SMALL["cfg3s"]
    hp = wl.make_host_problem(cfg)
    q = wl.draw_q(cfg, 0)
    dp, o, lse = run_decode(hp, q)
    assert dp.geom.prefix_part_tokens == tp and dp.geom.suffix_part_tokens == ts
    check_close(cfg, o, lse, *oracle_full(hp, q))
    dp.close()


def test_bad_page_id_is_reported_not_dereferenced():
    cfg = SMALL["cfg1"]
    hp = wl.make_host_problem(cfg)
    hp.tables.suffix_pages[2, 0] = hp.tables.num_pages + 7
    hp.tables.prefix_pages[0, 3] = -5
    dp = DeviceProblem.from_host(hp)
    dp.decode(to_device(cfg, wl.draw_q(cfg, 0)))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_ERR_INVALID_ARG
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK          # reading clears the word
    assert torch.isfinite(dp.o.float()).all()
    dp.close()


def test_validate_accepts_good_tables_and_rejects_aliased_pages():
    cfg = SMALL["cfg1"]
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    scratch = torch.empty(hp.tables.num_pages, dtype=torch.int32, device="cuda")
    assert mc.mc_kv_layout_validate(dp.layout, scratch, scratch.numel() * 4) == mc.MC_OK
    dp.close()
    hp.tables.suffix_pages[3, 0] = hp.tables.suffix_pages[4, 0]
    dp = DeviceProblem.from_host(hp)
    assert mc.mc_kv_layout_validate(dp.layout, scratch, scratch.numel() * 4) == mc.MC_ERR_INVALID_ARG
    assert mc.mc_kv_layout_validate(dp.layout, scratch, 4) == mc.MC_ERR_WORKSPACE_TOO_SMALL
    dp.close()


def test_host_errors_are_returned_immediately():
    cfg = SMALL["cfg0"]
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    q = to_device(cfg, wl.draw_q(cfg, 0))
    L = mc.lib()
    assert L.mc_decode_attn(dp.layout, q.data_ptr(), cfg.scale, dp.o.data_ptr(), dp.lse.data_ptr(), dp.ws_ptr,
                            dp.ws_bytes - 1, 0) == mc.MC_ERR_WORKSPACE_TOO_SMALL
    assert L.mc_decode_attn(dp.layout, q.data_ptr() + 4, cfg.scale, dp.o.data_ptr(), dp.lse.data_ptr(), dp.ws_ptr,
                            dp.ws_bytes, 0) == mc.MC_ERR_INVALID_ARG
    assert L.mc_decode_attn(dp.layout, 0, cfg.scale, dp.o.data_ptr(), dp.lse.data_ptr(), dp.ws_ptr, dp.ws_bytes,
                            0) == mc.MC_ERR_INVALID_ARG
    bad = mc.LayoutDesc.from_buffer_copy(dp.desc)
    bad.page_size = 48
    h = mc.c_void_p()
    assert L.mc_kv_layout_create(mc.byref(bad), mc.byref(h)) == mc.MC_ERR_UNSUPPORTED and not h.value
    bad = mc.LayoutDesc.from_buffer_copy(dp.desc)
    bad.num_q_heads = 3
    bad.num_kv_heads = 2
    assert L.mc_kv_layout_create(mc.byref(bad), mc.byref(h)) == mc.MC_ERR_INVALID_ARG
    dp.close()


def test_host_buffer_step_matches_device_step():
    cfg = SMALL["cfg2s"]
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    k_new, v_new = wl.draw_append(cfg, 1)
    q = wl.draw_q(cfg, 1)
    pin = lambda x: to_device(cfg, x, "cpu").pin_memory()
    o_h = torch.empty(cfg.B, cfg.Hq, cfg.d, dtype=dp.tdtype).pin_memory()
    lse_h = torch.empty(cfg.B, cfg.Hq, dtype=torch.float32).pin_memory()
    mc.mc_decode_step_host(dp.layout, pin(k_new), pin(v_new), pin(q), cfg.scale, o_h, lse_h, dp.ws_ptr, dp.ws_bytes)
    hp.append(k_new, v_new)
    check_close(cfg, o_h, lse_h, *oracle_full(hp, q))
    dp.close()


def test_launch_counter_counts_kernels():
    cfg = SMALL["cfg0"]
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    n0 = mc.mc_launch_count()
    dp.decode(to_device(cfg, wl.draw_q(cfg, 0)))
    assert mc.mc_launch_count() - n0 >= 3
    dp.close()


def test_step_is_capturable_in_a_cuda_graph_and_replays_with_growing_lengths():
    """append + decode enqueue only kernels, event records and stream waits, and read the lengths on the device:
    one captured step can be replayed for consecutive decode steps."""
    cfg = SMALL["cfg2s"]
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    q_buf = to_device(cfg, wl.draw_q(cfg, 0))
    k_buf, v_buf = (to_device(cfg, x) for x in wl.draw_append(cfg, 1))
    stream = torch.cuda.Stream()
    # one eager step on the capture stream first (lazy module loading must not happen during capture)
    with torch.cuda.stream(stream):
        mc.mc_decode_attn(dp.layout, q_buf, cfg.scale, dp.o, dp.lse, dp.ws_ptr, dp.ws_bytes, stream.cuda_stream)
    stream.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        mc.mc_kv_append(dp.layout, k_buf, v_buf, torch.cuda.current_stream().cuda_stream)
        mc.mc_decode_attn(dp.layout, q_buf, cfg.scale, dp.o, dp.lse, dp.ws_ptr, dp.ws_bytes,
                          torch.cuda.current_stream().cuda_stream)
    for step in range(1, 4):
        k_new, v_new = wl.draw_append(cfg, step)
        q = wl.draw_q(cfg, step)
        k_buf.copy_(to_device(cfg, k_new))
        v_buf.copy_(to_device(cfg, v_new))
        q_buf.copy_(to_device(cfg, q))
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        hp.append(k_new, v_new)
        check_close(cfg, dp.o, dp.lse, *oracle_full(hp, q))
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), hp.suffix_len)
    dp.close()
