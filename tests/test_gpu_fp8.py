"""The e4m3 KV cache with per-(page, kv head) scales on the GPU, through the C ABI, against the CPU oracle: attention
over the values the codes stand for at the bf16 tolerances (max-abs 2e-2, mean-abs 2e-3, lse 1e-3), and the
quantising append bit for bit (codes and scales are integer / exactly defined decisions)."""
import numpy as np
import pytest
import torch

from oracle import attention as orc
from oracle import fp8
from paper_2601_05475_b200 import binding as mc
from paper_2601_05475_b200 import workload as wl
from paper_2601_05475_b200.harness import (DeviceProblem, device_append, device_q, logical_rows, make_device_problem,
                                           to_device)

from fp8_problem import make as make_fp8

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)


def device_problem(fp: "fp8_problem.Fp8HostProblem") -> DeviceProblem:
    dev = lambda a: torch.from_numpy(a).cuda()
    hp = fp.hp
    return DeviceProblem(fp.cfg, fp.tables, fp.prefix_len, fp.suffix_len, dev(fp.k_pool), dev(fp.v_pool),
                         outer=[(lv.group_offsets, lv.length, lv.pages) for lv in hp.outer],
                         k_scale=dev(fp.k_scale), v_scale=dev(fp.v_scale))


def oracle(fp, q):
    levels = list(fp.outer) + [(fp.k_prefix, fp.v_prefix, fp.tables.group_offsets.tolist())]
    return orc.decode_attention_cascade(q, levels, fp.k_suffix, fp.v_suffix, fp.cfg.scale)


def check(o, lse, o_ref, lse_ref):
    o = o.float().cpu().numpy().astype(np.float64)
    lse = lse.cpu().numpy().astype(np.float64)
    assert np.isfinite(o).all() and not np.isnan(lse).any()
    err = np.abs(o - o_ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())
    empty = np.isneginf(lse_ref)
    assert np.array_equal(np.isneginf(lse), empty)
    assert empty.all() or np.abs(lse[~empty] - lse_ref[~empty]).max() <= 1e-3


def as_fp8(cfg, name, **kw):
    import dataclasses
    return dataclasses.replace(wl.scaled_down(cfg, name, **kw), dtype="fp8")


CASES = {
    "cfg1": (as_fp8(wl.CONFIGS["cfg1"], "cfg1-fp8"), ()),
    "cfg2s": (as_fp8(wl.CONFIGS["cfg2"], "cfg2s-fp8", C=8, prefix=("fixed", 1040), suffix=("uniform", 0, 600),
                     append_steps=4), ()),
    # ragged prefixes, K outlier rows (x8: rows that saturate their page's range), permuted pages
    "cfg3s": (as_fp8(wl.CONFIGS["cfg3"], "cfg3s-fp8", G=3, C=4, prefix=("loguniform", 90, 1500),
                     suffix=("uniform", 0, 700), permute_pages=True), ()),
    # suffixes long enough for several blocks of 32 pages and several chunks
    "cfg4s": (as_fp8(wl.CONFIGS["cfg4"], "cfg4s-fp8", G=2, C=3, prefix=("fixed", 512), suffix=("uniform", 1000, 2100),
                     append_steps=2), ()),
    # a three-level cascade
    "cascade": (as_fp8(wl.CONFIGS["cfg1"], "casc-fp8", G=4, C=8, prefix=("loguniform", 100, 900),
                       suffix=("uniform", 0, 300)), [([0, 32], [700]), ([0, 24, 32], [333, 130])]),
}


@pytest.mark.parametrize("tc", ["1", "0"])
@pytest.mark.parametrize("name", list(CASES))
def test_fp8_decode_matches_oracle(name, tc, monkeypatch):
    """tc = 1: the prefix levels run on the tensor-core pass over their widened copy (where the shape allows it);
    tc = 0: every candidate streams its group's e4m3 pages itself."""
    monkeypatch.setenv("MC_PREFIX_TC", tc)
    cfg, outer = CASES[name]
    fp = make_fp8(cfg, outer)
    dp = device_problem(fp)
    scratch = torch.empty(fp.tables.num_pages, dtype=torch.int32, device="cuda")
    assert mc.mc_kv_layout_validate(dp.layout, scratch, scratch.numel() * 4) == mc.MC_OK
    assert (dp.geom.prefix_ctas > 0) == (tc == "1")
    q = wl.draw_q(cfg, 0)
    o, lse = dp.decode(to_device(cfg, q))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    check(o, lse, *oracle(fp, q))
    dp.close()


def test_fp8_prefix_changes_take_effect_after_a_refresh():
    """The tensor-core prefix pass reads a widened copy of the prefix made when the layout was created: after the
    prefix pages change, mc_kv_layout_refresh_prefix brings the copy up to date."""
    cfg, _ = CASES["cfg2s"]
    fp = make_fp8(cfg)
    dp = device_problem(fp)
    assert dp.geom.prefix_ctas > 0
    q = wl.draw_q(cfg, 0)
    qd = to_device(cfg, q)
    dp.decode(qd)
    torch.cuda.synchronize()
    check(dp.o, dp.lse, *oracle(fp, q))
    # the first three prefix pages get V = 0 (code 0) and K scales twice as large
    for i in range(3):
        pid = int(fp.tables.prefix_pages[0, i])
        dp.v_pool[pid] = 0
        dp.k_scale[pid] *= 2
        fp.v_prefix[0][16 * i:16 * i + 16] = 0.0
        fp.k_prefix[0][16 * i:16 * i + 16] *= 2.0
    mc.mc_kv_layout_refresh_prefix(dp.layout)
    dp.decode(qd)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    check(dp.o, dp.lse, *oracle(fp, q))
    dp.close()


@pytest.mark.parametrize("ts", [0, 64])
def test_fp8_append_is_bit_exact_and_the_sweep_matches_oracle(ts, monkeypatch):
    """40 decode steps: every candidate crosses page boundaries (new scales) at its own step; appended K rows three
    times as large as usual (and two elements of the V rows) saturate against the scale their page already has; with
    64-token chunks appends open chunks that were empty when the layout was made."""
    if ts:
        monkeypatch.setenv("MC_SUFFIX_PART_TOKENS", str(ts))
    cfg = as_fp8(wl.CONFIGS["cfg2"], "sweep-fp8", C=6, prefix=("fixed", 200), suffix=("fixed", (0, 32, 64, 31, 96, 33)),
                 append_steps=40)
    fp = make_fp8(cfg, headroom_tokens=48)
    dp = device_problem(fp)
    for step in range(1, 41):
        k_new, v_new = wl.draw_append(cfg, step)
        if step % 7 == 3:
            k_new = wl._round_to_dtype(cfg, 3 * k_new)
            v_new[:, :, [5, 77]] = wl._round_to_dtype(cfg, 3 * v_new[:, :, [5, 77]])
        q = wl.draw_q(cfg, step)
        mc.mc_decode_step(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new), to_device(cfg, q), cfg.scale,
                          dp.o, dp.lse, dp.ws_ptr, dp.ws_bytes)
        fp.append(k_new, v_new)
        if step in (1, 2, 16, 17, 33, 40):
            torch.cuda.synchronize()
            check(dp.o, dp.lse, *oracle(fp, q))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), fp.suffix_len)
    # the cache itself: every code and every scale as the oracle's quantiser makes them
    used = np.unique(np.concatenate([fp.tables.suffix_pages[b, :(int(fp.suffix_len[b]) + 15) // 16] for b in range(cfg.B)]))
    np.testing.assert_array_equal(dp.k_scale.cpu().numpy()[used], fp.k_scale[used])
    np.testing.assert_array_equal(dp.v_scale.cpu().numpy()[used], fp.v_scale[used])
    kd, vd = dp.k_pool.cpu().numpy(), dp.v_pool.cpu().numpy()
    for b in range(cfg.B):
        n = int(fp.suffix_len[b])
        for t in range(n):
            pid = int(fp.tables.suffix_pages[b, t // 16])
            np.testing.assert_array_equal(kd[pid, :, t % 16], fp.k_pool[pid, :, t % 16])
            np.testing.assert_array_equal(vd[pid, :, t % 16], fp.v_pool[pid, :, t % 16])
    # some appended rows did saturate (the test would not notice a missing clamp otherwise)
    assert (kd[used] & 0x7F).max() == 0x7E and (vd[used] & 0x7F).max() == 0x7E
    # a full row is refused and reported
    for _ in range(wl.PAGE + 1):
        mc.mc_kv_append(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new))
    assert mc.mc_get_last_status(dp.layout) == mc.MC_ERR_INVALID_ARG
    dp.close()


def test_fp8_bad_page_and_host_errors():
    cfg, _ = CASES["cfg2s"]
    fp = make_fp8(cfg)
    dp = device_problem(fp)
    q = to_device(cfg, wl.draw_q(cfg, 0))
    bad = mc.LayoutDesc.from_buffer_copy(dp.desc)
    bad.k_scale = 0
    with pytest.raises(mc.McError) as e:
        mc.mc_kv_layout_create(bad)
    assert e.value.status == mc.MC_ERR_INVALID_ARG
    bad = mc.LayoutDesc.from_buffer_copy(dp.desc)
    bad.head_dim = 64
    with pytest.raises(mc.McError) as e:
        mc.mc_kv_layout_create(bad)
    assert e.value.status == mc.MC_ERR_UNSUPPORTED
    with pytest.raises(mc.McError) as e:
        mc.mc_kv_append_rope(dp.layout, q, q, None, None, 1e4)
    assert e.value.status == mc.MC_ERR_UNSUPPORTED
    # a page id outside the pool: skipped, reported, the rest of the row still finite
    dp.suffix_pages[2, 0] = fp.tables.num_pages + 3
    o, lse = dp.decode(q)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_ERR_INVALID_ARG
    assert torch.isfinite(o.float()).all()
    dp.close()


def test_fp8_full_size_cfg4_sampled_rows():
    """Configuration 4 with an e4m3 cache, as the benchmark times it: sampled rows are read back through the page
    tables (codes and scales), decoded by the oracle and attended in fp64; a few appended steps follow."""
    import dataclasses
    cfg = dataclasses.replace(wl.CONFIGS["cfg4"], name="cfg4-fp8", dtype="fp8")
    dp = make_device_problem(cfg, headroom_tokens=5)

    def check_rows(q, seed):
        rng = np.random.default_rng(seed)
        rows = [(int(rng.integers(cfg.B)), int(rng.integers(cfg.Hq))) for _ in range(8)] + [(0, 0), (cfg.B - 1, cfg.Hq - 1)]
        errs, lerrs = [], []
        for (b, hq) in rows:
            (kc, ks), (vc, vs) = logical_rows(dp, b, hq // cfg.g)
            K = fp8.e4m3_decode(kc) * ks[:, None].astype(np.float64)
            V = fp8.e4m3_decode(vc) * vs[:, None].astype(np.float64)
            o_ref, lse_ref = orc.attend(q[b, hq].float().cpu().numpy(), K, V, cfg.scale)
            errs.append(np.abs(dp.o[b, hq].float().cpu().numpy().astype(np.float64) - o_ref))
            lerrs.append(abs(float(dp.lse[b, hq]) - lse_ref))
        errs = np.stack(errs)
        assert errs.max() <= 2e-2 and errs.mean() <= 2e-3 and np.max(lerrs) <= 1e-3, (errs.max(), errs.mean(), np.max(lerrs))

    q = device_q(cfg, 0)
    dp.decode(q)
    torch.cuda.synchronize()
    assert torch.isfinite(dp.o.float()).all() and torch.isfinite(dp.lse).all()
    check_rows(q, 1)
    len0 = dp.suffix_len.clone()
    for step in range(1, 4):
        k_new, v_new = device_append(cfg, step)
        q = device_q(cfg, step)
        mc.mc_decode_step(dp.layout, k_new, v_new, q, cfg.scale, dp.o, dp.lse, dp.ws_ptr, dp.ws_bytes)
    torch.cuda.synchronize()
    assert torch.equal(dp.suffix_len, len0 + 3)
    check_rows(q, 2)
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    dp.close()
