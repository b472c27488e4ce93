"""mc_kv_append_tokens (several tokens per candidate in one call) through the C ABI against host models built from
the oracle's pieces: the cache rows bit for bit (bf16 / fp32 copies, e4m3 codes and scales) or within one unit in the
last place (rotated keys), the lengths, a decode step on top, and a prefill that writes what it then scores."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import attention as orc
from oracle import fp8
from oracle import rope
from paper_2601_05475_b200 import binding as mc
from paper_2601_05475_b200 import workload as wl
from paper_2601_05475_b200.harness import DeviceProblem, to_device

from fp8_problem import make as make_fp8
from test_gpu_fp8 import check as check_fp8, device_problem as fp8_device_problem, oracle as fp8_oracle

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

N_MAX = 37      # more than two pages: tokens of one call open pages themselves


def draw_tokens(cfg, seed):
    rng = np.random.default_rng(seed)
    shape = (cfg.B, N_MAX, cfg.Hkv, cfg.d)
    k = wl._round_to_dtype(cfg, rng.standard_normal(shape, dtype=np.float32))
    v = wl._round_to_dtype(cfg, rng.standard_normal(shape, dtype=np.float32))
    n = rng.integers(0, N_MAX + 1, size=cfg.B).astype(np.int32)
    n[0], n[-1] = N_MAX, 0
    return k, v, n


def check_decode(cfg, dp, hp, step):
    q = wl.draw_q(cfg, step)
    o, lse = dp.decode(to_device(cfg, q))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    o_ref, lse_ref = orc.decode_attention(q, hp.k_prefix, hp.v_prefix, hp.k_suffix, hp.v_suffix,
                                          hp.tables.group_offsets.tolist(), cfg.scale)
    err = np.abs(o.float().cpu().numpy().astype(np.float64) - o_ref)
    tol = (1e-5, 1e-5) if cfg.dtype == "f32" else (2e-2, 2e-3)
    assert err.max() <= tol[0] and err.mean() <= tol[1], (err.max(), err.mean())
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 1e-3


@pytest.mark.parametrize("name", ["bf16", "f32"])
def test_plain_append_of_many_tokens(name):
    cfg = {"bf16": wl.scaled_down(wl.CONFIGS["cfg2"], "many", C=8, prefix=("fixed", 300), suffix=("uniform", 0, 200)),
           "f32": wl.CONFIGS["cfg0"]}[name]
    hp = wl.make_host_problem(cfg, headroom_tokens=2 * N_MAX)
    dp = DeviceProblem.from_host(hp)
    for call in range(2):
        k, v, n = draw_tokens(cfg, 10 + call)
        s0 = hp.suffix_len.copy()
        mc.mc_kv_append_tokens(dp.layout, to_device(cfg, k), to_device(cfg, v), N_MAX, torch.from_numpy(n).cuda())
        torch.cuda.synchronize()
        assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
        for b in range(cfg.B):
            hp.k_suffix[b] = np.concatenate([hp.k_suffix[b], k[b, :n[b]]], axis=0)
            hp.v_suffix[b] = np.concatenate([hp.v_suffix[b], v[b, :n[b]]], axis=0)
            hp.suffix_len[b] += n[b]
        np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), s0 + n)
        # the rows as they sit in the pages
        kp = dp.k_pool.float().cpu().numpy()
        vp = dp.v_pool.float().cpu().numpy()
        for b in range(cfg.B):
            for t in range(n[b]):
                s = s0[b] + t
                pid = hp.tables.suffix_pages[b, s // 16]
                np.testing.assert_array_equal(kp[pid, :, s % 16], k[b, t])
                np.testing.assert_array_equal(vp[pid, :, s % 16], v[b, t])
        check_decode(cfg, dp, hp, call)
    # NULL counts: every candidate gets n_max tokens; here that overflows candidate rows: refused and reported
    k, v, _ = draw_tokens(cfg, 99)
    before = dp.suffix_len.clone()
    mc.mc_kv_append_tokens(dp.layout, to_device(cfg, k), to_device(cfg, v), N_MAX)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_ERR_INVALID_ARG
    b4 = before.cpu().numpy()
    full = np.array([b4[b] + N_MAX > hp.tables.max_suffix_pages * 16 or
                     (hp.tables.suffix_pages[b, b4[b] // 16:(b4[b] + N_MAX - 1) // 16 + 1] < 0).any() for b in range(cfg.B)])
    assert full.any()
    np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), before.cpu().numpy() + np.where(full, 0, N_MAX))
    with pytest.raises(mc.McError):       # the rotation's arguments without a rotation
        mc.mc_kv_append_tokens(dp.layout, to_device(cfg, k), to_device(cfg, v), N_MAX, None, to_device(cfg, k))
    dp.close()


def test_rotary_append_of_many_tokens():
    cfg = wl.scaled_down(wl.CONFIGS["cfg2"], "manyrope", C=4, prefix=("fixed", 300), suffix=("uniform", 0, 200))
    base = 10000.0
    hp = wl.make_host_problem(cfg, headroom_tokens=N_MAX)
    dp = DeviceProblem.from_host(hp)
    k, v, n = draw_tokens(cfg, 21)
    q = wl._round_to_dtype(cfg, np.random.default_rng(5).standard_normal((cfg.B, N_MAX, cfg.Hq, cfg.d), dtype=np.float32))
    s0 = hp.suffix_len.copy()
    q_dev = to_device(cfg, q)
    mc.mc_kv_append_tokens(dp.layout, to_device(cfg, k), to_device(cfg, v), N_MAX, torch.from_numpy(n).cuda(), q_dev,
                           None, base)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    kp = dp.k_pool.float().cpu().numpy()
    q_got = q_dev.float().cpu().numpy()
    half = cfg.d // 2
    for b in range(cfg.B):
        for t in range(n[b]):
            s = s0[b] + t
            pos = int(hp.prefix_len[b // cfg.C]) + int(s)
            pid = hp.tables.suffix_pages[b, s // 16]
            for rows_got, rows_in in ((kp[pid, :, s % 16], k[b, t]), (q_got[b, t], q[b, t])):
                for h in range(rows_in.shape[0]):
                    ref = rope.rope_rotate(rows_in[h], pos, base)
                    mag = np.hypot(ref[:half], ref[half:])
                    tol = np.concatenate([mag, mag]) * 2.0 ** -8 + 1e-6       # one unit in the last place of bf16
                    assert (np.abs(rows_got[h] - ref) <= tol).all()
        # tokens beyond the candidate's count are untouched
        np.testing.assert_array_equal(q_got[b, n[b]:], q[b, n[b]:])
    np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), s0 + n)
    dp.close()


def test_e4m3_append_of_many_tokens_is_bit_exact():
    cfg = dataclasses.replace(wl.scaled_down(wl.CONFIGS["cfg2"], "many8", C=6, prefix=("fixed", 200),
                                             suffix=("fixed", (0, 5, 16, 31, 40, 64))), dtype="fp8")
    fp = make_fp8(cfg, headroom_tokens=2 * N_MAX)
    dp = fp8_device_problem(fp)
    for call in range(2):
        k, v, n = draw_tokens(cfg, 30 + call)
        k[:, 7] *= 3                               # rows that saturate against a scale fixed earlier in the same call
        k = wl._round_to_dtype(cfg, k)
        mc.mc_kv_append_tokens(dp.layout, to_device(cfg, k), to_device(cfg, v), N_MAX, torch.from_numpy(n).cuda())
        for t in range(N_MAX):                     # the host model appends token by token
            for b in range(cfg.B):
                if t < n[b]:
                    fp.append_one(b, k[b, t], v[b, t])
        torch.cuda.synchronize()
        assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
        np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), fp.suffix_len)
        kd, vd = dp.k_pool.cpu().numpy(), dp.v_pool.cpu().numpy()
        ks, vs = dp.k_scale.cpu().numpy(), dp.v_scale.cpu().numpy()
        for b in range(cfg.B):
            for s in range(int(fp.suffix_len[b])):
                pid = int(fp.tables.suffix_pages[b, s // 16])
                np.testing.assert_array_equal(kd[pid, :, s % 16], fp.k_pool[pid, :, s % 16])
                np.testing.assert_array_equal(vd[pid, :, s % 16], fp.v_pool[pid, :, s % 16])
                np.testing.assert_array_equal(ks[pid], fp.k_scale[pid])
                np.testing.assert_array_equal(vs[pid], fp.v_scale[pid])
        q = wl.draw_q(cfg, call)
        dp.decode(to_device(cfg, q))
        torch.cuda.synchronize()
        check_fp8(dp.o, dp.lse, *fp8_oracle(fp, q))
    dp.close()


def test_prefill_writes_the_tokens_it_then_scores():
    """Two prompt groups x three candidates: the candidates' whole continuations are appended in one call, then every
    appended token is scored (one query per token, causal inside the candidate) through a cascade layout laid over the
    same pools whose outer level IS the decode layout's suffix tables."""
    cfg = wl.Config("prefill", "bf16", 2, 3, 16, 4, 128, ("loguniform", 50, 300), ("fixed", (0,) * 6), permute_pages=True,
                    seed=14)
    hp = wl.make_host_problem(cfg, headroom_tokens=N_MAX)
    dp = DeviceProblem.from_host(hp)
    k, v, n = draw_tokens(cfg, 41)
    n[-1] = 20
    mc.mc_kv_append_tokens(dp.layout, to_device(cfg, k), to_device(cfg, v), N_MAX, torch.from_numpy(n).cuda())
    torch.cuda.synchronize()
    # every (candidate, position) becomes a virtual candidate of the scoring layout
    seq_offsets = np.concatenate([[0], np.cumsum(n)]).astype(np.int32)
    Bv = int(seq_offsets[-1])
    group_offsets = seq_offsets[::cfg.C].copy()
    row_limit = np.concatenate([np.arange(1, m + 1) for m in n]).astype(np.int32)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()
    t = {"go": dev(group_offsets), "so": dev(seq_offsets), "rl": dev(row_limit)}
    d = mc.LayoutDesc.from_buffer_copy(dp.desc)
    d.batch, d.max_suffix_pages, d.suffix_pages, d.suffix_len = Bv, 0, 0, 0
    d.group_offsets = t["go"].data_ptr()
    lv = mc.PrefixLevel()
    lv.num_groups, lv.max_pages = cfg.B, hp.tables.max_suffix_pages
    lv.group_offsets, lv.pages, lv.len = t["so"].data_ptr(), dp.suffix_pages.data_ptr(), dp.suffix_len.data_ptr()
    lv.row_limit = t["rl"].data_ptr()
    layout = mc.mc_kv_layout_create_cascade(d, [lv])
    q = [wl._round_to_dtype(cfg, np.random.default_rng(50 + b).standard_normal((int(n[b]), cfg.Hq, cfg.d), dtype=np.float32))
         for b in range(cfg.B)]
    o = torch.empty(Bv, cfg.Hq, cfg.d, dtype=torch.bfloat16, device="cuda")
    lse = torch.empty(Bv, cfg.Hq, dtype=torch.float32, device="cuda")
    ws_bytes = mc.mc_workspace_bytes(layout)
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    mc.mc_decode_attn(layout, to_device(cfg, np.concatenate(q, axis=0)), cfg.scale, o, lse,
                      (ws.data_ptr() + 255) // 256 * 256, ws_bytes)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(layout) == mc.MC_OK
    o_ref, lse_ref = orc.scoring_attention(q, hp.k_prefix, hp.v_prefix, [k[b, :n[b]] for b in range(cfg.B)],
                                           [v[b, :n[b]] for b in range(cfg.B)], [0, cfg.C, 2 * cfg.C], cfg.scale)
    o_ref, lse_ref = np.concatenate(o_ref, axis=0), np.concatenate(lse_ref, axis=0)
    err = np.abs(o.float().cpu().numpy().astype(np.float64) - o_ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 1e-3
    mc.mc_kv_layout_destroy(layout)
    dp.close()
