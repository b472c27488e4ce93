"""The fused q/k/v projection + rotary embedding + append (mc_qkv_append) against the fp64 oracle (oracle/qkv.py),
element by element.

Tolerance.  The kernel multiplies bf16 operands exactly, sums in fp32 and rounds each output to bf16 once, after the
rotation.  Against the exact result y that leaves (a) the final rounding, at most 2^-9 of the output's magnitude -
for a rotated pair the magnitude of the pair, since the rotation is done on fp32 values and either component of the
result may be small - and (b) the error of the fp32 summation and rotation, bounded by a small multiple of
2^-24 * sum_i |x_i| |w_i| per feature (the forward error bound of a dot product, here with blocked partial sums).
The test allows 2^-8 * magnitude + 2^-18 * sum_i |x_i| |w_i| (the second term is about 2 * 10^-4 at hidden 4096)."""
import numpy as np
import pytest
import torch

from oracle import attention as orc
from oracle import qkv as oqkv
from paper_2601_05475_b200 import binding as mc
from paper_2601_05475_b200 import workload as wl
from paper_2601_05475_b200.harness import DeviceProblem, to_device

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

BASE = 10000.0


def bf16_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).cuda()


def tolerance(ref, x, w, Hq, Hkv, d, rotated):
    """Per element [B][N]: 2^-8 * magnitude (of the pair, where the head was rotated) + 2^-18 * sum |x||w|."""
    B = ref.shape[0]
    heads = ref.reshape(B, Hq + 2 * Hkv, d)
    mag = np.abs(heads).copy()
    if rotated:
        pair = np.hypot(heads[:, :Hq + Hkv, :d // 2], heads[:, :Hq + Hkv, d // 2:])
        mag[:, :Hq + Hkv] = np.concatenate([pair, pair], axis=-1)
    return mag.reshape(B, -1) * 2.0 ** -8 + oqkv.abs_dot(x, w) * 2.0 ** -18 + 1e-6


def pool_rows(dp, hp, b, s):
    page = hp.cfg.page
    pid, slot = int(hp.tables.suffix_pages[b, s // page]), s % page
    return dp.k_pool[pid, :, slot].float().cpu().numpy(), dp.v_pool[pid, :, slot].float().cpu().numpy()


def run_case(cfg, hidden, bias, base, headroom=4, pos_offset=None, steps=1):
    hp = wl.make_host_problem(cfg, headroom_tokens=headroom)
    dp = DeviceProblem.from_host(hp)
    w, b = wl.draw_qkv_weights(cfg, hidden, with_bias=bias)
    w_dev, b_dev = bf16_dev(w), (bf16_dev(b) if bias else None)
    plan = mc.mc_qkv_plan_create(dp.layout, w_dev, b_dev, hidden)
    q_out = torch.empty(cfg.B, cfg.Hq, cfg.d, dtype=torch.bfloat16, device="cuda")
    N = (cfg.Hq + 2 * cfg.Hkv) * cfg.d
    po_dev = torch.from_numpy(pos_offset.astype(np.int32)).cuda() if pos_offset is not None else None
    for step in range(steps):
        x = wl.draw_hidden(cfg, step, hidden)
        s0 = hp.suffix_len.copy()
        pos = (pos_offset if pos_offset is not None else np.repeat(hp.prefix_len, cfg.C)) + s0
        mc.mc_qkv_append(plan, bf16_dev(x), q_out, po_dev, base)
        torch.cuda.synchronize()
        assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
        q_ref, k_ref, v_ref = oqkv.qkv_step(x, w, b, pos, base, cfg.Hq, cfg.Hkv, cfg.d)
        ref = np.concatenate([q_ref.reshape(cfg.B, -1), k_ref.reshape(cfg.B, -1), v_ref.reshape(cfg.B, -1)], axis=1)
        # the unrotated projection is what the magnitudes of the error bound refer to
        tol = tolerance(oqkv.project(x, w, b), x, w, cfg.Hq, cfg.Hkv, cfg.d, base > 0)
        got = np.zeros((cfg.B, N))
        got[:, :cfg.Hq * cfg.d] = q_out.float().cpu().numpy().reshape(cfg.B, -1)
        for bb in range(cfg.B):
            kr, vr = pool_rows(dp, hp, bb, int(s0[bb]))
            got[bb, cfg.Hq * cfg.d:(cfg.Hq + cfg.Hkv) * cfg.d] = kr.ravel()
            got[bb, (cfg.Hq + cfg.Hkv) * cfg.d:] = vr.ravel()
        err = np.abs(got - ref)
        assert (err <= tol).all(), (float((err / tol).max()), np.unravel_index(np.argmax(err / tol), err.shape))
        np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), s0 + 1)
        # host mirror: the suffix grows by the token as it now sits in the cache
        for bb in range(cfg.B):
            kr, vr = pool_rows(dp, hp, bb, int(s0[bb]))
            hp.k_suffix[bb] = np.concatenate([hp.k_suffix[bb], kr[None]], axis=0)
            hp.v_suffix[bb] = np.concatenate([hp.v_suffix[bb], vr[None]], axis=0)
        hp.suffix_len = hp.suffix_len + 1
    return dp, hp, plan, q_out


CASES = {
    # name: (config, hidden, bias, theta_base)
    "one_tile": (wl.scaled_down(wl.CONFIGS["cfg2"], "q1", C=8, prefix=("fixed", 300), suffix=("uniform", 0, 100)),
                 512, True, BASE),
    "ragged_rows": (wl.Config("q2", "bf16", 3, 37, 16, 4, 128, ("loguniform", 20, 400), ("uniform", 0, 60),
                              permute_pages=True), 320, False, BASE),             # 111 candidates, 5 k-blocks
    "two_tiles": (wl.Config("q3", "bf16", 2, 90, 16, 2, 128, ("fixed", 64), ("uniform", 0, 40), permute_pages=True),
                  1024, True, BASE),                                               # 180 candidates: two row tiles
    "two_passes": (wl.Config("q4", "bf16", 1, 300, 8, 2, 128, ("fixed", 32), ("uniform", 0, 20)), 256, True, BASE),
    "no_rotation": (wl.scaled_down(wl.CONFIGS["cfg2"], "q5", C=4, prefix=("fixed", 100), suffix=("uniform", 0, 50)),
                    256, True, 0.0),
    "model_width": (wl.scaled_down(wl.CONFIGS["cfg4"], "q6", G=1, C=16, prefix=("fixed", 128), suffix=("uniform", 0, 90)),
                    4096, False, 500000.0),                                        # 80 heads x 4096: 84 MB of weights
}


@pytest.mark.parametrize("name", list(CASES))
def test_projection_rotation_and_append_match_the_oracle(name):
    cfg, hidden, bias, base = CASES[name]
    dp, hp, plan, _ = run_case(cfg, hidden, bias, base)
    pieces, ctas, ws = mc.mc_qkv_plan_geometry(plan)
    assert pieces >= 1 and ctas >= 1 and ws > 0
    mc.mc_qkv_plan_destroy(plan)
    dp.close()


@pytest.mark.parametrize("ctas", ["1", "7", "33", "320"])
def test_result_does_not_depend_on_how_the_stream_is_shared_out(monkeypatch, ctas):
    """One CTA for everything, shares that end inside head pairs, one k-block per CTA (320 = 40 pairs x 8 k-blocks)."""
    monkeypatch.setenv("MC_QKV_CTAS", ctas)
    cfg, hidden, bias, base = CASES["one_tile"]
    dp, hp, plan, _ = run_case(cfg, hidden, bias, base)
    pieces, n, _ = mc.mc_qkv_plan_geometry(plan)
    assert n == int(ctas) and pieces == {"1": 1, "7": 2, "33": 2, "320": 8}[ctas]
    mc.mc_qkv_plan_destroy(plan)
    dp.close()


def test_positions_from_the_caller_and_several_steps_feed_the_attention():
    """Three fused steps with caller-given position offsets, each followed by the attention over the grown cache
    with the queries the projection wrote: the whole decode layer front to back against the oracles."""
    cfg = wl.Config("q7", "bf16", 2, 6, 16, 2, 128, ("fixed", 200), ("fixed", (0, 15, 16, 31, 47, 5)), permute_pages=True)
    hidden = 384
    pos_offset = np.arange(cfg.B) * 1000 + 7
    hp = wl.make_host_problem(cfg, headroom_tokens=4)
    dp = DeviceProblem.from_host(hp)
    w, b = wl.draw_qkv_weights(cfg, hidden)
    w_dev, b_dev = bf16_dev(w), bf16_dev(b)
    plan = mc.mc_qkv_plan_create(dp.layout, w_dev, b_dev, hidden)
    q_out = torch.empty(cfg.B, cfg.Hq, cfg.d, dtype=torch.bfloat16, device="cuda")
    po = torch.from_numpy(pos_offset.astype(np.int32)).cuda()
    for step in range(3):
        x = wl.draw_hidden(cfg, step, hidden)
        s0 = hp.suffix_len.copy()
        mc.mc_qkv_append(plan, bf16_dev(x), q_out, po, BASE)
        o, lse = dp.decode(q_out)
        torch.cuda.synchronize()
        assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
        q_ref, k_ref, v_ref = oqkv.qkv_step(x, w, b, pos_offset + s0, BASE, cfg.Hq, cfg.Hkv, cfg.d)
        # the attention is checked on the inputs the device actually holds (bf16 q and cache rows): its own
        # tolerance is about its own arithmetic, the projection's error was checked above
        q_got = q_out.float().cpu().numpy()
        assert np.abs(q_got - q_ref).max() <= 2.0 ** -7 * np.abs(q_ref).max() + 1e-3
        for bb in range(cfg.B):
            kr, vr = pool_rows(dp, hp, bb, int(s0[bb]))
            assert np.abs(kr - k_ref[bb]).max() <= 2.0 ** -7 * np.abs(k_ref[bb]).max() + 1e-3
            assert np.abs(vr - v_ref[bb]).max() <= 2.0 ** -7 * np.abs(v_ref[bb]).max() + 1e-3
            hp.k_suffix[bb] = np.concatenate([hp.k_suffix[bb], kr[None]], axis=0)
            hp.v_suffix[bb] = np.concatenate([hp.v_suffix[bb], vr[None]], axis=0)
        hp.suffix_len = hp.suffix_len + 1
        o_ref, lse_ref = orc.decode_attention(q_got, hp.k_prefix, hp.v_prefix, hp.k_suffix, hp.v_suffix,
                                              hp.tables.group_offsets.tolist(), cfg.scale)
        err = np.abs(o.float().cpu().numpy() - o_ref)
        assert err.max() <= 2e-2 and err.mean() <= 2e-3
        assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 1e-3
    mc.mc_qkv_plan_destroy(plan)
    dp.close()


def test_full_rows_get_their_query_but_no_token():
    cfg = wl.Config("q8", "bf16", 1, 4, 16, 2, 128, ("fixed", 40), ("fixed", (16, 3, 32, 9)))
    hidden = 128
    hp = wl.make_host_problem(cfg, headroom_tokens=0)       # candidates 0 and 2 end exactly on a page: no room left
    dp = DeviceProblem.from_host(hp)
    w, _ = wl.draw_qkv_weights(cfg, hidden, with_bias=False)
    w_dev = bf16_dev(w)                                     # borrowed by the plan: must stay alive
    plan = mc.mc_qkv_plan_create(dp.layout, w_dev, None, hidden)
    x = wl.draw_hidden(cfg, 0, hidden)
    q_out = torch.zeros(cfg.B, cfg.Hq, cfg.d, dtype=torch.bfloat16, device="cuda")
    before_k = dp.k_pool.clone()
    mc.mc_qkv_append(plan, bf16_dev(x), q_out, None, BASE)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_ERR_INVALID_ARG
    np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), hp.suffix_len + np.array([0, 1, 0, 1]))
    pos = np.repeat(hp.prefix_len, cfg.C) + hp.suffix_len
    q_ref, _, _ = oqkv.qkv_step(x, w, None, pos, BASE, cfg.Hq, cfg.Hkv, cfg.d)
    assert np.abs(q_out.float().cpu().numpy() - q_ref).max() <= 2.0 ** -7 * np.abs(q_ref).max() + 1e-3
    changed = (dp.k_pool != before_k).any(dim=-1).any(dim=1).nonzero().cpu().numpy()       # (page, slot) pairs written
    expect = sorted((int(hp.tables.suffix_pages[b, hp.suffix_len[b] // 16]), int(hp.suffix_len[b] % 16)) for b in (1, 3))
    assert sorted(map(tuple, changed.tolist())) == expect
    mc.mc_qkv_plan_destroy(plan)
    dp.close()


def test_expired_wait_is_reported_and_the_next_call_is_correct(monkeypatch):
    """The product's waits (for a copy, for the tensor pipe, for the epilogue) are bounded like those of the attention
    kernels: with a limit of zero cycles (read when the plan is made) the first wait that is not already satisfied
    gives up, MC_ERR_TIMEOUT is latched, every kernel returns, and a plan with the ordinary limit then works.
    Nothing is made to fault or to hang; what the expired call wrote is not looked at."""
    cfg, hidden, bias, base = CASES["one_tile"]
    hp = wl.make_host_problem(cfg, headroom_tokens=4)
    dp = DeviceProblem.from_host(hp)
    w, b = wl.draw_qkv_weights(cfg, hidden)
    w_dev, b_dev = bf16_dev(w), bf16_dev(b)
    monkeypatch.setenv("MC_WAIT_CYCLES", "0")
    plan = mc.mc_qkv_plan_create(dp.layout, w_dev, b_dev, hidden)
    q_out = torch.empty(cfg.B, cfg.Hq, cfg.d, dtype=torch.bfloat16, device="cuda")
    mc.mc_qkv_append(plan, bf16_dev(wl.draw_hidden(cfg, 0, hidden)), q_out, None, base)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_ERR_TIMEOUT
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    mc.mc_qkv_plan_destroy(plan)
    dp.close()
    monkeypatch.delenv("MC_WAIT_CYCLES")
    dp, hp, plan, _ = run_case(cfg, hidden, bias, base)
    mc.mc_qkv_plan_destroy(plan)
    dp.close()


def test_arguments_are_checked():
    cfg, hidden, _, _ = CASES["one_tile"]
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    w, _ = wl.draw_qkv_weights(cfg, hidden, with_bias=False)
    w_dev = bf16_dev(w)
    h = mc.c_void_p()
    L = mc.lib()
    assert L.mc_qkv_plan_create(dp.layout, w_dev.data_ptr(), None, 100, mc.byref(h)) == mc.MC_ERR_INVALID_ARG
    assert L.mc_qkv_plan_create(dp.layout, w_dev.data_ptr() + 2, None, hidden, mc.byref(h)) == mc.MC_ERR_INVALID_ARG
    assert L.mc_qkv_plan_create(None, w_dev.data_ptr(), None, hidden, mc.byref(h)) == mc.MC_ERR_INVALID_ARG
    f32 = wl.CONFIGS["cfg0"]
    dp32 = DeviceProblem.from_host(wl.make_host_problem(f32))
    assert L.mc_qkv_plan_create(dp32.layout, w_dev.data_ptr(), None, hidden, mc.byref(h)) == mc.MC_ERR_UNSUPPORTED
    plan = mc.mc_qkv_plan_create(dp.layout, w_dev, None, hidden)
    x = bf16_dev(wl.draw_hidden(cfg, 0, hidden))
    q_out = torch.empty(cfg.B, cfg.Hq, cfg.d, dtype=torch.bfloat16, device="cuda")
    po = torch.zeros(cfg.B, dtype=torch.int32, device="cuda")
    assert L.mc_qkv_append(plan, x.data_ptr(), q_out.data_ptr(), po.data_ptr(), 0.0, None) == mc.MC_ERR_INVALID_ARG
    assert L.mc_qkv_append(plan, x.data_ptr(), q_out.data_ptr(), None, -1.0, None) == mc.MC_ERR_INVALID_ARG
    assert L.mc_qkv_append(plan, None, q_out.data_ptr(), None, BASE, None) == mc.MC_ERR_INVALID_ARG
    assert L.mc_qkv_plan_destroy(None) == mc.MC_OK
    mc.mc_qkv_plan_destroy(plan)
    dp.close()
    dp32.close()
