"""Caches with 32- and 64-token pages: the library walks them in 16-token blocks through tables it derives from the
caller's.  Every case compares with the fp64 oracle on the logical (unpaged) sequences, which know nothing of pages;
appended rows are also looked up in the pool image at the slot the layout defines."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import attention as orc
from oracle import rope
from paper_2601_05475_b200 import binding as mc
from paper_2601_05475_b200 import workload as wl
from paper_2601_05475_b200.harness import DeviceProblem, to_device

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

PAGES = [32, 64]


def paged(cfg, page, **kw):
    return dataclasses.replace(cfg, name=f"{cfg.name}_p{page}", page=page, **kw)


def oracle_full(hp, q):
    levels = [(lv.k, lv.v, lv.group_offsets.tolist()) for lv in hp.outer]
    if levels:
        levels.append((hp.k_prefix, hp.v_prefix, hp.tables.group_offsets.tolist()))
        return orc.decode_attention_cascade(q, levels, hp.k_suffix, hp.v_suffix, hp.cfg.scale)
    return orc.decode_attention(q, hp.k_prefix, hp.v_prefix, hp.k_suffix, hp.v_suffix,
                                hp.tables.group_offsets.tolist(), hp.cfg.scale)


def check(cfg, o_gpu, lse_gpu, o_ref, lse_ref):
    o = o_gpu.float().cpu().numpy().astype(np.float64)
    lse = lse_gpu.cpu().numpy().astype(np.float64)
    err = np.abs(o - o_ref)
    assert np.isfinite(o).all()
    if cfg.dtype == "f32":
        assert err.max() <= 1e-5, err.max()
    else:
        assert err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())
    empty = np.isneginf(lse_ref)
    assert np.array_equal(np.isneginf(lse), empty)
    assert empty.all() or np.abs(lse[~empty] - lse_ref[~empty]).max() <= 1e-3


BASE = {
    "f32": wl.CONFIGS["cfg0"],
    "flat": wl.scaled_down(wl.CONFIGS["cfg2"], "flat", C=8, prefix=("fixed", 1040), suffix=("uniform", 0, 600)),
    "ragged": wl.scaled_down(wl.CONFIGS["cfg3"], "ragged", G=3, C=4, prefix=("loguniform", 90, 1500),
                             suffix=("uniform", 0, 700), permute_pages=True),
    "long": wl.scaled_down(wl.CONFIGS["cfg4"], "long", G=2, C=3, prefix=("fixed", 512), suffix=("uniform", 1000, 2100)),
    "d64": wl.Config("d64", "bf16", 2, 5, 16, 4, 64, ("fixed", 333), ("uniform", 0, 300), permute_pages=True),
}


@pytest.mark.parametrize("page", PAGES)
@pytest.mark.parametrize("name", list(BASE))
def test_decode_matches_oracle(name, page):
    cfg = paged(BASE[name], page)
    hp = wl.make_host_problem(cfg)
    assert hp.k_pool.shape[2] == page
    dp = DeviceProblem.from_host(hp)
    q = wl.draw_q(cfg, 0)
    o, lse = dp.decode(to_device(cfg, q))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    check(cfg, o, lse, *oracle_full(hp, q))
    dp.close()


@pytest.mark.parametrize("page", PAGES)
@pytest.mark.parametrize("env", [{"MC_SUFFIX_TMA": "0"}, {"MC_PREFIX_TC": "0"}, {"MC_FORCE_FMA": "1"}, {"MC_PDL": "0"}],
                         ids=lambda e: "-".join(f"{k}={v}" for k, v in e.items()))
def test_every_kernel_family_walks_the_larger_pages(monkeypatch, env, page):
    for k, v in env.items():
        monkeypatch.setenv(k, v)
    cfg = paged(BASE["ragged"], page)
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    q = wl.draw_q(cfg, 1)
    o, lse = dp.decode(to_device(cfg, q))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    check(cfg, o, lse, *oracle_full(hp, q))
    dp.close()


@pytest.mark.parametrize("page", PAGES)
@pytest.mark.parametrize("pairs", ["1", "0"])
def test_several_row_tiles_and_a_cascade(monkeypatch, pairs, page):
    """40 candidates x 8 query heads per kv head = 320 stacked rows per group (three row tiles), two prefix splits and
    an outer level shared by both groups: the tensor-core prefix kernels, with and without row pairs."""
    monkeypatch.setenv("MC_PREFIX_PAIRS", pairs)
    monkeypatch.setenv("MC_PREFIX_PART_TOKENS", "256")
    cfg = paged(wl.Config("tiles", "bf16", 2, 40, 32, 4, 128, ("fixed", 500), ("uniform", 0, 90), permute_pages=True), page)
    hp = wl.make_host_problem(cfg)
    wl.add_outer_level(hp, [0, cfg.B], [270])
    dp = DeviceProblem.from_host(hp)
    assert dp.geom.prefix_ctas > 0
    q = wl.draw_q(cfg, 0)
    o, lse = dp.decode(to_device(cfg, q))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    check(cfg, o, lse, *oracle_full(hp, q))
    dp.close()


def slot_of(hp, b, s):
    page = hp.cfg.page
    return int(hp.tables.suffix_pages[b, s // page]), s % page


@pytest.mark.parametrize("page", PAGES)
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_appends_cross_block_and_page_boundaries(dtype, page):
    """70 one-token steps from suffix lengths on both sides of 16-token and page boundaries; every appended row is
    looked up in the pool at [page id][kv head][slot in page], and every fifth step is compared with the oracle."""
    cfg = paged(wl.Config("app", dtype, 1, 6, 8, 2, 64 if dtype == "f32" else 128, ("fixed", 150),
                          ("fixed", (0, 15, 16, 31, page - 1, page)), permute_pages=True, append_steps=70), page)
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    for step in range(1, cfg.append_steps + 1):
        k_new, v_new = wl.draw_append(cfg, step)
        q = wl.draw_q(cfg, step)
        s0 = hp.suffix_len.copy()
        if step % 2:
            mc.mc_kv_append(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new))
            dp.decode(to_device(cfg, q))
        else:
            mc.mc_decode_step(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new), to_device(cfg, q), cfg.scale,
                              dp.o, dp.lse, dp.ws_ptr, dp.ws_bytes)
        hp.append(k_new, v_new)
        if step % 5 == 0 or step in (1, 2):
            torch.cuda.synchronize()
            check(cfg, dp.o, dp.lse, *oracle_full(hp, q))
        if step % 9 == 0:
            kp, vp = dp.k_pool.float().cpu().numpy(), dp.v_pool.float().cpu().numpy()
            for b in range(cfg.B):
                pid, slot = slot_of(hp, b, int(s0[b]))
                np.testing.assert_array_equal(kp[pid, :, slot], k_new[b])
                np.testing.assert_array_equal(vp[pid, :, slot], v_new[b])
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), hp.suffix_len)
    for _ in range(page + 1):          # beyond the head-room: refused and reported
        mc.mc_kv_append(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new))
    assert mc.mc_get_last_status(dp.layout) == mc.MC_ERR_INVALID_ARG
    dp.close()


@pytest.mark.parametrize("page", PAGES)
def test_many_tokens_and_rotary_appends_land_in_their_slots(page):
    n_max, base = 37, 10000.0
    cfg = paged(wl.scaled_down(wl.CONFIGS["cfg2"], "many", C=4, prefix=("fixed", 300), suffix=("uniform", 0, 200)), page)
    hp = wl.make_host_problem(cfg, headroom_tokens=2 * n_max + 1)
    dp = DeviceProblem.from_host(hp)
    rng = np.random.default_rng(page)
    draw = lambda *shape: wl._round_to_dtype(cfg, rng.standard_normal(shape, dtype=np.float32))
    # plain
    k, v = draw(cfg.B, n_max, cfg.Hkv, cfg.d), draw(cfg.B, n_max, cfg.Hkv, cfg.d)
    n = np.array([n_max, 0, 5, 36], dtype=np.int32)
    s0 = hp.suffix_len.copy()
    mc.mc_kv_append_tokens(dp.layout, to_device(cfg, k), to_device(cfg, v), n_max, torch.from_numpy(n).cuda())
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    kp, vp = dp.k_pool.float().cpu().numpy(), dp.v_pool.float().cpu().numpy()
    for b in range(cfg.B):
        for t in range(n[b]):
            pid, slot = slot_of(hp, b, int(s0[b]) + t)
            np.testing.assert_array_equal(kp[pid, :, slot], k[b, t])
            np.testing.assert_array_equal(vp[pid, :, slot], v[b, t])
        hp.k_suffix[b] = np.concatenate([hp.k_suffix[b], k[b, :n[b]]], axis=0)
        hp.v_suffix[b] = np.concatenate([hp.v_suffix[b], v[b, :n[b]]], axis=0)
        hp.suffix_len[b] += n[b]
    q = wl.draw_q(cfg, 3)
    o, lse = dp.decode(to_device(cfg, q))
    torch.cuda.synchronize()
    check(cfg, o, lse, *oracle_full(hp, q))
    # one rotated token per candidate (Su et al., "RoFormer": pair (i, i + d/2) turned by pos * base^(-2i/d))
    k1, v1 = draw(cfg.B, cfg.Hkv, cfg.d), draw(cfg.B, cfg.Hkv, cfg.d)
    s0 = hp.suffix_len.copy()
    mc.mc_kv_append_rope(dp.layout, to_device(cfg, k1), to_device(cfg, v1), None, None, base)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    kp, vp = dp.k_pool.float().cpu().numpy(), dp.v_pool.float().cpu().numpy()
    half = cfg.d // 2
    for b in range(cfg.B):
        pid, slot = slot_of(hp, b, int(s0[b]))
        pos = int(hp.prefix_len[b // cfg.C]) + int(s0[b])
        np.testing.assert_array_equal(vp[pid, :, slot], v1[b])
        for h in range(cfg.Hkv):
            ref = rope.rope_rotate(k1[b, h], pos, base)
            mag = np.hypot(ref[:half], ref[half:])
            assert (np.abs(kp[pid, h, slot] - ref) <= np.concatenate([mag, mag]) * 2.0 ** -8 + 1e-6).all()
    # several rotated tokens
    k, v = draw(cfg.B, n_max, cfg.Hkv, cfg.d), draw(cfg.B, n_max, cfg.Hkv, cfg.d)
    s0 = s0 + 1
    mc.mc_kv_append_tokens(dp.layout, to_device(cfg, k), to_device(cfg, v), n_max, torch.from_numpy(n).cuda(), None,
                           None, base)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    kp = dp.k_pool.float().cpu().numpy()
    for b in range(cfg.B):
        for t in range(0, n[b], 7):
            pid, slot = slot_of(hp, b, int(s0[b]) + t)
            pos = int(hp.prefix_len[b // cfg.C]) + int(s0[b]) + t
            ref = rope.rope_rotate(k[b, t, 1], pos, base)
            mag = np.hypot(ref[:half], ref[half:])
            assert (np.abs(kp[pid, 1, slot] - ref) <= np.concatenate([mag, mag]) * 2.0 ** -8 + 1e-6).all()
    np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), s0 + n)
    dp.close()


@pytest.mark.parametrize("page", PAGES)
def test_tables_are_a_snapshot_until_refreshed(page):
    """The layout reads the caller's tables when it is made and when mc_kv_layout_refresh_tables is called: a page
    handed to a growing suffix afterwards is not seen before the refresh and is used after it."""
    cfg = paged(wl.Config("grow", "bf16", 1, 3, 16, 2, 128, ("fixed", 100), ("fixed", (page, 5, 2 * page)),
                          permute_pages=True), page)
    hp = wl.make_host_problem(cfg, headroom_tokens=page + 2)       # pages for two more tokens exist in the pools ...
    held_back = hp.tables.suffix_pages.copy()
    for b in range(cfg.B):                                          # ... but the tables do not name them yet
        hp.tables.suffix_pages[b, (int(hp.suffix_len[b]) + page - 1) // page:] = -1
    dp = DeviceProblem.from_host(hp)
    k_new, v_new = wl.draw_append(cfg, 1)
    mc.mc_kv_append(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_ERR_INVALID_ARG          # candidates 0 and 2 have no page
    np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), hp.suffix_len + np.array([0, 1, 0]))
    dp.suffix_pages.copy_(torch.from_numpy(held_back))             # the caller assigns the pages
    mc.mc_kv_append(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_ERR_INVALID_ARG          # not seen: the layout holds a snapshot
    np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), hp.suffix_len + np.array([0, 2, 0]))
    mc.mc_kv_layout_refresh_tables(dp.layout)
    hp.tables.suffix_pages[:] = held_back
    # candidate 1 took both appends, 0 and 2 neither; one more append to all: now every candidate has room
    mc.mc_kv_append(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    counts = [1, 3, 1]
    for b in range(cfg.B):
        for _ in range(counts[b]):
            hp.k_suffix[b] = np.concatenate([hp.k_suffix[b], k_new[b][None]], axis=0)
            hp.v_suffix[b] = np.concatenate([hp.v_suffix[b], v_new[b][None]], axis=0)
        hp.suffix_len[b] += counts[b]
    np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), hp.suffix_len)
    q = wl.draw_q(cfg, 1)
    o, lse = dp.decode(to_device(cfg, q))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    check(cfg, o, lse, *oracle_full(hp, q))
    dp.close()


@pytest.mark.parametrize("page", PAGES)
def test_validate_and_bad_ids(page):
    cfg = paged(BASE["flat"], page)
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    units = hp.tables.num_pages * (page // 16)
    scratch = torch.empty(units, dtype=torch.int32, device="cuda")
    assert mc.mc_kv_layout_validate(dp.layout, scratch, units * 4) == mc.MC_OK
    assert mc.mc_kv_layout_validate(dp.layout, scratch, hp.tables.num_pages * 4) == mc.MC_ERR_WORKSPACE_TOO_SMALL
    # validation reads the tables as they are now
    good = dp.suffix_pages.clone()
    dp.suffix_pages[3, 0] = dp.suffix_pages[4, 0]
    assert mc.mc_kv_layout_validate(dp.layout, scratch, units * 4) == mc.MC_ERR_INVALID_ARG
    dp.suffix_pages.copy_(good)
    dp.suffix_pages[2, 0] = hp.tables.num_pages + 7          # an id no pool has: skipped and reported, never read
    dp.prefix_pages[0, 3] = -5
    mc.mc_kv_layout_refresh_tables(dp.layout)
    dp.decode(to_device(cfg, wl.draw_q(cfg, 0)))
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_ERR_INVALID_ARG
    assert torch.isfinite(dp.o.float()).all()
    dp.close()


def test_unsupported_page_sizes_are_refused():
    cfg = BASE["flat"]
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    h = mc.c_void_p()
    for size in (0, 8, 48, 128):
        bad = mc.LayoutDesc.from_buffer_copy(dp.desc)
        bad.page_size = size
        assert mc.lib().mc_kv_layout_create(mc.byref(bad), mc.byref(h)) == mc.MC_ERR_UNSUPPORTED and not h.value
    bad = mc.LayoutDesc.from_buffer_copy(dp.desc)       # the allocation-free entry point walks 16-token pages only
    bad.page_size = 32
    q = to_device(cfg, wl.draw_q(cfg, 0))
    assert mc.lib().mc_decode_attn_static(mc.byref(bad), q.data_ptr(), cfg.scale, dp.o.data_ptr(), dp.lse.data_ptr(),
                                          0, 0) == mc.MC_ERR_UNSUPPORTED
    dp.close()
