"""Host logic of the seeded workload generator: lengths, page tables, paging round trip, bf16 bits."""
import numpy as np
import pytest

from paper_2601_05475_b200 import workload as wl


def test_bf16_bits_match_torch_rounding():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(size=5000).astype(np.float32) * 10,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.0078125, 1.01171875, 65504.0, 1e-30, 3.3895e38],
                                 dtype=np.float32)])
    bits = wl.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, ref)
    back = wl.bf16_bits_to_f32(bits)
    np.testing.assert_array_equal(back, torch.from_numpy(x).to(torch.bfloat16).float().numpy())


@pytest.mark.parametrize("name", ["cfg0", "cfg1", "cfg2", "cfg3", "cfg4"])
def test_lengths_follow_the_stated_distributions(name):
    cfg = wl.CONFIGS[name]
    pl, sl = wl.draw_lengths(cfg)
    assert pl.shape == (cfg.G,) and sl.shape == (cfg.B,)
    if cfg.prefix[0] == "fixed":
        assert (pl == cfg.prefix[1]).all()
    else:
        assert (pl >= cfg.prefix[1]).all() and (pl <= cfg.prefix[2]).all() and len(set(pl.tolist())) > 1
    if cfg.suffix[0] == "fixed":
        assert sl.tolist() == list(cfg.suffix[1])
    else:
        assert (sl >= cfg.suffix[1]).all() and (sl <= cfg.suffix[2]).all()
    pl2, sl2 = wl.draw_lengths(cfg)
    np.testing.assert_array_equal(pl, pl2)
    np.testing.assert_array_equal(sl, sl2)


@pytest.mark.parametrize("name", ["cfg0", "cfg1", "cfg3", "cfg4"])
def test_page_tables_are_a_partition(name):
    cfg = wl.CONFIGS[name]
    pl, sl = wl.draw_lengths(cfg)
    t = wl.build_page_tables(cfg, pl, sl)
    used = np.concatenate([t.prefix_pages[t.prefix_pages >= 0], t.suffix_pages[t.suffix_pages >= 0]])
    assert used.size == t.num_pages and np.array_equal(np.sort(used), np.arange(t.num_pages))
    # enough pages for the current length plus the append head-room, suffix on pages of its own
    for b in range(cfg.B):
        assert (t.suffix_pages[b] >= 0).sum() * wl.PAGE >= sl[b] + cfg.append_steps
    for j in range(cfg.G):
        assert (t.prefix_pages[j] >= 0).sum() == (pl[j] + wl.PAGE - 1) // wl.PAGE
    if cfg.permute_pages:
        assert not np.array_equal(used, np.arange(t.num_pages))
    assert t.group_offsets.tolist() == [j * cfg.C for j in range(cfg.G + 1)]


@pytest.mark.parametrize("name,permute", [("cfg0", False), ("cfg0", True), ("cfg1", True)])
def test_paged_image_round_trips_to_the_logical_view(name, permute):
    cfg = wl.CONFIGS[name]
    hp = wl.make_host_problem(cfg, permute=permute)
    widen = (lambda a: a) if cfg.dtype == "f32" else wl.bf16_bits_to_f32
    for j in range(cfg.G):
        for h in range(cfg.Hkv):
            got = widen(wl.gather_logical(hp.k_pool, hp.tables.prefix_pages[j], int(hp.prefix_len[j]), h))
            np.testing.assert_array_equal(got, hp.k_prefix[j][:, h, :])
    for b in range(cfg.B):
        for h in range(cfg.Hkv):
            got = widen(wl.gather_logical(hp.v_pool, hp.tables.suffix_pages[b], int(hp.suffix_len[b]), h))
            np.testing.assert_array_equal(got, hp.v_suffix[b][:, h, :])
    # slots past the end of a sequence hold the sentinel
    b = 1
    n = int(hp.suffix_len[b])
    if n % wl.PAGE:
        page = hp.tables.suffix_pages[b][n // wl.PAGE]
        assert (widen(hp.k_pool[page, 0, n % wl.PAGE:]) == widen(wl.storage_array(cfg, np.float32([wl.SENTINEL])))[0]).all()


def test_outlier_rows_are_whole_rows_scaled():
    cfg = wl.scaled_down(wl.CONFIGS["cfg3"], "cfg3-small", G=2, C=2, prefix=("loguniform", 1024, 2048),
                         suffix=("uniform", 0, 64))
    hp = wl.make_host_problem(cfg)
    k = hp.k_prefix[0]                              # [P][Hkv][d]
    rms = np.sqrt((k.astype(np.float64) ** 2).mean(axis=2))
    frac = (rms > 4.0).mean()
    assert 0.002 < frac < 0.03                      # about 1 % of (token, head) rows have rms near 8
    assert abs(np.median(rms) - 1.0) < 0.1


def test_append_draws_are_per_step_and_q_changes():
    cfg = wl.CONFIGS["cfg1"]
    k1, v1 = wl.draw_append(cfg, 1)
    k2, _ = wl.draw_append(cfg, 2)
    assert k1.shape == (cfg.B, cfg.Hkv, cfg.d) and not np.array_equal(k1, k2) and not np.array_equal(k1, v1)
    assert not np.array_equal(wl.draw_q(cfg, 0), wl.draw_q(cfg, 1))
    np.testing.assert_array_equal(wl.draw_q(cfg, 3), wl.draw_q(cfg, 3))


def test_unique_bytes_accounting():
    cfg = wl.CONFIGS["cfg2"]
    pl, sl = wl.draw_lengths(cfg)
    ub = wl.unique_bytes(cfg, pl, sl)
    assert ub["kv_prefix"] == 8192 * 4096
    assert ub["kv_suffix"] == int(sl.sum()) * 4096
    assert ub["q_o"] == 2 * 64 * 64 * 128 * 2 and ub["lse"] == 64 * 64 * 4


def test_search_batch_is_seeded_and_shaped():
    a, b = wl.draw_search_batch(5, K=8, T=8, seed=1), wl.draw_search_batch(5, K=8, T=8, seed=1)
    assert a["N"] == 40 and a["speedup"].shape == (8, 40) and a["correct"].dtype == np.uint8
    for k in ("speedup", "correct", "len", "logits", "group_offsets"):
        np.testing.assert_array_equal(a[k], b[k])
    assert a["len"].min() >= 1 and a["len"].max() <= 8 and a["group_offsets"].tolist() == list(range(0, 41, 8))
    assert 0.5 < a["correct"].mean() < 0.9 and (a["speedup"] > 0).all()
    assert not np.array_equal(a["speedup"], wl.draw_search_batch(5, K=8, T=8, seed=2)["speedup"])
