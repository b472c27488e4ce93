"""GPU parity of mc_kv_append_rope (rotary position embedding fused with the append) against the fp64 oracle:
the rotated key row as it lands in the paged cache, the query rotated in place, V untouched, lengths advanced, and a
decode step on top of it.  Tolerance: the result is rounded to the storage type once, so one unit in the last place
of it (bf16: 2^-8 relative to the pair's magnitude; fp32: 1e-5 absolute on unit-variance data)."""
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

BASE = 10000.0
CASES = {
    "bf16": (wl.scaled_down(wl.CONFIGS["cfg2"], "rope2", C=8, prefix=("fixed", 1040), suffix=("uniform", 0, 600),
                            append_steps=3), []),
    "f32": (wl.CONFIGS["cfg0"], []),
    # positions count the tokens of every cascade level in front of the candidate
    "bf16-3-levels": (wl.Config("ropec", "bf16", 4, 8, 32, 8, 128, ("loguniform", 100, 900), ("uniform", 0, 300),
                                seed=7), [([0, 32], [700]), ([0, 24, 32], [333, 64])]),
}


def positions(hp):
    go = hp.tables.group_offsets
    pos = np.array(hp.suffix_len, dtype=np.int64)
    for j in range(len(go) - 1):
        pos[go[j]:go[j + 1]] += int(hp.prefix_len[j])
    for lv in hp.outer:
        for j in range(len(lv.group_offsets) - 1):
            pos[lv.group_offsets[j]:lv.group_offsets[j + 1]] += lv.k[j].shape[0]
    return pos


def pair_tolerance(cfg, ref):
    """One unit in the last place of the storage type at the magnitude of the (real, imaginary) pair."""
    if cfg.dtype == "f32":
        return np.full(ref.shape, 1e-5)
    h = ref.shape[-1] // 2
    mag = np.hypot(ref[..., :h], ref[..., h:])
    return np.concatenate([mag, mag], axis=-1) * 2.0 ** -8 + 1e-6


def cache_rows(dp, hp, pool, s_before):
    """The rows the append wrote: [B][Hkv][d] read back from the paged pool."""
    cfg = hp.cfg
    p = pool.float().cpu().numpy().reshape(hp.tables.num_pages, cfg.Hkv, wl.PAGE, cfg.d)
    sp = hp.tables.suffix_pages
    return np.stack([p[sp[b, s_before[b] // wl.PAGE], :, s_before[b] % wl.PAGE, :] for b in range(cfg.B)])


@pytest.mark.parametrize("name", list(CASES))
def test_rope_append_matches_oracle(name):
    cfg, outer = CASES[name]
    hp = wl.make_host_problem(cfg, headroom_tokens=8)
    for i, (go, lens) in enumerate(outer):
        wl.add_outer_level(hp, go, lens, i)
    dp = DeviceProblem.from_host(hp)
    for step in (1, 2):
        k_new, v_new = wl.draw_append(cfg, step)
        q = wl.draw_q(cfg, step)
        pos = positions(hp)
        s_before = np.array(hp.suffix_len).copy()
        q_dev = to_device(cfg, q)
        mc.mc_kv_append_rope(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new), q_dev, None, BASE)
        torch.cuda.synchronize()
        assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
        k_ref = rope.rope_rows(k_new, pos, BASE)
        q_ref = rope.rope_rows(q, pos, BASE)
        k_got = cache_rows(dp, hp, dp.k_pool, s_before)
        q_got = q_dev.float().cpu().numpy()
        assert (np.abs(k_got - k_ref) <= pair_tolerance(cfg, k_ref)).all(), np.abs(k_got - k_ref).max()
        assert (np.abs(q_got - q_ref) <= pair_tolerance(cfg, q_ref)).all(), np.abs(q_got - q_ref).max()
        np.testing.assert_array_equal(cache_rows(dp, hp, dp.v_pool, s_before), v_new)       # V is only copied
        np.testing.assert_array_equal(dp.suffix_len.cpu().numpy(), s_before + 1)
        # the decode step that follows sees the rotated key: oracle attention over the oracle's rotated rows
        # (rounded to the storage type, as the cache holds them)
        hp.append(wl._round_to_dtype(cfg, k_ref.astype(np.float32)), v_new)
        o, lse = dp.decode(q_dev)
        torch.cuda.synchronize()
        q_in = q_got.astype(np.float64)
        if hp.outer:
            levels = [(lv.k, lv.v, lv.group_offsets.tolist()) for lv in hp.outer]
            levels.append((hp.k_prefix, hp.v_prefix, hp.tables.group_offsets.tolist()))
            o_ref, lse_ref = orc.decode_attention_cascade(q_in, levels, hp.k_suffix, hp.v_suffix, cfg.scale)
        else:
            o_ref, lse_ref = orc.decode_attention(q_in, hp.k_prefix, hp.v_prefix, hp.k_suffix, hp.v_suffix,
                                                  hp.tables.group_offsets.tolist(), cfg.scale)
        err = np.abs(o.float().cpu().numpy() - o_ref)
        assert err.max() <= (1e-5 if cfg.dtype == "f32" else 2e-2), err.max()
    dp.close()


def test_rope_append_with_given_offsets_and_without_query():
    cfg, _ = CASES["bf16"]
    hp = wl.make_host_problem(cfg, headroom_tokens=8)
    dp = DeviceProblem.from_host(hp)
    k_new, v_new = wl.draw_append(cfg, 1)
    off = np.arange(cfg.B, dtype=np.int32) * 9001 + 5          # large positions: the angle needs double precision
    s_before = np.array(hp.suffix_len).copy()
    mc.mc_kv_append_rope(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new), None,
                         torch.from_numpy(off).cuda(), 500000.0)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    k_ref = rope.rope_rows(k_new, off.astype(np.int64) + s_before, 500000.0)
    k_got = cache_rows(dp, hp, dp.k_pool, s_before)
    assert (np.abs(k_got - k_ref) <= pair_tolerance(cfg, k_ref)).all(), np.abs(k_got - k_ref).max()
    with pytest.raises(mc.McError):
        mc.mc_kv_append_rope(dp.layout, to_device(cfg, k_new), to_device(cfg, v_new), None, None, 0.0)
    dp.close()
