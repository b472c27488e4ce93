"""mc_decode_attn_static: the allocation-free entry point (scratch compiled into the library).

Some callers may not allocate device memory at all - a serving loop whose memory was handed out at
start-up, a plug-in barred from the device heap.  For them the library carries a fixed 16 MiB scratch
array.  This test calls the entry point through the C ABI twice in a row (the array is shared and keeps
the first call's contents) and checks both results against the regular mc_decode_attn and, because the entry
point cuts the token ranges by a rule of its own, against the CPU oracle as well; the second call must leave
the amount of free device memory as it found it.  It is collected last so that a run stopping at the first
failure has already run every other test.
"""
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


@pytest.mark.parametrize("name", ["cfg1", "cfg0"])
def test_static_entry_point_matches_regular_one_twice_in_a_row(name):
    cfg = wl.CONFIGS[name]
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    o_s = torch.empty_like(dp.o)
    lse_s = torch.empty_like(dp.lse)
    for step in range(2):                       # second call meets the first call's leftovers in the scratch
        q_np = wl.draw_q(cfg, step)
        q = to_device(cfg, q_np)
        o_ref, lse_ref = dp.decode(q)
        o_s.fill_(float("nan"))
        lse_s.fill_(float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        assert mc.mc_decode_attn_static(dp.desc, q, cfg.scale, o_s, lse_s, status) == mc.MC_OK
        torch.cuda.synchronize()
        if step == 1:                           # (the first call on a device loads the module that holds the array)
            assert torch.cuda.mem_get_info()[0] == free_before
        assert int(status.item()) == mc.MC_OK
        tol = (1e-5, 1e-5) if cfg.dtype == "f32" else (2e-2, 2e-3)
        err = (o_s.float() - o_ref.float()).abs()
        assert err.max().item() <= tol[0] and err.mean().item() <= tol[1]
        assert (lse_s - lse_ref).abs().max().item() <= 1e-3
        # ... and against the oracle itself
        o_orc, lse_orc = orc.decode_attention(q_np, hp.k_prefix, hp.v_prefix, hp.k_suffix, hp.v_suffix,
                                              hp.tables.group_offsets.tolist(), cfg.scale)
        err = np.abs(o_s.float().cpu().numpy().astype(np.float64) - o_orc)
        assert err.max() <= tol[0] and err.mean() <= tol[1], (err.max(), err.mean())
        lse_np = lse_s.cpu().numpy().astype(np.float64)
        assert not np.isnan(lse_np).any()
        empty = np.isneginf(lse_orc)
        assert np.array_equal(np.isneginf(lse_np), empty)
        assert np.abs(lse_np[~empty] - lse_orc[~empty]).max() <= 1e-3
    dp.close()


def test_static_entry_point_refuses_what_does_not_fit_and_reports_bad_pages():
    cfg = wl.CONFIGS["cfg1"]
    hp = wl.make_host_problem(cfg)
    dp = DeviceProblem.from_host(hp)
    q = to_device(cfg, wl.draw_q(cfg, 0))
    assert mc.mc_static_scratch_bytes() == 16 << 20
    big = mc.LayoutDesc.from_buffer_copy(dp.desc)
    big.batch, big.num_groups = 4096, 1          # 4096*32 rows of partials cannot fit 16 MiB
    assert mc.mc_decode_attn_static(big, q, cfg.scale, dp.o, dp.lse) == mc.MC_ERR_WORKSPACE_TOO_SMALL
    assert mc.mc_decode_attn_static(dp.desc, None, cfg.scale, dp.o, dp.lse) == mc.MC_ERR_INVALID_ARG
    # a page id outside the pool is skipped and shows up in the caller's status word
    dp.suffix_pages[2, 0] = hp.tables.num_pages + 3
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert mc.mc_decode_attn_static(dp.desc, q, cfg.scale, dp.o, dp.lse, status) == mc.MC_OK
    torch.cuda.synchronize()
    assert int(status.item()) == mc.MC_ERR_INVALID_ARG and torch.isfinite(dp.o.float()).all()
    dp.close()
