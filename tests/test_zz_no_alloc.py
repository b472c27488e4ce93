"""mc_decode_attn_static: the allocation-free entry point (scratch compiled into the library).

Some callers may not allocate device memory at all - a serving loop whose memory was handed out at
start-up, a plug-in barred from the device heap.  For them the library carries a fixed 16 MiB scratch
array.  This test calls the entry point through the C ABI twice in a row (the array is shared and keeps
the first call's contents) and checks both results against the regular mc_decode_attn.  It is collected
last so that a run stopping at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

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
        q = to_device(cfg, wl.draw_q(cfg, step))
        o_ref, lse_ref = dp.decode(q)
        o_s.fill_(float("nan"))
        lse_s.fill_(float("nan"))
        assert mc.mc_decode_attn_static(dp.desc, q, cfg.scale, o_s, lse_s, status) == mc.MC_OK
        torch.cuda.synchronize()
        assert int(status.item()) == mc.MC_OK
        err = (o_s.float() - o_ref.float()).abs()
        if cfg.dtype == "f32":
            assert err.max().item() <= 1e-5
        else:
            assert err.max().item() <= 2e-2 and err.mean().item() <= 2e-3
        assert (lse_s - lse_ref).abs().max().item() <= 1e-3
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
