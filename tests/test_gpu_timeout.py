"""A bounded device-side wait that runs out: the kernels stop, report MC_ERR_TIMEOUT through the status word and
return, and the context stays usable.

Every wait of the TMA-fed kernels (on an mbarrier that a copy or a tensor-core product completes) has a limit in SM
clock cycles, about one second by default, taken from MC_WAIT_CYCLES when a layout is created.  Here the limit is
zero cycles, so the first wait that is not already satisfied gives up - nothing is made to fault or to hang: the
roles of a CTA see the abort flag or their own expired wait, stop issuing work, grant the copies and products that
are still in flight a millisecond to land, free their tensor memory and exit.  The results of such a step are
meaningless and are not looked at."""
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

# 8 candidates: one 128-row tile per (group, kv head), the prefix kernel with two tile streams; 40 candidates: three
# row tiles, the row-pair prefix kernel
CFGS = {"one-tile": wl.scaled_down(wl.CONFIGS["cfg2"], "timeout", C=8, prefix=("fixed", 1040), suffix=("uniform", 0, 600)),
        "row-pairs": wl.scaled_down(wl.CONFIGS["cfg2"], "timeout-rp", C=40, prefix=("fixed", 1040), suffix=("uniform", 0, 300))}


@pytest.mark.parametrize("passes,shape", [("prefix", "one-tile"), ("suffix", "one-tile"), ("step", "one-tile"),
                                          ("prefix", "row-pairs"), ("step", "row-pairs")])
def test_expired_wait_is_reported_and_the_next_call_is_correct(passes, shape, monkeypatch):
    CFG = CFGS[shape]
    hp = wl.make_host_problem(CFG)
    q_np = wl.draw_q(CFG, 0)
    q = to_device(CFG, q_np)
    monkeypatch.setenv("MC_WAIT_CYCLES", "0")
    dp = DeviceProblem.from_host(hp)                    # its kernels get the zero limit
    assert dp.geom.prefix_ctas > 0                      # the tcgen05 prefix kernel and the TMA-fed suffix kernel
    o_part, lse_part = dp.new_parts()
    if passes == "prefix":
        mc.mc_prefix_attn(dp.layout, q, CFG.scale, o_part, lse_part)
    elif passes == "suffix":
        mc.mc_suffix_attn(dp.layout, q, CFG.scale, o_part, lse_part)
    else:
        dp.decode(q)
    torch.cuda.synchronize()                            # the kernels returned
    assert mc.mc_get_last_status(dp.layout) == mc.MC_ERR_TIMEOUT
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK  # reading the word clears it
    dp.close()
    # the context is intact: a layout made with the ordinary limit computes the step correctly
    monkeypatch.delenv("MC_WAIT_CYCLES")
    dp = DeviceProblem.from_host(hp)
    o, lse = dp.decode(q)
    torch.cuda.synchronize()
    assert mc.mc_get_last_status(dp.layout) == mc.MC_OK
    o_ref, lse_ref = orc.decode_attention(q_np, hp.k_prefix, hp.v_prefix, hp.k_suffix, hp.v_suffix,
                                          hp.tables.group_offsets.tolist(), CFG.scale)
    err = np.abs(o.float().cpu().numpy().astype(np.float64) - o_ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 1e-3
    dp.close()
