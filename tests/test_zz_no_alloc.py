"""moe_dispatch_noalloc: the dispatch variant for callers that cannot provide scratch memory
(plugins running inside a pre-planned arena, allocation-free serving loops).  Its scratch is a
fixed array inside the library, shared by every call on a device, so the test runs it twice in a
row on different routings and requires both results to equal moe_dispatch's, bit for bit.
Collected last on purpose: a run that stops at the first failure has then run everything else."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2605_05607_b200 import binding as B
from paper_2605_05607_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def run_both(cfg):
    run = H.Run(cfg, inputs=synth.make_routing_inputs(cfg, "cuda") | {"w1": None, "w3": None, "w2": None})
    run.route()
    run.dispatch()                                        # existing entry point (workspace scratch)
    lay2 = B.alloc_layout(run.shape)
    xg2 = torch.zeros_like(run.xg)
    status = torch.full((8,), -1, dtype=torch.int32, device="cuda")
    B.moe_dispatch_noalloc(run.shape, run.t["x"], run.idx, lay2, xg2, status)
    torch.cuda.synchronize()
    assert status.tolist() == [0] * 8
    n_disp = int(run.lay.group_offsets[cfg.G].item())
    for name in ("expert_counts", "expert_offsets", "group_counts", "group_offsets", "pair_row", "row_pair",
                 "al", "row_src"):
        assert torch.equal(getattr(lay2, name), getattr(run.lay, name)), name
    assert torch.equal(lay2.disp_token[:n_disp], run.lay.disp_token[:n_disp])
    assert torch.equal(xg2[:n_disp].view(torch.int16), run.xg[:n_disp].view(torch.int16))
    # and directly against the oracle's layout and dispatched copy of the same routing
    saved, run.lay, run.xg = (run.lay, run.xg), lay2, xg2
    lay_ref = H.check_layout(run, run.host_idx())
    assert np.array_equal(H.bf16_host(xg2)[:n_disp], O.dispatch(H.bf16_host(run.t["x"]), lay_ref))
    run.lay, run.xg = saved
    return n_disp


def test_noalloc_dispatch_matches_dispatch_twice_in_a_row():
    # second call: other tokens, other shape, fewer mask words in use - stale contents of the
    # shared array from the first call must not leak into it
    a = run_both(synth.MoEConfig("na1", T=1000, d=256, f=64, E=32, k=4, G=8, bias="zipf", zipf_s=1.2, seed=21))
    b = run_both(synth.MoEConfig("na2", T=333, d=136, f=64, E=12, k=3, G=4, seed=22))
    c = run_both(synth.MoEConfig("na1", T=1000, d=256, f=64, E=32, k=4, G=8, bias="zipf", zipf_s=1.2, seed=23))
    assert a > 0 and b > 0 and c > 0


def test_noalloc_layout_only_limit_and_status():
    cfg = synth.MoEConfig("na3", T=64, d=64, f=64, E=8, k=2, G=4, seed=24)
    run = H.Run(cfg, inputs=synth.make_routing_inputs(cfg, "cuda") | {"w1": None, "w3": None, "w2": None})
    run.route()
    run.dispatch()
    lay2 = B.alloc_layout(run.shape)
    B.moe_dispatch_noalloc(run.shape, None, run.idx, lay2, None)          # layout only
    assert torch.equal(lay2.row_src, run.lay.row_src) and torch.equal(lay2.al, run.lay.al)
    # a shape whose tables exceed the built-in array is refused on the host, nothing is launched
    big = synth.CONFIGS["C5a"]
    need = 256 + 8 * (big.E + big.G) * ((big.T + 31) // 32)
    assert need > B.MOE_NOALLOC_SCRATCH_BYTES
    with pytest.raises(B.MoEError) as ei:
        B.moe_dispatch_noalloc(B.make_shape(big), None, run.idx, lay2, None)
    assert ei.value.code == B.MOE_ERR_SCRATCH_LIMIT and "scratch" in str(ei.value)
    # device-side conditions reach status_out
    run.idx[3] = 77
    status = torch.zeros(8, dtype=torch.int32, device="cuda")
    B.moe_dispatch_noalloc(run.shape, None, run.idx, lay2, None, status)
    torch.cuda.synchronize()
    assert status[0].item() == B.MOE_DEV_INDEX_OUT_OF_RANGE and status[3].item() == 77
