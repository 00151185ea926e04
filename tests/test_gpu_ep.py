"""Expert-parallel execution (group g on rank g) emulated on one GPU: all ranks run their three phases in one
process and the exchange is slicing / concatenation.  The result must be the dense layer definition (the oracle)
and agree with the single-GPU moe_layer on the same tokens and the full expert set."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2605_05607_b200 import binding as B
from paper_2605_05607_b200 import ep, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("base", [
    synth.MoEConfig("ep-a", T=0, d=256, f=320, E=16, k=4, G=4, seed=31),
    synth.MoEConfig("ep-b", T=0, d=192, f=128, E=24, k=6, G=8, score_fn=1, bias="zipf", zipf_s=1.2, seed=32),
    synth.MoEConfig("ep-c", T=0, d=128, f=256, E=8, k=2, G=8, seed=33),          # one expert per rank: nothing to trim
], ids=lambda c: c.name)
def test_emulated_expert_parallel_layer(base):
    world = base.G
    tokens = [137 + 61 * s for s in range(world)]                 # a different number of tokens on every rank
    tokens[1] = 1
    full = synth.make_inputs(base.with_(T=8), "cuda")             # the layer's weights (shared gate, all experts)
    m = base.m
    ranks, xs, cfgs = [], [], []
    for s in range(world):
        cfg = base.with_(T=tokens[s], seed=base.seed * 10 + s)
        x = synth.make_inputs(cfg.with_(E=1, k=1, G=1, f=8), "cuda")["x"]   # only x is taken from this draw
        sl = slice(s * m, (s + 1) * m)
        ranks.append(ep.EpRank(cfg, s, full["w_gate"], full["bias"], full["w1"][sl].contiguous(),
                               full["w3"][sl].contiguous(), full["w2"][sl].contiguous()))
        xs.append(x)
        cfgs.append(cfg)
    for _ in range(2):                                             # twice: buffers are reused between calls
        ys = ep.emulate(ranks, xs)
    torch.cuda.synchronize()
    for s in range(world):
        assert all(code == 0 for code in ranks[s].status()), (s, ranks[s].status())
        cfg = cfgs[s]
        # the single-GPU layer on the same tokens with every expert resident
        run = H.Run(cfg, inputs={"x": xs[s], "w_gate": full["w_gate"], "bias": full["bias"], "w1": full["w1"],
                                 "w3": full["w3"], "w2": full["w2"]})
        run.layer(logits=run.logits, topk_idx=run.idx, topk_w=run.w)
        torch.cuda.synchronize()
        y_ep = O.bf16_to_f64(H.bf16_host(ys[s])[: cfg.T])
        y_one = O.bf16_to_f64(H.bf16_host(run.y)[: cfg.T])
        mx, mean = H.out_errors(y_ep, y_one)
        assert mx <= 1e-2 and mean <= 3e-3, (s, mx, mean)          # the partial rows travel as bf16
        # and against the dense definition, routing taken from this rank's own logits
        assert torch.equal(ranks[s].idx[: cfg.P], run.idx[: cfg.P])
        _, _, _, y_def = O.layer(H.bf16_host(xs[s]), run.host_logits(), run.host_bias(), H.bf16_host(full["w1"]),
                                 H.bf16_host(full["w3"]), H.bf16_host(full["w2"]), cfg.k, cfg.score_fn)
        H.assert_close_out(y_ep, y_def, f"rank {s} y")


def test_ep_pack_lists_are_the_trimmed_targets():
    cfg = synth.MoEConfig("ep-pack", T=500, d=64, f=64, E=12, k=5, G=3, seed=41)
    run = H.Run(cfg, inputs=synth.make_routing_inputs(cfg, "cuda") | {"w1": None, "w3": None, "w2": None})
    run.route()
    run.dispatch()
    m, kk = cfg.m, min(cfg.k, cfg.m)
    cap = cfg.T * min(cfg.k, cfg.G)
    send_idx = torch.zeros(cap, kk, dtype=torch.int32, device="cuda")
    send_w = torch.zeros(cap, kk, dtype=torch.float32, device="cuda")
    B.moe_ep_pack(run.shape, run.idx, run.w, run.lay, send_idx, send_w)
    idx, w = run.host_idx(), run.host_w()
    lay = O.layout(idx, cfg.E, cfg.G)
    got_i, got_w = send_idx.cpu().numpy(), send_w.cpu().numpy()
    for n in range(lay["n_disp"]):
        t = int(lay["disp_token"][n])
        g = int(np.searchsorted(lay["group_offsets"], n, side="right") - 1)
        want = [(int(idx[t, j]) - g * m, w[t, j]) for j in range(cfg.k) if idx[t, j] // m == g]
        assert 1 <= len(want) <= kk
        assert got_i[n, : len(want)].tolist() == [e for e, _ in want] and (got_i[n, len(want):] == -1).all()
        assert np.array_equal(got_w[n, : len(want)], np.float32([x for _, x in want])) and not got_w[n, len(want):].any()


def test_forward_over_nccl_with_one_rank():
    """EpRank.forward with a real NCCL process group of size 1 (all this box offers): the exchange degenerates
    to a copy, everything else is the code path several GPUs would run."""
    import os
    import socket
    import torch.distributed as dist
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK="0", WORLD_SIZE="1")
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        cfg = synth.MoEConfig("ep-nccl1", T=300, d=128, f=192, E=6, k=3, G=1, seed=51)
        t = synth.make_inputs(cfg, "cuda")
        rank = ep.EpRank(cfg, 0, t["w_gate"], t["bias"], t["w1"], t["w3"], t["w2"])
        y = rank.forward(t["x"]).clone()
        torch.cuda.synchronize()
        assert all(c == 0 for c in rank.status())
        run = H.Run(cfg, inputs=t)
        run.layer()
        torch.cuda.synchronize()
        mx, mean = H.out_errors(O.bf16_to_f64(H.bf16_host(y)), O.bf16_to_f64(H.bf16_host(run.y)[: cfg.T]))
        assert mx <= 1e-2 and mean <= 3e-3, (mx, mean)
    finally:
        dist.destroy_process_group()
