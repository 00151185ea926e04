"""GPU parity of the backward pass (moe_layer_backward) against the fp64 oracle, for the routing the GPU's own forward
produced: dx and every expert's weight gradients on small shapes (ragged sizes, empty experts, top-1 .. top-16), sampled
experts and tokens at full size.  bf16 operands, fp32 accumulation, intermediates (dO, dH, h, dA1, dA3, dXs) rounded to
bf16: the same bars as the forward outputs, max|gpu - ref| <= 2e-2 max|ref| and sum|gpu - ref| / sum|ref| <= 5e-3
(observed: 4-6e-3 and 2.7-3.7e-3)."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2605_05607_b200 import binding as B
from paper_2605_05607_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

MAX_REL, MEAN_REL = H.MAX_REL, H.MEAN_REL


def close(got, ref, what):
    mx, mean = H.out_errors(got, ref)
    assert mx <= MAX_REL and mean <= MEAN_REL, f"{what}: max rel {mx:.3e}, mean rel {mean:.3e}"


class Backward:
    def __init__(self, cfg, seed=77):
        self.cfg = cfg
        self.run = run = H.Run(cfg)
        run.route()
        run.dispatch()                     # layout (and xg, unused here)
        g = torch.Generator(device="cuda")
        g.manual_seed(seed)
        T, d, f, E = cfg.T, cfg.d, cfg.f, cfg.E
        self.dy = torch.randn(max(T, 1), d, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        self.dx = torch.full((max(T, 1), d), 7.0, dtype=torch.bfloat16, device="cuda")
        self.dw1 = torch.full((E, d, f), 7.0, dtype=torch.bfloat16, device="cuda")
        self.dw3 = torch.full((E, d, f), 7.0, dtype=torch.bfloat16, device="cuda")
        self.dw2 = torch.full((E, f, d), 7.0, dtype=torch.bfloat16, device="cuda")
        self.ws = torch.zeros(B.moe_backward_workspace_bytes(run.shape), dtype=torch.uint8, device="cuda")

    def __call__(self):
        r, t = self.run, self.run.t
        B.moe_layer_backward(r.shape, t["x"], self.dy, r.idx, r.w, r.lay, t["w1"], t["w3"], t["w2"], self.dx, self.dw1,
                             self.dw3, self.dw2, self.ws)
        torch.cuda.synchronize()
        st = B.moe_status(self.ws)
        assert st[0] == 0 and st[4] == 0, f"device status {st}"


SMALL = [
    synth.CONFIGS["C1"],
    synth.MoEConfig("ragged", T=333, d=200, f=328, E=12, k=3, G=4, bias="zipf", zipf_s=1.5, seed=2),
    synth.MoEConfig("k1", T=150, d=128, f=192, E=4, k=1, G=2, seed=3),
    synth.MoEConfig("one-expert", T=300, d=192, f=448, E=1, k=1, G=1, seed=6),
    synth.MoEConfig("topk16", T=130, d=128, f=64, E=64, k=16, G=8, score_fn=1, seed=13),
    synth.MoEConfig("rows257", T=257, d=64, f=192, E=2, k=2, G=1, seed=10),
    synth.MoEConfig("T1", T=1, d=64, f=64, E=8, k=2, G=2, seed=9),
]


@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: c.name)
def test_backward_matches_oracle(cfg):
    bw = Backward(cfg)
    bw()
    run = bw.run
    xb = H.bf16_host(run.t["x"])
    dy = O.bf16_to_f64(H.bf16_host(bw.dy))[: cfg.T]
    idx, w = run.host_idx(), run.host_w()
    w1, w3, w2 = (H.bf16_host(run.t[n]) for n in ("w1", "w3", "w2"))
    dx_ref, grads = O.layer_backward(xb, idx, w, w1, w3, w2, dy)
    close(O.bf16_to_f64(H.bf16_host(bw.dx))[: cfg.T], dx_ref, "dx")
    g1 = O.bf16_to_f64(H.bf16_host(bw.dw1))
    g3 = O.bf16_to_f64(H.bf16_host(bw.dw3))
    g2 = O.bf16_to_f64(H.bf16_host(bw.dw2))
    r1, r3, r2 = np.zeros_like(g1), np.zeros_like(g3), np.zeros_like(g2)
    for e, (a, b, c) in grads.items():
        r1[e], r3[e], r2[e] = a, b, c
    close(g1, r1, "dW1")
    close(g3, r3, "dW3")
    close(g2, r2, "dW2")
    unused = [e for e in range(cfg.E) if e not in grads]
    for e in unused:                                   # experts nobody selected: exact zeros, not stale memory
        assert not g1[e].any() and not g3[e].any() and not g2[e].any(), e
    # a second call on the same workspace gives the same bits
    keep = [t.clone() for t in (bw.dx, bw.dw1, bw.dw3, bw.dw2)]
    bw()
    for a, b in zip(keep, (bw.dx, bw.dw1, bw.dw3, bw.dw2)):
        assert torch.equal(a, b)


def test_backward_rejects_forward_only_flags_and_short_workspace():
    cfg = synth.CONFIGS["C1"]
    bw = Backward(cfg)
    r, t = bw.run, bw.run.t
    with pytest.raises(B.MoEError):
        B.moe_layer_backward(B.make_shape(cfg, B.MOE_FLAG_FUSED_FFN), t["x"], bw.dy, r.idx, r.w, r.lay, t["w1"], t["w3"],
                             t["w2"], bw.dx, bw.dw1, bw.dw3, bw.dw2, bw.ws)
    with pytest.raises(B.MoEError) as ei:
        B.moe_layer_backward(r.shape, t["x"], bw.dy, r.idx, r.w, r.lay, t["w1"], t["w3"], t["w2"], bw.dx, bw.dw1, bw.dw3,
                             bw.dw2, bw.ws[:4096])
    assert ei.value.code == B.MOE_ERR_WORKSPACE_TOO_SMALL


class Slabs:
    def __init__(self, w):
        self.w = w

    def __getitem__(self, e):
        return synth.bf16_bits(self.w[int(e)])


@pytest.mark.parametrize("name", ["C3", "C4", "C5a"])
def test_backward_fullsize_sampled(name):
    """Full size (C4: 131 072 expert rows; C3: Zipf-skewed with empty and tiny experts; C5a: the benchmark's workload,
    262 144 expert rows, 22.5 GB of weights and as much of gradients): weight gradients of the most
    loaded, the least loaded and two more experts in full, dx on 24 sampled tokens."""
    cfg = synth.ALL_CONFIGS[name]
    bw = Backward(cfg)
    bw()
    run = bw.run
    idx, w = run.host_idx(), run.host_w()
    xb = H.bf16_host(run.t["x"])
    dy = O.bf16_to_f64(H.bf16_host(bw.dy))
    counts = np.bincount(idx.reshape(-1), minlength=cfg.E)
    live = np.nonzero(counts)[0]
    picks = sorted({int(live[np.argmax(counts[live])]), int(live[np.argmin(counts[live])]), int(live[len(live) // 3]),
                    int(live[-1])})
    w1, w3, w2 = Slabs(run.t["w1"]), Slabs(run.t["w3"]), Slabs(run.t["w2"])
    _, grads = O.layer_backward(xb, idx, w, w1, w3, w2, dy, experts=picks)
    for e in picks:
        close(O.bf16_to_f64(H.bf16_host(bw.dw1[e])), grads[e][0], f"{name} dW1[{e}]")
        close(O.bf16_to_f64(H.bf16_host(bw.dw3[e])), grads[e][1], f"{name} dW3[{e}]")
        close(O.bf16_to_f64(H.bf16_host(bw.dw2[e])), grads[e][2], f"{name} dW2[{e}]")
    for e in np.nonzero(counts == 0)[0][:4]:
        assert not bw.dw1[int(e)].any() and not bw.dw2[int(e)].any()
    toks = synth.sample_tokens(cfg, 96)[::4][:24]
    dx_ref, _ = O.layer_backward(xb[toks], idx[toks], w[toks], w1, w3, w2, dy[toks])
    close(O.bf16_to_f64(H.bf16_host(bw.dx[torch.from_numpy(toks).cuda()])), dx_ref, f"{name} dx")


GATE_CASES = SMALL + [
    synth.MoEConfig("sigmoid-locality", T=260, d=192, f=256, E=16, k=4, G=4, score_fn=1, bias="locality", seed=21),
    synth.MoEConfig("softmax-zipf-k8", T=200, d=256, f=128, E=32, k=8, G=8, bias="zipf", zipf_s=1.1, seed=22),
]


def _gate_backward(bw):
    run, cfg = bw.run, bw.cfg
    dwg = torch.full((cfg.d, cfg.E), 7.0, dtype=torch.float32, device="cuda")
    B.moe_gate_backward(run.shape, run.logits, run.t["bias"], run.idx, run.w, run.lay, run.t["w_gate"], bw.dx, dwg, bw.ws)
    torch.cuda.synchronize()
    st = B.moe_status(bw.ws)
    assert st[0] == 0 and st[4] == 0, f"device status {st}"
    return dwg


@pytest.mark.parametrize("cfg", GATE_CASES, ids=lambda c: c.name)
def test_gate_backward_matches_oracle(cfg):
    """moe_layer_backward followed by moe_gate_backward: dw_gate against the oracle's gate gradient, the total dx
    against expert path + gate path; softmax and sigmoid scores, no bias / per-expert bias / per-token bias."""
    bw = Backward(cfg)
    bw()
    run = bw.run
    dx_experts = bw.dx.clone()
    dwg = _gate_backward(bw)
    xb = H.bf16_host(run.t["x"])
    dy = O.bf16_to_f64(H.bf16_host(bw.dy))[: cfg.T]
    idx, w = run.host_idx(), run.host_w()
    w1, w3, w2 = (H.bf16_host(run.t[n]) for n in ("w1", "w3", "w2"))
    wg = run.t["w_gate"].cpu().numpy()
    dwg_ref, dxg_ref, dkey_ref, _ = O.gate_backward(xb, wg, run.host_bias(), idx, cfg.score_fn, w1, w3, w2, dy)
    got = dwg.cpu().numpy().astype(np.float64)
    if cfg.k == 1:
        # a single selected expert has weight 1 whatever its key: nothing reaches the gate, exactly
        assert not got.any() and torch.equal(bw.dx, dx_experts)
        assert np.abs(dwg_ref).max() <= 1e-12
        return
    if cfg.T >= 16:
        close(got, dwg_ref, "dw_gate")
    else:
        # one token: every entry of dw_gate carries the same two key gradients, so nothing averages out and the
        # mean error IS the error of one bf16-rounded dot product; only the max bar applies
        mx, _ = H.out_errors(got, dwg_ref)
        assert mx <= MAX_REL, f"dw_gate: max rel {mx:.3e}"
    dx_ref, _ = O.layer_backward(xb, idx, w, w1, w3, w2, dy)
    close(O.bf16_to_f64(H.bf16_host(bw.dx))[: cfg.T], dx_ref + dxg_ref, "dx with the gate path")
    # the gate path by itself: what the call added to dx (bf16 roundings of both sides allowed for)
    added = O.bf16_to_f64(H.bf16_host(bw.dx))[: cfg.T] - O.bf16_to_f64(H.bf16_host(dx_experts))[: cfg.T]
    tol = 2.0 ** -7 * np.abs(dx_ref + dxg_ref) + 2e-2 * np.abs(dxg_ref).max()
    assert np.all(np.abs(added - dxg_ref) <= tol), "gate path of dx"
    # columns of experts nobody selected are exact zeros
    unused = np.setdiff1d(np.arange(cfg.E), np.unique(idx))
    assert not got[:, unused].any()
    # deterministic: the whole backward again gives the same bits
    keep = (bw.dx.clone(), dwg.clone())
    bw()
    dwg2 = _gate_backward(bw)
    assert torch.equal(keep[0], bw.dx) and torch.equal(keep[1], dwg2)


def test_gate_backward_argument_checks():
    cfg = synth.MoEConfig("sig", T=64, d=64, f=64, E=8, k=2, G=2, score_fn=1, seed=5)
    bw = Backward(cfg)
    bw()
    run = bw.run
    dwg = torch.zeros(cfg.d, cfg.E, dtype=torch.float32, device="cuda")
    with pytest.raises(B.MoEError) as ei:      # sigmoid scores need the forward's logits
        B.moe_gate_backward(run.shape, None, run.t["bias"], run.idx, run.w, run.lay, run.t["w_gate"], bw.dx, dwg, bw.ws)
    assert ei.value.code == B.MOE_ERR_INVALID_ARG
    with pytest.raises(B.MoEError) as ei:
        B.moe_gate_backward(run.shape, run.logits, run.t["bias"], run.idx, run.w, run.lay, run.t["w_gate"], bw.dx, dwg,
                            bw.ws[:4096])
    assert ei.value.code == B.MOE_ERR_WORKSPACE_TOO_SMALL


def test_gate_backward_fullsize_sampled():
    """C4 at full size (per-token locality bias, softmax): the dw_gate columns of four experts in full and the total dx
    on 16 sampled tokens.  The oracle needs dL/dw of every pair of the sampled experts / tokens only."""
    cfg = synth.ALL_CONFIGS["C4"]
    bw = Backward(cfg)
    bw()
    run = bw.run
    dwg = _gate_backward(bw)
    idx, w = run.host_idx(), run.host_w()
    xb = H.bf16_host(run.t["x"])
    dy = O.bf16_to_f64(H.bf16_host(bw.dy))
    wg = run.t["w_gate"].cpu().numpy()
    bias = run.host_bias()
    w1, w3, w2 = Slabs(run.t["w1"]), Slabs(run.t["w3"]), Slabs(run.t["w2"])
    # tokens: a sample for dx, plus every token of two lightly loaded experts for their dw_gate columns
    counts = np.bincount(idx.reshape(-1), minlength=cfg.E)
    picks = [int(e) for e in np.argsort(counts)[:2]]
    toks = synth.sample_tokens(cfg, 64)[::4][:16]
    need = np.unique(np.concatenate([toks] + [np.nonzero((idx == e).any(axis=1))[0] for e in picks]))
    b = None if bias is None else (bias if bias.ndim == 1 else bias[need])
    _, dxg, dkey, _ = O.gate_backward(xb[need], wg, b, idx[need], cfg.score_fn, w1, w3, w2, dy[need])
    x64 = O.bf16_to_f64(xb[need])
    got = dwg.cpu().numpy().astype(np.float64)
    for e in picks:
        col = np.zeros(cfg.d)
        hit_t, hit_j = np.nonzero(idx[need] == e)
        col = (dkey[hit_t, hit_j][:, None] * x64[hit_t]).sum(axis=0)
        close(got[:, e], col, f"dw_gate[:, {e}]")
    pos = np.searchsorted(need, toks)
    dx_ref, _ = O.layer_backward(xb[toks], idx[toks], w[toks], w1, w3, w2, dy[toks])
    close(O.bf16_to_f64(H.bf16_host(bw.dx[torch.from_numpy(toks).cuda()])), dx_ref + dxg[pos], "C4 dx with the gate path")


def test_backward_on_a_sparse_routing_table():
    """MOE_FLAG_SPARSE_TOPK (slots of topk_idx may be -1, one token without any slot): dx and the weight gradients
    against the oracle restricted to the slots in use; the token without slots gets a zero row of dx."""
    cfg = synth.MoEConfig("sparse-bwd", T=300, d=128, f=192, E=12, k=4, G=3, seed=21)
    run = H.Run(cfg, B.MOE_FLAG_SPARSE_TOPK)
    run.route()
    rng = np.random.default_rng(3)
    idx = run.host_idx().copy()
    drop = rng.random(idx.shape) < 0.4
    drop[5] = True
    drop[6] = False
    idx[drop] = -1
    run.idx[: cfg.P] = torch.from_numpy(idx.reshape(-1)).cuda()
    run.dispatch()
    g = torch.Generator(device="cuda")
    g.manual_seed(5)
    dy = torch.randn(cfg.T, cfg.d, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    dx = torch.full((cfg.T, cfg.d), 7.0, dtype=torch.bfloat16, device="cuda")
    dw = {n: torch.full_like(run.t[n], 7.0) for n in ("w1", "w3", "w2")}
    ws = torch.zeros(B.moe_backward_workspace_bytes(run.shape), dtype=torch.uint8, device="cuda")
    B.moe_layer_backward(run.shape, run.t["x"], dy, run.idx, run.w, run.lay, run.t["w1"], run.t["w3"], run.t["w2"], dx,
                         dw["w1"], dw["w3"], dw["w2"], ws)
    torch.cuda.synchronize()
    assert B.moe_status(ws)[0] == 0
    w1, w3, w2 = (H.bf16_host(run.t[n]) for n in ("w1", "w3", "w2"))
    dx_ref, grads = O.layer_backward(H.bf16_host(run.t["x"]), idx, run.host_w(), w1, w3, w2,
                                     O.bf16_to_f64(H.bf16_host(dy)))
    got = O.bf16_to_f64(H.bf16_host(dx))
    close(got, dx_ref, "sparse dx")
    assert not got[5].any() and not dx_ref[5].any()
    for n, pos in (("w1", 0), ("w3", 1), ("w2", 2)):
        ref = np.zeros(tuple(run.t[n].shape))
        for e, gr in grads.items():
            ref[e] = gr[pos]
        close(O.bf16_to_f64(H.bf16_host(dw[n])), ref, f"sparse d{n}")
