"""Full-size parity: the five benchmark configurations through moe_layer (the launch configuration
bench.py times).  Routing and layout are compared in full (bit-exact); expert outputs on sampled
rows of sampled experts and the layer output on sampled tokens, one by one against the oracle."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2605_05607_b200 import binding as B
from paper_2605_05607_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


class Slabs:
    """Expert weight matrices fetched from the device one expert at a time."""

    def __init__(self, w):
        self.w = w

    def __getitem__(self, e):
        return synth.bf16_bits(self.w[int(e)])


def sample_expert_rows(lay, E, rng, per_expert=2, spread=32):
    """Rows to check expert outputs on: the first and the last row of `spread` experts taken evenly over [0, E)
    (so a wrong tile decode of any region of the expert range shows), plus the most and the least loaded expert
    with a few more rows each (first / last / random: both ends of the m-tile range, partial tiles)."""
    counts = lay["expert_counts"]
    off = lay["expert_offsets"].astype(np.int64)
    live = np.nonzero(counts)[0]
    rows = []
    for e in np.unique(live[np.linspace(0, live.size - 1, min(spread, live.size)).astype(np.int64)]):
        rows += [off[e], off[e + 1] - 1][:per_expert]
    for e in (int(live[np.argmax(counts[live])]), int(live[np.argmin(counts[live])])):
        lo, hi = int(off[e]), int(off[e + 1])
        rows += list(range(lo, min(lo + 4, hi))) + list(range(max(hi - 4, lo), hi)) + list(rng.integers(lo, hi, size=4))
    return np.unique(np.asarray(rows, dtype=np.int64))


# C2..C5b: the benchmark configurations; S32 / M16 / L32: three of the paper's own evaluation shapes
# (Small at top-32 of 64 experts, Medium at top-16, Large at top-32: 2^20 expert rows, element
# offsets beyond 2^32 in o), 32 groups.  Two more rows run a layer option at full size: Combine inside GEMM-2's
# epilogue on C4 (its fp32 accumulators outgrow L2 only at this size) and the gate weight applied in Combine on C3.
@pytest.mark.parametrize("name,flags", [("C2", 0), ("C3", 0), ("C4", 0), ("C5a", 0), ("C5b", 0), ("S32", 0), ("M16", 0),
                                        ("L32", 0), ("C4", B.MOE_FLAG_COMBINE_IN_EPILOGUE),
                                        ("C3", B.MOE_FLAG_WEIGHT_IN_COMBINE)])
def test_fullsize_layer(name, flags):
    cfg = synth.ALL_CONFIGS[name]
    run = H.Run(cfg, flags)
    lay_dev = B.alloc_layout(run.shape)
    run.layer(logits=run.logits, topk_idx=run.idx, topk_w=run.w, layout=lay_dev)
    torch.cuda.synchronize()
    st = run.status()
    assert st[0] == 0 and st[4] == 0, f"device status {st}"
    run.lay = lay_dev
    idx_ref, w_ref = H.check_route(run)               # logits 1e-4; idx bit-exact; weights 1e-6
    lay = H.check_layout(run, idx_ref)                # counts / offsets / permutation bit-exact
    P, T, k = cfg.P, cfg.T, cfg.k
    assert lay["n_disp"] <= T * min(k, cfg.G)
    if cfg.G == cfg.E:
        assert lay["n_disp"] == P                     # one expert per group: nothing to de-duplicate
    xb = H.bf16_host(run.t["x"])
    w_gpu = run.host_w()
    in_combine = bool(flags & B.MOE_FLAG_WEIGHT_IN_COMBINE)

    if not flags & B.MOE_FLAG_COMBINE_IN_EPILOGUE:    # (that form never writes o)
        # expert outputs o (kept in the workspace by moe_layer): two rows of 32 experts spread over the expert range,
        # more rows of the most and the least loaded expert
        off = B.moe_workspace_layout(run.shape)
        o_dev = run.ws[off["o"]: off["o"] + P * cfg.d * 2].view(torch.bfloat16).reshape(P, cfg.d)
        rows = sample_expert_rows(lay, cfg.E, np.random.default_rng(1))
        # the fused path feeds GEMM-1 from x; the oracle's dispatched copy holds the same bytes
        xg = O.dispatch(xb, lay)
        o_ref = O.expert_ffn(xg, lay, None if in_combine else w_gpu, Slabs(run.t["w1"]), Slabs(run.t["w3"]),
                             Slabs(run.t["w2"]), rows=rows)
        o_gpu = O.bf16_to_f64(H.bf16_host(o_dev[torch.from_numpy(rows).cuda()]))
        H.assert_close_out(o_gpu, o_ref, f"{name} expert rows")

        # combine on sampled tokens from the GPU's own o (all k rows of each token)
        toks = synth.sample_tokens(cfg, 96)
        need = np.unique(lay["pair_row"].reshape(T, k)[toks].reshape(-1))
        o_need = O.bf16_to_f64(H.bf16_host(o_dev[torch.from_numpy(need).cuda()]))
        _, _, y_ref = O.combine(o_need, lay, idx_ref, w_gpu if in_combine else None, cfg.E, cfg.G, tokens=toks,
                                o_rows=need)
        y_gpu = O.bf16_to_f64(H.bf16_host(run.y[torch.from_numpy(toks).cuda()]))
        tol = 2.0 ** -8 * np.abs(y_ref) + 2.0 ** -22 * np.abs(y_ref).max() + 1e-30
        assert np.all(np.abs(y_gpu - y_ref) <= tol), f"{name} combine"

    # whole layer against the dense definition on 16 tokens spread over the batch (first, last and between)
    few = synth.sample_tokens(cfg, 96)[:: 96 // 16][:16]
    b = run.host_bias()
    _, _, _, y_def = O.layer(xb, run.host_logits(), b, Slabs(run.t["w1"]), Slabs(run.t["w3"]), Slabs(run.t["w2"]),
                             k, cfg.score_fn, tokens=few)
    y_few = O.bf16_to_f64(H.bf16_host(run.y[torch.from_numpy(few).cuda()]))
    H.assert_close_out(y_few, y_def, f"{name} layer y")


class QuantSlabs:
    """Per-expert FP8 weights computed by the oracle from the bf16 slab of that expert only."""

    def __init__(self, w, which):
        from oracle import fp8_oracle as F
        self.w, self.which, self.F, self.cache = w, which, F, {}
        self.shape = (w.shape[0], w.shape[2], w.shape[1])          # [E, N, K]

    def __getitem__(self, e):
        e = int(e)
        if e not in self.cache:
            q, s = self.F.quantize_weights(O.bf16_to_f64(synth.bf16_bits(self.w[e]))[None])
            self.cache[e] = (q[0], s[0])
        return self.cache[e][self.which]


@pytest.mark.parametrize("name", ["C4", "S32", "C5a"])
def test_fullsize_layer_fp8(name):
    """moe_layer_fp8 at full size: routing and layout in full, quantised operands bit for bit on
    sampled experts, expert outputs on sampled rows and the layer output on sampled tokens."""
    from oracle import fp8_oracle as F
    cfg = synth.ALL_CONFIGS[name]
    run = H.Run(cfg)
    t = run.t
    E, d, f, P, T, k = cfg.E, cfg.d, cfg.f, cfg.P, cfg.T, cfg.k
    wq, sc = {}, {}
    for nm, (K, N) in (("w1", (d, f)), ("w3", (d, f)), ("w2", (f, d))):
        wq[nm] = torch.zeros(E, N, K, dtype=torch.uint8, device="cuda")
        sc[nm] = torch.zeros(E, N, dtype=torch.float32, device="cuda")
        B.moe_quantize_weights(t[nm], wq[nm], sc[nm])
    lay_dev = B.alloc_layout(run.shape)
    B.moe_layer_fp8(run.shape, t["x"], t["w_gate"], t["bias"], wq["w1"], sc["w1"], wq["w3"], sc["w3"], wq["w2"],
                    sc["w2"], run.y, run.ws, logits=run.logits, topk_idx=run.idx, topk_w=run.w, layout=lay_dev)
    torch.cuda.synchronize()
    st = run.status()
    assert st[0] == 0 and st[4] == 0, f"device status {st}"
    run.lay = lay_dev
    idx_ref, _ = H.check_route(run)
    lay = H.check_layout(run, idx_ref)
    counts = lay["expert_counts"]
    live = np.nonzero(counts)[0]
    rng = np.random.default_rng(2)
    picks = sorted({int(live[np.argmax(counts[live])]), int(live[np.argmin(counts[live])]), int(rng.choice(live))})
    slabs = {nm: (QuantSlabs(t[nm], 0), QuantSlabs(t[nm], 1)) for nm in ("w1", "w3", "w2")}
    for e in picks:      # the GPU's quantised weights of the sampled experts, bit for bit
        for nm in ("w1", "w3", "w2"):
            assert np.array_equal(wq[nm][e].cpu().numpy(), slabs[nm][0][e]), (nm, e)
            assert np.array_equal(sc[nm][e].cpu().numpy(), slabs[nm][1][e]), (nm, e)
    rows = []
    for e in picks:
        lo, hi = int(lay["expert_offsets"][e]), int(lay["expert_offsets"][e + 1])
        rows.append(np.unique(np.concatenate([np.arange(lo, min(lo + 6, hi)), np.arange(max(hi - 6, lo), hi),
                                              rng.integers(lo, hi, size=6)])))
    rows = np.unique(np.concatenate(rows))
    xq, sx = F.quantize_rows(O.bf16_to_f64(H.bf16_host(t["x"])))
    dt = lay["disp_token"].astype(np.int64)
    o_ref = F.expert_ffn_fp8(xq[dt], sx[dt], lay, run.host_w(), slabs["w1"][0], slabs["w1"][1], slabs["w3"][0],
                             slabs["w3"][1], slabs["w2"][0], slabs["w2"][1], rows=rows)
    off = B.moe_workspace_layout(run.shape)
    o_dev = run.ws[off["o"]: off["o"] + P * d * 2].view(torch.bfloat16).reshape(P, d)
    o_gpu = O.bf16_to_f64(H.bf16_host(o_dev[torch.from_numpy(rows).cuda()]))
    H.assert_close_out(o_gpu, o_ref, f"{name} fp8 expert rows")
    # combine on sampled tokens from the GPU's own o
    toks = synth.sample_tokens(cfg, 64)
    need = np.unique(lay["pair_row"].reshape(T, k)[toks].reshape(-1))
    o_need = O.bf16_to_f64(H.bf16_host(o_dev[torch.from_numpy(need).cuda()]))
    _, _, y_ref = O.combine(o_need, lay, idx_ref, None, E, cfg.G, tokens=toks, o_rows=need)
    y_gpu = O.bf16_to_f64(H.bf16_host(run.y[torch.from_numpy(toks).cuda()]))
    tol = 2.0 ** -8 * np.abs(y_ref) + 2.0 ** -22 * np.abs(y_ref).max() + 1e-30
    assert np.all(np.abs(y_gpu - y_ref) <= tol), f"{name} fp8 combine"


@pytest.mark.parametrize("name", ["C4", "C3"])
def test_fullsize_single_kernel_ffn_equals_two_kernels(name):
    """MOE_FLAG_FUSED_FFN at full size (C4: 131 072 expert rows in 1 024-row experts; C3: Zipf-skewed, empty and
    tiny experts): the tracker-paced single kernel writes the same o, bit for bit, as GEMM-1 followed by GEMM-2."""
    cfg = synth.ALL_CONFIGS[name]
    run = H.Run(cfg)
    run.route()
    run.dispatch()
    run.ffn()
    o_two = run.o.clone()
    F, PART, DISP = B.MOE_FLAG_FUSED_FFN, B.MOE_FLAG_SM_PARTITION, B.MOE_FLAG_TRACK_DISPATCH
    for flags in (F, F | PART, F | DISP):
        fused = H.Run(cfg, flags, inputs=run.t)
        fused.idx, fused.w, fused.lay, fused.xg = run.idx, run.w, run.lay, run.xg
        fused.o.fill_(3.0)
        fused.ffn()
        torch.cuda.synchronize()
        assert fused.status()[0] == 0, flags
        assert torch.equal(fused.o[: cfg.P], o_two[: cfg.P]), flags
        del fused


@pytest.mark.parametrize("name", ["C3", "C4", "C5a"])
def test_fullsize_tracker_paced_layer_equals_the_separate_kernels(name):
    """The whole layer after the layout as one tracker-paced kernel (GEMM-1, GEMM-2 and Combine tasks; with
    MOE_FLAG_TRACK_DISPATCH also Dispatch tasks; interleaved and with the SM partition) at full size: y must equal
    the default path (separate GEMM and combine kernels, itself held to the oracle above) bit for bit, and so must
    the CTA-pair GEMM-1 on the per-expert layout tensors."""
    cfg = synth.ALL_CONFIGS[name]
    run = H.Run(cfg)
    run.layer()
    torch.cuda.synchronize()
    assert run.status()[0] == 0
    y_ref = run.y.clone()
    F, PART, DISP = B.MOE_FLAG_FUSED_FFN, B.MOE_FLAG_SM_PARTITION, B.MOE_FLAG_TRACK_DISPATCH
    for flags in (F, F | PART, F | DISP, F | PART | DISP, B.MOE_FLAG_GEMM1_PAIR):
        other = H.Run(cfg, flags, inputs=run.t)
        for _ in range(2):                               # the tracker tables are cleared by every call
            other.y.fill_(5.0)
            other.layer()
            torch.cuda.synchronize()
            assert other.status()[0] == 0, (flags, other.status())
            assert torch.equal(other.y[: cfg.T], y_ref[: cfg.T]), flags
        del other


def test_gemm1_is_bit_reproducible_over_many_runs():
    """GEMM-1's gathered rows reach the tensor core through cp.async copies that arrive on the stage barrier by
    themselves, with no proxy fence between the copies and the UMMA that reads them.  If that publication were not
    sound, a row would now and then be multiplied before it had landed: twenty runs of the expert FFN on C4 (131 072
    rows, 4 096-deep K) must give the same o bit for bit, and the first run is held to the oracle by the tests above."""
    cfg = synth.ALL_CONFIGS["C4"]
    run = H.Run(cfg, B.MOE_FLAG_GEMM1_GATHER)
    run.route()
    run.dispatch()
    run.ffn()
    torch.cuda.synchronize()
    first = run.o.clone()
    for i in range(20):
        run.o.fill_(1.0)
        run.ffn()
        torch.cuda.synchronize()
        assert torch.equal(run.o[: cfg.P], first[: cfg.P]), i
    assert run.status()[0] == 0
