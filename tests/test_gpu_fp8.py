"""GPU parity of the FP8 (E4M3) form of the expert FFN against its oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import fp8_oracle as F
from oracle import moe_oracle as O
from paper_2605_05607_b200 import binding as B
from paper_2605_05607_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_quantize_rows_bit_exact():
    g = torch.Generator(device="cuda").manual_seed(5)
    x = (torch.randn(300, 200, generator=g, device="cuda") * 3).to(torch.bfloat16)
    x[7] = 0
    x[9, 3] = 1e30                                   # a huge element: everything else in the row underflows
    q = torch.zeros(300, 200, dtype=torch.uint8, device="cuda")
    s = torch.zeros(300, dtype=torch.float32, device="cuda")
    B.moe_quantize_rows(x, q, s)
    q_ref, s_ref = F.quantize_rows(O.bf16_to_f64(H.bf16_host(x)))
    assert np.array_equal(s.cpu().numpy(), s_ref)
    assert np.array_equal(q.cpu().numpy(), q_ref)


def test_quantize_weights_bit_exact():
    g = torch.Generator(device="cuda").manual_seed(6)
    w = (torch.randn(3, 70, 45, generator=g, device="cuda") * 0.1).to(torch.bfloat16)   # ragged in K and N
    wq = torch.zeros(3, 45, 70, dtype=torch.uint8, device="cuda")
    s = torch.zeros(3, 45, dtype=torch.float32, device="cuda")
    B.moe_quantize_weights(w, wq, s)
    q_ref, s_ref = F.quantize_weights(O.bf16_to_f64(H.bf16_host(w)))
    assert np.array_equal(s.cpu().numpy(), s_ref)
    assert np.array_equal(wq.cpu().numpy(), q_ref)


FP8_CASES = [
    synth.CONFIGS["C1"],
    synth.MoEConfig("fp8-ragged", T=333, d=208, f=176, E=6, k=3, G=3, seed=3),          # K and N tails, partial tiles
    synth.MoEConfig("fp8-sigmoid", T=700, d=384, f=640, E=16, k=4, G=4, score_fn=1, bias="zipf", zipf_s=1.0, seed=4),
]


@pytest.mark.parametrize("cfg", FP8_CASES, ids=lambda c: c.name)
def test_expert_ffn_fp8_matches_its_oracle(cfg):
    run = H.Run(cfg)
    run.route()
    run.dispatch()
    idx_ref, _ = H.check_route(run)
    lay = H.check_layout(run, idx_ref)
    t = run.t
    E, d, f = cfg.E, cfg.d, cfg.f
    dev = "cuda"
    rows = run.xg.shape[0]
    xq = torch.zeros(rows, d, dtype=torch.uint8, device=dev)
    sx = torch.zeros(rows, dtype=torch.float32, device=dev)
    B.moe_quantize_rows(run.xg, xq, sx)
    wq, ws_ = {}, {}
    for name, (K, N) in (("w1", (d, f)), ("w3", (d, f)), ("w2", (f, d))):
        wq[name] = torch.zeros(E, N, K, dtype=torch.uint8, device=dev)
        ws_[name] = torch.zeros(E, N, dtype=torch.float32, device=dev)
        B.moe_quantize_weights(t[name], wq[name], ws_[name])
    B.moe_expert_ffn_fp8(run.shape, xq, sx, run.lay, run.w, wq["w1"], ws_["w1"], wq["w3"], ws_["w3"],
                         wq["w2"], ws_["w2"], run.o, run.ws)
    torch.cuda.synchronize()
    assert run.status()[0] == 0
    n = lay["n_disp"]
    # quantised operands are compared bit for bit first (both sides take the rounding decisions in fp32)
    xq_ref, sx_ref = F.quantize_rows(O.bf16_to_f64(H.bf16_host(run.xg)[:n]))
    assert np.array_equal(xq.cpu().numpy()[:n], xq_ref) and np.array_equal(sx.cpu().numpy()[:n], sx_ref)
    ref_w = {}
    for name in ("w1", "w3", "w2"):
        ref_w[name] = F.quantize_weights(O.bf16_to_f64(H.bf16_host(t[name])))
        assert np.array_equal(wq[name].cpu().numpy(), ref_w[name][0]), name
        assert np.array_equal(ws_[name].cpu().numpy(), ref_w[name][1]), name
    o_ref = F.expert_ffn_fp8(xq_ref, sx_ref, lay, run.host_w(), *ref_w["w1"], *ref_w["w3"], *ref_w["w2"])
    o_gpu = O.bf16_to_f64(H.bf16_host(run.o)[: cfg.P])
    H.assert_close_out(o_gpu, o_ref, "fp8 expert_ffn o")
    # and the FP8 result stays within the format's error of the exact (unquantised) FFN
    xg_ref = O.dispatch(H.bf16_host(t["x"]), lay)
    o_exact = O.expert_ffn(xg_ref, lay, run.host_w(), H.bf16_host(t["w1"]), H.bf16_host(t["w3"]), H.bf16_host(t["w2"]))
    mx, mean = H.out_errors(o_gpu, o_exact)
    assert mean < 8e-2, (mx, mean)


def test_fp8_shape_limits():
    cfg = synth.MoEConfig("fp8-bad", T=16, d=72, f=64, E=4, k=2, G=2)     # d % 16 != 0
    run = H.Run(cfg, inputs=synth.make_routing_inputs(cfg, "cuda") | {"w1": None, "w3": None, "w2": None})
    z8 = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    zf = torch.zeros(1024, dtype=torch.float32, device="cuda")
    with pytest.raises(B.MoEError) as ei:
        B.moe_expert_ffn_fp8(run.shape, z8, zf, run.lay, zf, z8, zf, z8, zf, z8, zf, run.o, run.ws)
    assert ei.value.code == B.MOE_ERR_UNSUPPORTED_SHAPE


def _quantized_weights(t, cfg):
    E, d, f = cfg.E, cfg.d, cfg.f
    wq, sc = {}, {}
    for name, (K, N) in (("w1", (d, f)), ("w3", (d, f)), ("w2", (f, d))):
        wq[name] = torch.zeros(E, N, K, dtype=torch.uint8, device="cuda")
        sc[name] = torch.zeros(E, N, dtype=torch.float32, device="cuda")
        B.moe_quantize_weights(t[name], wq[name], sc[name])
    return wq, sc


@pytest.mark.parametrize("cfg", FP8_CASES, ids=lambda c: c.name)
@pytest.mark.parametrize("flags", [0, B.MOE_FLAG_COMBINE_IN_EPILOGUE, B.MOE_FLAG_WEIGHT_IN_COMBINE],
                         ids=["combine-kernel", "combine-in-epilogue", "weight-in-combine"])
def test_layer_fp8_matches_its_oracle(cfg, flags):
    run = H.Run(cfg, flags)
    t = run.t
    wq, sc = _quantized_weights(t, cfg)
    lay_dev = B.alloc_layout(run.shape)
    for _ in range(2):
        run.y.fill_(3.0)
        B.moe_layer_fp8(run.shape, t["x"], t["w_gate"], t["bias"], wq["w1"], sc["w1"], wq["w3"], sc["w3"], wq["w2"],
                        sc["w2"], run.y, run.ws, logits=run.logits, topk_idx=run.idx, topk_w=run.w, layout=lay_dev)
    torch.cuda.synchronize()
    assert run.status()[0] == 0
    run.lay = lay_dev
    idx_ref, _ = H.check_route(run)          # routing runs on the bf16 activations, as in moe_layer
    lay = H.check_layout(run, idx_ref)
    # per-token quantisation commutes with the dispatch copy: quantise x, then take the dispatched rows
    xq, sx = F.quantize_rows(O.bf16_to_f64(H.bf16_host(t["x"])))
    dt = lay["disp_token"].astype(np.int64)
    ref_w = {n: F.quantize_weights(O.bf16_to_f64(H.bf16_host(t[n]))) for n in ("w1", "w3", "w2")}
    in_combine = bool(flags & B.MOE_FLAG_WEIGHT_IN_COMBINE)
    o_ref = F.expert_ffn_fp8(xq[dt], sx[dt], lay, None if in_combine else run.host_w(), *ref_w["w1"], *ref_w["w3"],
                             *ref_w["w2"])
    _, _, y_ref = O.combine(o_ref, lay, idx_ref, run.host_w() if in_combine else None, cfg.E, cfg.G)
    y_gpu = O.bf16_to_f64(H.bf16_host(run.y)[: cfg.T])
    H.assert_close_out(y_gpu, y_ref, "fp8 layer y")


def test_fp8_random_shape_sweep():
    """Seeded sweep over small random shapes for the FP8 layer: ragged T, K and N tails (any multiple of 16),
    k / G / E combinations, both score functions, all three flag settings."""
    rng = np.random.default_rng(77)
    flag_cycle = [0, B.MOE_FLAG_COMBINE_IN_EPILOGUE, B.MOE_FLAG_WEIGHT_IN_COMBINE]
    for i in range(9):
        E = int(rng.choice([1, 2, 4, 6, 8, 12, 24]))
        G = int(rng.choice([g for g in range(1, E + 1) if E % g == 0]))
        k = int(rng.integers(1, min(E, 5) + 1))
        cfg = synth.MoEConfig(f"fp8sweep{i}", T=int(rng.integers(1, 400)), d=16 * int(rng.integers(1, 24)),
                              f=16 * int(rng.integers(1, 24)), E=E, k=k, G=G, score_fn=int(rng.integers(0, 2)),
                              bias=str(rng.choice(["none", "zipf"])), zipf_s=1.0, seed=300 + i)
        flags = flag_cycle[i % 3]
        run = H.Run(cfg, flags)
        t = run.t
        wq, sc = _quantized_weights(t, cfg)
        lay_dev = B.alloc_layout(run.shape)
        B.moe_layer_fp8(run.shape, t["x"], t["w_gate"], t["bias"], wq["w1"], sc["w1"], wq["w3"], sc["w3"], wq["w2"],
                        sc["w2"], run.y, run.ws, logits=run.logits, topk_idx=run.idx, topk_w=run.w, layout=lay_dev)
        torch.cuda.synchronize()
        assert run.status()[0] == 0, cfg
        run.lay = lay_dev
        idx_ref, _ = H.check_route(run)
        lay = H.check_layout(run, idx_ref)
        xq, sx = F.quantize_rows(O.bf16_to_f64(H.bf16_host(t["x"])))
        dt = lay["disp_token"].astype(np.int64)
        ref_w = {n: F.quantize_weights(O.bf16_to_f64(H.bf16_host(t[n]))) for n in ("w1", "w3", "w2")}
        in_combine = bool(flags & B.MOE_FLAG_WEIGHT_IN_COMBINE)
        o_ref = F.expert_ffn_fp8(xq[dt], sx[dt], lay, None if in_combine else run.host_w(), *ref_w["w1"],
                                 *ref_w["w3"], *ref_w["w2"])
        _, _, y_ref = O.combine(o_ref, lay, idx_ref, run.host_w() if in_combine else None, cfg.E, cfg.G)
        y_gpu = O.bf16_to_f64(H.bf16_host(run.y)[: cfg.T])
        H.assert_close_out(y_gpu, y_ref, f"{cfg}")
