"""GPU parity tests: every stage of the path, called through the C ABI, against
the CPU oracle on the same seeded inputs.  Integers bit-exact; outputs within
max|gpu-ref| <= 2e-2 max|ref| and sum|gpu-ref|/sum|ref| <= 5e-3; logits 1e-4."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2605_05607_b200 import binding as B
from paper_2605_05607_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

C1 = synth.CONFIGS["C1"]
SMALL = [
    C1,
    C1.with_(name="C1-sigmoid-wcombine", score_fn=1),
    # ragged everything: T not a multiple of 32/128, d and f with K/N tails, empty experts likely
    synth.MoEConfig("ragged", T=333, d=200, f=328, E=12, k=3, G=4, bias="zipf", zipf_s=1.5, seed=2),
    synth.MoEConfig("k1", T=150, d=128, f=192, E=4, k=1, G=2, seed=3),
    synth.MoEConfig("kE-G1", T=70, d=64, f=64, E=4, k=4, G=1, seed=4),
    synth.MoEConfig("G=E-local", T=200, d=256, f=128, E=16, k=4, G=16, bias="locality", boost=2.0, seed=5),
    synth.MoEConfig("one-expert", T=300, d=192, f=448, E=1, k=1, G=1, seed=6),
    synth.MoEConfig("gptoss-ish", T=512, d=2880 // 5, f=2880 // 5, E=32, k=4, G=8, bias="zipf", zipf_s=1.1, seed=7),
    # more experts than one 256-column gate tile, experts per lane > 8 in top-k, sigmoid scores
    synth.MoEConfig("E320", T=260, d=136, f=72, E=320, k=6, G=10, score_fn=1, seed=8),
    # a single token; many tokens in a single expert pair tile boundary (257 rows: 128 + 128 + 1)
    synth.MoEConfig("T1", T=1, d=64, f=64, E=8, k=2, G=2, seed=9),
    synth.MoEConfig("rows257", T=257, d=64, f=192, E=2, k=2, G=1, seed=10),
    # the paper's evaluation sweeps top-k over 8 / 16 / 32 (Table I): many slots per token, most in one group
    synth.MoEConfig("topk16", T=130, d=128, f=64, E=64, k=16, G=8, score_fn=1, seed=13),
    synth.MoEConfig("topk32", T=90, d=64, f=64, E=64, k=32, G=4, bias="locality", boost=2.0, seed=14),
    # long K: GEMM-1 takes its split-ring pipeline (K >= 6144), with a K tail (6216 = 97 * 64 + 8)
    synth.MoEConfig("longK", T=300, d=6216, f=72, E=3, k=2, G=3, seed=11),
]


def staged(cfg, flags=0):
    run = H.Run(cfg, flags)
    run.route()
    idx_ref, w_ref = H.check_route(run)
    run.dispatch()
    lay = H.check_layout(run, idx_ref)
    n = lay["n_disp"]
    xb = H.bf16_host(run.t["x"])
    xg_ref = O.dispatch(xb, lay)
    assert np.array_equal(H.bf16_host(run.xg)[:n], xg_ref), "dispatch is not a byte copy"
    run.ffn()
    w_gpu = run.host_w()
    in_combine = bool(flags & B.MOE_FLAG_WEIGHT_IN_COMBINE)
    o_ref = O.expert_ffn(xg_ref, lay, None if in_combine else w_gpu, H.bf16_host(run.t["w1"]),
                         H.bf16_host(run.t["w3"]), H.bf16_host(run.t["w2"]))
    o_gpu = O.bf16_to_f64(H.bf16_host(run.o)[: cfg.P])
    H.assert_close_out(o_gpu, o_ref, "expert_ffn o")
    pg = torch.zeros(max(n, 1), cfg.d, dtype=torch.bfloat16, device="cuda")
    run.combine(pg)
    # combine is checked against the oracle's combine of the GPU's own o (isolates this stage)
    pg_n, pg_ref, y_ref = O.combine(o_gpu, lay, idx_ref, w_gpu if in_combine else None, cfg.E, cfg.G)
    y_gpu = O.bf16_to_f64(H.bf16_host(run.y)[: cfg.T])
    tol = 2.0 ** -8 * np.abs(y_ref) + 1e-30 + 2.0 ** -22 * np.abs(y_ref).max()
    assert np.all(np.abs(y_gpu - y_ref) <= tol), "combine y"
    pg_gpu = O.bf16_to_f64(H.bf16_host(pg)[:n])
    tol = 2.0 ** -8 * np.abs(pg_ref) + 1e-30 + 2.0 ** -22 * max(np.abs(pg_ref).max(), 1e-30)
    assert np.array_equal(pg_n, np.arange(n)) and np.all(np.abs(pg_gpu - pg_ref) <= tol), "combine pg"
    # and the whole staged path against the dense definition
    _, _, _, y_def = O.layer(xb, run.host_logits(), run.host_bias(), H.bf16_host(run.t["w1"]),
                             H.bf16_host(run.t["w3"]), H.bf16_host(run.t["w2"]), cfg.k, cfg.score_fn)
    H.assert_close_out(y_gpu, y_def, "staged y")
    st = run.status()
    assert st[0] == 0 and st[4] == 0, f"device status {st}"
    return run, y_gpu, y_def


@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: c.name)
def test_staged_path_matches_oracle(cfg):
    flags = B.MOE_FLAG_WEIGHT_IN_COMBINE if "wcombine" in cfg.name else 0
    staged(cfg, flags)


@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: c.name)
def test_fused_layer_matches_oracle_and_staged(cfg):
    run, y_staged, y_def = staged(cfg)
    y2 = torch.zeros_like(run.y)
    logits = torch.zeros_like(run.logits)
    idx = torch.zeros_like(run.idx)
    w = torch.zeros_like(run.w)
    lay2 = B.alloc_layout(run.shape)
    run.layer(y=y2, logits=logits, topk_idx=idx, topk_w=w, layout=lay2)
    assert torch.equal(idx, run.idx) and torch.equal(logits, run.logits) and torch.equal(w, run.w)
    for name in ("expert_offsets", "group_offsets", "pair_row", "row_pair", "row_src", "al"):
        assert torch.equal(getattr(lay2, name), getattr(run.lay, name)), name
    y_fused = O.bf16_to_f64(H.bf16_host(y2)[: cfg.T])
    H.assert_close_out(y_fused, y_def, "fused y")
    # gathering from x instead of the dispatched copy feeds the GEMM the same bytes
    assert np.array_equal(y_fused, y_staged)
    # optional outputs left NULL: same y
    y3 = torch.zeros_like(run.y)
    run.layer(y=y3)
    assert torch.equal(y3, y2)
    assert run.status()[0] == 0
    # Combine inside GEMM-2's epilogue (fp32 reductions in arrival order).  The default form rounds
    # every o row to bf16 before summing, this one sums unrounded fp32 rows: the two agree within
    # that rounding (k terms, 2^-9 relative each), and both meet the output bar against the oracle
    if "wcombine" not in cfg.name:
        run_e = H.Run(cfg, B.MOE_FLAG_COMBINE_IN_EPILOGUE, inputs=run.t)
        for _ in range(2):   # twice: the accumulators are cleared by every call
            y4 = torch.full_like(run.y, 7.0)
            run_e.layer(y=y4)
        y_epi = O.bf16_to_f64(H.bf16_host(y4)[: cfg.T])
        H.assert_close_out(y_epi, y_def, "epilogue-combine y")
        mx, mean = H.out_errors(y_epi, y_fused)
        assert mx <= 1e-2 and mean <= 3e-3, f"epilogue-combine y vs default fused y: {mx:.2e} {mean:.2e}"
        assert run_e.status()[0] == 0


def test_topk_ties_lowest_index_wins():
    # logits quantised to a handful of values: ties everywhere, incl. at the k / k+1 border
    cfg = synth.MoEConfig("ties", T=777, d=64, f=64, E=40, k=6, G=4)
    run = H.Run(cfg, inputs=synth.make_routing_inputs(cfg, "cuda") | {"w1": None, "w3": None, "w2": None})
    g = torch.Generator(device="cuda").manual_seed(11)
    vals = torch.tensor([-1.0, -0.0, 0.0, 0.5, 0.5, 2.0], device="cuda")
    logits = vals[torch.randint(0, 6, (cfg.T, cfg.E), generator=g, device="cuda")].contiguous()
    run.logits = logits.reshape(-1).clone()
    for score_fn in (0, 1):
        shape = B.make_shape(cfg.with_(score_fn=score_fn))
        B.moe_route(shape, None, None, None, run.logits, run.idx, run.w, run.ws)
        idx_ref, w_ref = O.route(logits.cpu().numpy(), None, cfg.k, score_fn)
        assert np.array_equal(run.host_idx(), idx_ref)
        assert np.abs(run.host_w() - w_ref).max() <= H.WEIGHT_ABS
    # all-equal keys -> experts 0..k-1, weights 1/k
    run.logits.fill_(0.25)
    B.moe_route(run.shape, None, None, None, run.logits, run.idx, run.w, run.ws)
    assert np.array_equal(run.host_idx(), np.tile(np.arange(cfg.k, dtype=np.int32), (cfg.T, 1)))
    assert np.allclose(run.host_w(), 1.0 / cfg.k, atol=1e-7)
    assert run.status()[5] == 0


def test_bias_forms_and_nonfinite_warning():
    cfg = synth.MoEConfig("bias", T=100, d=64, f=64, E=64, k=4, G=8, bias="locality", boost=2.0, seed=9)
    run = H.Run(cfg, inputs=synth.make_routing_inputs(cfg, "cuda") | {"w1": None, "w3": None, "w2": None})
    run.route()
    H.check_route(run)                                   # [T, E] bias
    zcfg = cfg.with_(bias="zipf", zipf_s=1.2)
    run2 = H.Run(zcfg, inputs=synth.make_routing_inputs(zcfg, "cuda") | {"w1": None, "w3": None, "w2": None})
    run2.route()
    H.check_route(run2)                                  # [E] bias
    assert run2.status()[5] == 0
    run2.logits[5] = float("inf")
    B.moe_route(run2.shape, None, None, run2.t["bias"], run2.logits, run2.idx, run2.w, run2.ws)
    assert run2.status()[5] & B.MOE_WARN_NONFINITE_LOGIT


def test_combine_identity_experts_and_linearity():
    # "identity experts": feed o[r] := xg[row_src[r]]; weights sum to 1, so combine returns x
    for k in (1, 2, 4):
        cfg = synth.MoEConfig(f"ident{k}", T=260, d=520, f=64, E=8, k=k, G=4, seed=k)
        run = H.Run(cfg, B.MOE_FLAG_WEIGHT_IN_COMBINE,
                    inputs=synth.make_routing_inputs(cfg, "cuda") | {"w1": None, "w3": None, "w2": None})
        run.route()
        run.dispatch()
        run.o = run.xg[run.lay.row_src[: cfg.P].long()].contiguous()
        run.combine()
        x = O.bf16_to_f64(H.bf16_host(run.t["x"]))
        y = O.bf16_to_f64(H.bf16_host(run.y)[: cfg.T])
        if k == 1:
            assert np.array_equal(y, x)                  # pure un-permute, bit-exact
        else:
            assert np.all(np.abs(y - x) <= 2.0 ** -7 * np.abs(x) + 1e-30)
        # linearity in a power of two is exact
        y1 = run.y.clone()
        run.o = (run.o.float() * 4.0).to(torch.bfloat16)
        run.combine()
        assert torch.equal(run.y.float(), y1.float() * 4.0)


def test_degenerate_and_error_paths():
    cfg = synth.MoEConfig("empty", T=0, d=64, f=64, E=4, k=2, G=2)
    run = H.Run(cfg, inputs={"x": torch.zeros(1, 64, dtype=torch.bfloat16, device="cuda"),
                             "w_gate": torch.zeros(64, 4, device="cuda"), "bias": None,
                             "w1": torch.zeros(4, 64, 64, dtype=torch.bfloat16, device="cuda"),
                             "w3": torch.zeros(4, 64, 64, dtype=torch.bfloat16, device="cuda"),
                             "w2": torch.zeros(4, 64, 64, dtype=torch.bfloat16, device="cuda")})
    run.route(); run.dispatch(); run.ffn(); run.combine(); run.layer()
    torch.cuda.synchronize()
    assert run.status()[0] == 0
    assert run.lay.expert_offsets[:5].tolist() == [0] * 5
    # flag combinations without meaning are refused before anything is launched
    both = B.MOE_FLAG_WEIGHT_IN_COMBINE | B.MOE_FLAG_COMBINE_IN_EPILOGUE
    with pytest.raises(B.MoEError):
        B.alloc_workspace(B.make_shape(cfg.with_(T=8), both))
    run_e = H.Run(cfg.with_(T=8), B.MOE_FLAG_COMBINE_IN_EPILOGUE, inputs=run.t)
    with pytest.raises(B.MoEError):
        run_e.ffn()
    with pytest.raises(B.MoEError):
        run_e.combine()
    # an out-of-range expert index is reported, not dereferenced
    cfg = synth.MoEConfig("badidx", T=40, d=64, f=64, E=4, k=2, G=2)
    run = H.Run(cfg, inputs=synth.make_routing_inputs(cfg, "cuda") | {"w1": None, "w3": None, "w2": None})
    run.route()
    run.idx[7] = 99
    run.dispatch()
    st = run.status()
    assert st[0] == B.MOE_DEV_INDEX_OUT_OF_RANGE and st[3] == 99
    B.moe_status_reset(run.ws)
    assert run.status()[0] == 0
    # ... by Combine too: the bad slot (token 3, slot 1) is skipped, the token's other row is still summed
    assert int(run.lay.pair_row[7]) == -1
    run.o.copy_(torch.randn(run.o.shape, device="cuda").to(torch.bfloat16))
    run.combine()
    st = run.status()
    assert st[0] == B.MOE_DEV_INDEX_OUT_OF_RANGE and st[1] == B.KERNEL_IDS["combine"] and st[3] == 99, st
    assert torch.equal(run.y[3], run.o[int(run.lay.pair_row[6])])
    B.moe_status_reset(run.ws)


def test_route_limits_E1024_k32():
    cfg = synth.MoEConfig("E1024", T=130, d=72, f=64, E=1024, k=32, G=8, bias="zipf", zipf_s=0.7, seed=12)
    run = H.Run(cfg, inputs=synth.make_routing_inputs(cfg, "cuda") | {"w1": None, "w3": None, "w2": None})
    run.route()
    idx_ref, _ = H.check_route(run)
    run.dispatch()
    H.check_layout(run, idx_ref)
    assert run.status()[0] == 0


def test_random_shape_sweep():
    """Seeded sweep over small random shapes: ragged T, K and N tails (any multiple of 8), every
    k / G / E combination the limits allow, both score functions, both weight placements."""
    rng = np.random.default_rng(2024)
    for i in range(14):
        E = int(rng.choice([1, 2, 3, 4, 6, 8, 12, 16, 24, 48]))
        G = int(rng.choice([g for g in range(1, E + 1) if E % g == 0]))
        k = int(rng.integers(1, min(E, 6) + 1))
        cfg = synth.MoEConfig(f"sweep{i}", T=int(rng.integers(1, 420)), d=8 * int(rng.integers(1, 40)),
                              f=8 * int(rng.integers(1, 40)), E=E, k=k, G=G, score_fn=int(rng.integers(0, 2)),
                              bias=str(rng.choice(["none", "zipf", "locality"])), zipf_s=1.0, boost=1.5, seed=100 + i)
        flags = B.MOE_FLAG_WEIGHT_IN_COMBINE if i % 3 == 0 else 0
        run, y_staged, y_def = staged(cfg, flags)
        y2 = torch.zeros_like(run.y)
        run.layer(y=y2)
        y_fused = O.bf16_to_f64(H.bf16_host(y2)[: cfg.T])
        H.assert_close_out(y_fused, y_def, f"{cfg} fused")
        assert np.array_equal(y_fused, y_staged), cfg


def test_layer_is_capturable_in_a_cuda_graph():
    """Every entry point only enqueues work on the caller's stream (no allocation, no sync), so a
    warmed-up moe_layer call can be captured once and replayed: same bytes as the eager call."""
    cfg = synth.CONFIGS["C1"]
    run = H.Run(cfg)
    run.layer()                       # first call: one-time host set-up (kernel attributes, occupancy query)
    torch.cuda.synchronize()
    y_eager = run.y.clone()
    y_graph = torch.zeros_like(run.y)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            run.layer(y=y_graph)
    for _ in range(2):
        y_graph.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(y_graph, y_eager)
    assert run.status()[0] == 0


@pytest.mark.parametrize("form", ["pair", "single"])
def test_both_gemm2_forms_on_the_same_layer(form):
    """GEMM-2 has a CTA-pair form (256-row tiles) and a single-CTA form (128-row tiles, taken when experts are
    small on average); the library picks by shape, MOE_FLAG_GEMM2_PAIR / MOE_FLAG_GEMM2_SINGLE force one.  Both
    must meet the parity bars on a layer with ragged and empty experts."""
    cfg = synth.MoEConfig("g2forms", T=1500, d=320, f=448, E=12, k=3, G=4, bias="zipf", zipf_s=1.3, seed=9)
    staged(cfg, B.MOE_FLAG_GEMM2_PAIR if form == "pair" else B.MOE_FLAG_GEMM2_SINGLE)


def test_bounded_wait_gives_up_and_the_context_stays_usable():
    """Every wait in the kernels is bounded: a wait that can never be satisfied ends with a status, not a
    hang.  The self-test kernel waits on a barrier nothing signals; afterwards the same workspace, once
    reset, runs the layer as before."""
    cfg = synth.CONFIGS["C1"]
    run = H.Run(cfg)
    run.layer()
    torch.cuda.synchronize()
    y_before = run.y.clone()
    B.moe_selftest_wait_timeout(run.ws, 300_000)            # 300 us budget
    st = run.status()
    assert st[0] == B.MOE_DEV_TIMEOUT and st[1] == 9, st
    assert 300 <= st[2] < 20_000, st                         # waited microseconds: the budget, not much more
    assert st[4] == 1                                        # abort word: later kernels on this workspace skip their work
    with pytest.raises(B.MoEError):
        B.moe_selftest_wait_timeout(run.ws, 10)              # budget below 1 us is refused on the host
    B.moe_status_reset(run.ws)
    assert run.status()[0] == 0
    run.y.zero_()
    run.layer()
    torch.cuda.synchronize()
    assert torch.equal(run.y, y_before) and run.status()[0] == 0


def test_traffic_stats_match_the_oracle_and_the_papers_printed_figures():
    """DeepSeek-V3-shaped routing (256 experts, top-8) over 32 groups: the layout's distinct-destination
    count gives the paper's "340 %" useless AllGather traffic, "nearly 50 %" redundant share and "near 2x"
    ideal speed-up (Sec. I, II-B, II-C); the same numbers as the oracle's counter."""
    import json, os
    cfg = synth.MoEConfig("ds-route", T=8192, d=256, f=64, E=256, k=8, G=32, score_fn=1)
    run = H.Run(cfg, inputs=synth.make_routing_inputs(cfg, "cuda") | {"w1": None, "w3": None, "w2": None})
    run.route()
    run.dispatch()
    got = B.moe_traffic_stats(run.shape, run.lay)
    idx_ref, _ = O.route(run.host_logits(), run.host_bias(), cfg.k, cfg.score_fn)
    D = O.distinct_groups_per_token(idx_ref, cfg.E, cfg.G)
    ref = O.redundancy_figures(D, cfg.G, cfg.k)
    assert got["T"] == cfg.T and got["P"] == cfg.P and abs(got["D"] - D) < 1e-12
    for name in ("allgather_useless", "redundant_share", "ideal_speedup"):
        assert abs(got[name] - ref[name]) < 1e-12, name
    assert abs(got["dedup"] - (1 - D / cfg.k)) < 1e-12
    gold = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_traffic_figures.json")))
    assert abs(got["allgather_useless"] - gold["allgather_useless_k8"]) <= gold["allgather_useless_tol"]
    assert gold["redundant_share_min_k8"] <= got["redundant_share"] <= gold["redundant_share_max"]
    assert gold["ideal_speedup_min_k8"] <= got["ideal_speedup"] <= gold["ideal_speedup_max"]


class Guarded:
    """A tensor carved out of a larger canary-filled allocation: writes before its start or past its end
    show up as damaged canaries (the check does not rely on an external memory checker)."""
    PAD = 4096

    def __init__(self, numel, dtype, fill=None):
        esz = torch.empty(0, dtype=dtype).element_size()
        nbytes = (numel * esz + 127) // 128 * 128
        self.raw = torch.full((self.PAD + nbytes + self.PAD,), 0xA5, dtype=torch.uint8, device="cuda")
        self.t = self.raw[self.PAD: self.PAD + numel * esz].view(dtype)
        self.lo, self.hi = self.PAD, self.PAD + numel * esz
        if fill is not None:
            self.t.fill_(fill)

    def intact(self):
        return bool((self.raw[: self.lo] == 0xA5).all()) and bool((self.raw[self.hi:] == 0xA5).all())


@pytest.mark.parametrize("cfg", [
    synth.MoEConfig("guard-a", T=257, d=136, f=200, E=6, k=3, G=3, seed=5),
    synth.MoEConfig("guard-b", T=1000, d=272, f=80, E=20, k=5, G=5, bias="zipf", zipf_s=1.5, seed=6),
    synth.MoEConfig("guard-c", T=130, d=512, f=1024, E=4, k=4, G=2, score_fn=1, seed=7),
], ids=lambda c: c.name)
def test_no_entry_point_writes_outside_its_buffers(cfg):
    """Every output buffer of every entry point sits between canaries (exact sizes, no slack): ragged shapes,
    partial tiles and K / N tails must not write a byte outside."""
    t = synth.make_inputs(cfg, "cuda")
    shape = B.make_shape(cfg)
    T, E, k, d, P, G = cfg.T, cfg.E, cfg.k, cfg.d, cfg.P, cfg.G
    g = {
        "ws": Guarded(B.moe_workspace_bytes(shape), torch.uint8, 0),
        "logits": Guarded(T * E, torch.float32), "idx": Guarded(P, torch.int32), "w": Guarded(P, torch.float32),
        "xg": Guarded(T * min(k, G) * d, torch.bfloat16), "o": Guarded(P * d, torch.bfloat16),
        "y": Guarded(T * d, torch.bfloat16), "pg": Guarded(T * min(k, G) * d, torch.bfloat16),
        "expert_counts": Guarded(E, torch.int32), "expert_offsets": Guarded(E + 1, torch.int32),
        "group_counts": Guarded(G, torch.int32), "group_offsets": Guarded(G + 1, torch.int32),
        "pair_row": Guarded(P, torch.int32), "row_pair": Guarded(P, torch.int32), "al": Guarded(G * T, torch.int32),
        "disp_token": Guarded(T * min(k, G), torch.int32), "row_src": Guarded(P, torch.int32),
    }
    lay = B.Layout(**{n: g[n].t for n in ("expert_counts", "expert_offsets", "group_counts", "group_offsets",
                                          "pair_row", "row_pair", "al", "disp_token", "row_src")})
    ws = g["ws"].t
    xg = g["xg"].t.view(-1, d)
    o = g["o"].t.view(-1, d)
    y = g["y"].t.view(-1, d)
    B.moe_route(shape, t["x"], t["w_gate"], t["bias"], g["logits"].t, g["idx"].t, g["w"].t, ws)
    B.moe_dispatch(shape, t["x"], g["idx"].t, lay, xg, ws)
    B.moe_expert_ffn(shape, xg, lay, g["w"].t, t["w1"], t["w3"], t["w2"], o, ws)
    B.moe_combine(shape, o, lay, g["idx"].t, g["w"].t, g["pg"].t.view(-1, d), y, ws)
    B.moe_layer(shape, t["x"], t["w_gate"], t["bias"], t["w1"], t["w3"], t["w2"], y, ws, logits=g["logits"].t,
                topk_idx=g["idx"].t, topk_w=g["w"].t, layout=lay)
    B.moe_layer(B.make_shape(cfg, B.MOE_FLAG_COMBINE_IN_EPILOGUE), t["x"], t["w_gate"], t["bias"], t["w1"], t["w3"],
                t["w2"], y, ws)
    # the option forms use more of the workspace: each with a workspace of exactly its own size
    F, PART, DISP = B.MOE_FLAG_FUSED_FFN, B.MOE_FLAG_SM_PARTITION, B.MOE_FLAG_TRACK_DISPATCH
    for i, flags in enumerate((F, F | PART | DISP, B.MOE_FLAG_GEMM1_PAIR)):
        sh = B.make_shape(cfg, flags)
        g[f"ws_opt{i}"] = Guarded(B.moe_workspace_bytes(sh), torch.uint8, 0)
        B.moe_layer(sh, t["x"], t["w_gate"], t["bias"], t["w1"], t["w3"], t["w2"], y, g[f"ws_opt{i}"].t)
        B.moe_expert_ffn(sh, xg, lay, g["w"].t, t["w1"], t["w3"], t["w2"], o, g[f"ws_opt{i}"].t)
    # backward: gradients and its workspace, sized exactly
    g["bws"] = Guarded(B.moe_backward_workspace_bytes(shape), torch.uint8, 0)
    g["dx"] = Guarded(T * d, torch.bfloat16)
    for n in ("w1", "w3", "w2"):
        g["d" + n] = Guarded(t[n].numel(), torch.bfloat16)
    B.moe_layer_backward(shape, t["x"], y, g["idx"].t, g["w"].t, lay, t["w1"], t["w3"], t["w2"], g["dx"].t.view(-1, d),
                         g["dw1"].t.view_as(t["w1"]), g["dw3"].t.view_as(t["w3"]), g["dw2"].t.view_as(t["w2"]), g["bws"].t)
    g["dw_gate"] = Guarded(d * E, torch.float32)
    B.moe_gate_backward(shape, g["logits"].t, t["bias"], g["idx"].t, g["w"].t, lay, t["w_gate"], g["dx"].t.view(-1, d),
                        g["dw_gate"].t.view(d, E), g["bws"].t)
    if cfg.d % 16 == 0 and cfg.f % 16 == 0:
        wq = {n: Guarded(t[n].numel(), torch.uint8) for n in ("w1", "w3", "w2")}
        sc = {n: Guarded(E * t[n].shape[2], torch.float32) for n in ("w1", "w3", "w2")}
        for n in wq:
            B.moe_quantize_weights(t[n], wq[n].t.view(E, t[n].shape[2], t[n].shape[1]), sc[n].t.view(E, -1))
        B.moe_layer_fp8(shape, t["x"], t["w_gate"], t["bias"], wq["w1"].t, sc["w1"].t, wq["w3"].t, sc["w3"].t,
                        wq["w2"].t, sc["w2"].t, y, ws)
        g.update({f"wq_{n}": wq[n] for n in wq})
        g.update({f"sc_{n}": sc[n] for n in sc})
    torch.cuda.synchronize()
    assert B.moe_status(ws)[0] == 0 and B.moe_status(g["bws"].t)[0] == 0
    bad = [n for n, buf in g.items() if not buf.intact()]
    assert not bad, f"canaries damaged around: {bad}"


def test_sparse_topk_tables():
    """MOE_FLAG_SPARSE_TOPK: slots of topk_idx may be -1 (the routing table of rows received behind one switch
    port, trimmed to that port's experts).  Layout arrays against a brute-force enumeration written here,
    outputs against the dense definition restricted to the slots in use."""
    cfg = synth.MoEConfig("sparse", T=300, d=128, f=192, E=12, k=4, G=3, seed=21)
    flags = B.MOE_FLAG_SPARSE_TOPK
    run = H.Run(cfg, flags)
    run.route()
    rng = np.random.default_rng(3)
    idx = run.host_idx().copy()
    drop = rng.random(idx.shape) < 0.4
    drop[5] = True                                   # a token with no slot in use at all
    drop[6] = False
    idx[drop] = -1
    run.idx[: cfg.P] = torch.from_numpy(idx.reshape(-1)).cuda()
    run.dispatch()
    T, k, E, G, m = cfg.T, cfg.k, cfg.E, cfg.G, cfg.E // cfg.G
    # brute force: expert-sorted rows by (expert, token); one dispatched row per distinct (token, group)
    pairs = sorted((int(idx[t, j]), t, j) for t in range(T) for j in range(k) if idx[t, j] >= 0)
    counts = np.zeros(E, np.int64)
    for e, _, _ in pairs:
        counts[e] += 1
    eoff = np.concatenate([[0], np.cumsum(counts)])
    pair_row = -np.ones(T * k, np.int64)
    row_pair = np.array([t * k + j for _, t, j in pairs], np.int64)
    pair_row[row_pair] = np.arange(len(pairs))
    touch = sorted({(int(idx[t, j]) // m, t) for t in range(T) for j in range(k) if idx[t, j] >= 0})
    gcount = np.bincount([g for g, _ in touch], minlength=G)
    goff = np.concatenate([[0], np.cumsum(gcount)])
    al = -np.ones((G, T), np.int64)
    seen = np.zeros(G, np.int64)
    for g, t in touch:
        al[g, t] = seen[g]
        seen[g] += 1
    L = run.lay
    npairs = len(pairs)
    assert np.array_equal(L.expert_counts.cpu().numpy()[:E], counts)
    assert np.array_equal(L.expert_offsets.cpu().numpy()[: E + 1], eoff) and eoff[-1] == npairs < cfg.P
    assert np.array_equal(L.pair_row.cpu().numpy()[: T * k], pair_row)
    assert np.array_equal(L.row_pair.cpu().numpy()[:npairs], row_pair)
    assert np.array_equal(L.group_offsets.cpu().numpy()[: G + 1], goff)
    assert np.array_equal(L.al.cpu().numpy()[: G * T].reshape(G, T), al)
    row_src = np.array([goff[e // m] + al[e // m, t] for e, t, _ in pairs], np.int64)
    assert np.array_equal(L.row_src.cpu().numpy()[:npairs], row_src)
    assert run.status()[0] == 0
    # expert FFN + combine on the sparse table
    run.ffn()
    pg = torch.zeros(max(int(goff[-1]), 1), cfg.d, dtype=torch.bfloat16, device="cuda")
    run.combine(pg)
    torch.cuda.synchronize()
    assert run.status()[0] == 0
    xb = O.bf16_to_f64(H.bf16_host(run.t["x"]))
    w = run.host_w()
    wb = {n: H.bf16_host(run.t[n]) for n in ("w1", "w3", "w2")}
    y_ref = np.zeros((T, cfg.d))
    for t in range(T):
        for j in range(k):
            if idx[t, j] >= 0:
                e = int(idx[t, j])
                y_ref[t] += w[t, j] * O.expert_ffn_rows(xb[t:t + 1], wb["w1"][e], wb["w3"][e], wb["w2"][e])[0]
    y_gpu = O.bf16_to_f64(H.bf16_host(run.y)[:T])
    H.assert_close_out(y_gpu, y_ref, "sparse y")
    assert not y_gpu[5].any()                        # no slot in use: the row of y is zero
    # the flag is refused where the library picks the experts itself
    with pytest.raises(B.MoEError):
        run.layer()


@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: c.name)
def test_single_kernel_ffn_with_tile_tracker(cfg):
    """MOE_FLAG_FUSED_FFN: the stages after the layout as one persistent kernel paced by the token tracker (tile
    status counters DAcc / TBCnt1 / TBCnt2 and the per-token output-readiness counter): GEMM-1, GEMM-2, in the layer
    also the Combine tasks, with MOE_FLAG_TRACK_DISPATCH also the Dispatch tasks, interleaved or with the SM
    partition.  Expert outputs and y must equal the separate kernels bit for bit (same operands, same accumulation
    order per element), in the staged entry point and in the fused layer, twice in a row (the tracker is cleared by
    every call)."""
    if "wcombine" in cfg.name:
        pytest.skip("covered by the default-weight cases")
    run = H.Run(cfg)
    run.route()
    run.dispatch()
    run.ffn()
    o_two = run.o.clone()
    run.layer()
    y_two = run.y.clone()
    F, PART, DISP = B.MOE_FLAG_FUSED_FFN, B.MOE_FLAG_SM_PARTITION, B.MOE_FLAG_TRACK_DISPATCH
    for flags in (F, F | PART, F | DISP, F | PART | DISP):
        _check_single_kernel(cfg, run, flags, o_two, y_two)


def _check_single_kernel(cfg, run, flags, o_two, y_two):
    fused = H.Run(cfg, flags, inputs=run.t)
    fused.route()
    fused.dispatch()
    for _ in range(2):
        fused.o.fill_(7.0)
        fused.ffn()
        torch.cuda.synchronize()
        assert fused.status()[0] == 0, fused.status()
        assert torch.equal(fused.o[: cfg.P], o_two[: cfg.P])
        fused.y.fill_(7.0)
        fused.layer()
        torch.cuda.synchronize()
        assert fused.status()[0] == 0
        assert torch.equal(fused.y[: cfg.T], y_two[: cfg.T])


@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: c.name)
def test_pair_gemm1_on_the_per_expert_layout_tensors(cfg):
    """MOE_FLAG_GEMM1_PAIR: Dispatch writes one dense row per (token, expert) in expert-sorted order and GEMM-1
    reads them as TMA tiles on CTA pairs.  Same operands and the same accumulation order per element as the
    gathering form, so expert outputs and the layer output must equal it bit for bit; the staged path is also held
    to the oracle."""
    if "wcombine" in cfg.name:
        pytest.skip("covered by the default-weight cases")
    run = H.Run(cfg)
    run.route()
    run.dispatch()
    run.ffn()
    run.layer()
    torch.cuda.synchronize()
    o_ref, y_ref = run.o.clone(), run.y.clone()
    _check_single_kernel(cfg, run, B.MOE_FLAG_GEMM1_PAIR, o_ref, y_ref)
    staged(cfg, B.MOE_FLAG_GEMM1_PAIR)


def test_tensor_map_cache_is_transparent():
    """The TMA descriptors are cached by (address, extents, strides, box).  Same inputs through a warm cache, a cleared
    cache, and a cache that has been flooded by another shape in between must give bit-identical outputs; and a new
    tensor that lands at a recycled address with another shape must get its own descriptor."""
    cfg = synth.CONFIGS["C1"]
    run = H.Run(cfg)
    run.layer()
    torch.cuda.synchronize()
    y0 = H.bf16_host(run.y).copy()
    run.layer()                       # warm cache
    torch.cuda.synchronize()
    assert np.array_equal(H.bf16_host(run.y), y0)
    B.moe_clear_cache()
    run.layer()                       # everything encoded again
    torch.cuda.synchronize()
    assert np.array_equal(H.bf16_host(run.y), y0)
    # more distinct maps than the cache holds, some of them at addresses the allocator hands out again
    for i in range(12):
        other = H.Run(cfg.with_(name=f"c1_{i}", T=128 + 64 * i, d=256 + 64 * (i % 3), f=512))
        other.layer()
        torch.cuda.synchronize()
        assert other.status()[0] == 0
        del other
    run.layer()
    torch.cuda.synchronize()
    assert np.array_equal(H.bf16_host(run.y), y0)
    assert run.status()[0] == 0
    # the same check against the oracle on a shape that reuses freed memory
    torch.cuda.empty_cache()
    cfg2 = cfg.with_(name="c1_small", T=192, d=384, f=768)
    r2 = H.Run(cfg2)
    r2.layer(logits=r2.logits)
    torch.cuda.synchronize()
    _, _, _, y_def = O.layer(H.bf16_host(r2.t["x"]), r2.host_logits(), r2.host_bias(), H.bf16_host(r2.t["w1"]),
                             H.bf16_host(r2.t["w3"]), H.bf16_host(r2.t["w2"]), cfg2.k, cfg2.score_fn)
    H.assert_close_out(O.bf16_to_f64(H.bf16_host(r2.y)[: cfg2.T]), y_def, "layer after cache churn")
    assert r2.status()[0] == 0
