"""Shared pieces of the GPU parity tests: run a stage through the C ABI and
compare with the CPU oracle on the same seeded inputs."""
import numpy as np
import torch

from oracle import moe_oracle as O
from paper_2605_05607_b200 import binding as B
from paper_2605_05607_b200 import synth

# output tolerance (bf16 operands, fp32 accumulation): max|gpu - ref| <= 2e-2 max|ref| and
# sum|gpu - ref| / sum|ref| <= 5e-3; fp32 logits: max|gpu - ref| <= 1e-4 max|ref|
MAX_REL = 2e-2
MEAN_REL = 5e-3
LOGIT_REL = 1e-4
WEIGHT_ABS = 1e-6


def out_errors(got: np.ndarray, ref: np.ndarray):
    diff = np.abs(got.astype(np.float64) - ref)
    return diff.max() / max(np.abs(ref).max(), 1e-300), diff.sum() / max(np.abs(ref).sum(), 1e-300)


def assert_close_out(got, ref, what=""):
    mx, mean = out_errors(got, ref)
    assert mx <= MAX_REL and mean <= MEAN_REL, f"{what}: max rel {mx:.3e} (bar {MAX_REL}), mean rel {mean:.3e} (bar {MEAN_REL})"
    return mx, mean


def bf16_host(t: torch.Tensor) -> np.ndarray:
    return synth.bf16_bits(t)


class Run:
    """Holds device buffers of one configuration and the staged GPU results."""

    def __init__(self, cfg, flags=0, inputs=None):
        self.cfg = cfg
        self.shape = B.make_shape(cfg, flags)
        self.t = inputs if inputs is not None else synth.make_inputs(cfg, "cuda")
        self.ws = B.alloc_workspace(self.shape)
        dev = "cuda"
        T, E, k, d = cfg.T, cfg.E, cfg.k, cfg.d
        self.logits = torch.zeros(max(T * E, 1), dtype=torch.float32, device=dev)
        self.idx = torch.zeros(max(T * k, 4), dtype=torch.int32, device=dev)
        self.w = torch.zeros(max(T * k, 4), dtype=torch.float32, device=dev)
        self.lay = B.alloc_layout(self.shape)
        self.xg = torch.zeros(max(T * min(k, cfg.G), 1), d, dtype=torch.bfloat16, device=dev)
        self.o = torch.zeros(max(T * k, 1), d, dtype=torch.bfloat16, device=dev)
        self.y = torch.zeros(max(T, 1), d, dtype=torch.bfloat16, device=dev)

    def status(self):
        return B.moe_status(self.ws)

    def route(self):
        t = self.t
        B.moe_route(self.shape, t["x"], t["w_gate"], t["bias"], self.logits, self.idx, self.w, self.ws)

    def dispatch(self):
        B.moe_dispatch(self.shape, self.t["x"], self.idx, self.lay, self.xg, self.ws)

    def ffn(self):
        t = self.t
        B.moe_expert_ffn(self.shape, self.xg, self.lay, self.w, t["w1"], t["w3"], t["w2"], self.o, self.ws)

    def combine(self, pg=None):
        B.moe_combine(self.shape, self.o, self.lay, self.idx, self.w, pg, self.y, self.ws)

    def layer(self, y=None, **kw):
        t = self.t
        B.moe_layer(self.shape, t["x"], t["w_gate"], t["bias"], t["w1"], t["w3"], t["w2"],
                    self.y if y is None else y, self.ws, **kw)

    # host views
    def host_logits(self):
        return self.logits[: self.cfg.T * self.cfg.E].cpu().numpy().reshape(self.cfg.T, self.cfg.E)

    def host_idx(self):
        return self.idx[: self.cfg.P].cpu().numpy().reshape(self.cfg.T, self.cfg.k)

    def host_w(self):
        return self.w[: self.cfg.P].cpu().numpy().reshape(self.cfg.T, self.cfg.k)

    def host_bias(self):
        b = self.t["bias"]
        return None if b is None else b.cpu().numpy()


def check_route(run: Run):
    """logits within 1e-4 relative of the fp64 oracle; routing recomputed by the oracle from the
    GPU's own fp32 logits must match bit-exactly; weights within 1e-6."""
    cfg = run.cfg
    logits = run.host_logits()
    ref = O.gate_logits(bf16_host(run.t["x"]), run.t["w_gate"].cpu().numpy())
    err = np.abs(logits.astype(np.float64) - ref).max() / np.abs(ref).max()
    assert err <= LOGIT_REL, f"logits rel err {err:.3e}"
    idx_ref, w_ref = O.route(logits, run.host_bias(), cfg.k, cfg.score_fn)
    idx = run.host_idx()
    assert idx.dtype == np.int32 and np.array_equal(idx, idx_ref), "topk_idx differs from the oracle"
    w = run.host_w()
    assert np.abs(w.astype(np.float64) - w_ref).max() <= WEIGHT_ABS
    assert np.abs(w.astype(np.float64).sum(axis=1) - 1.0).max() <= 4 * 2.0 ** -24 * cfg.k
    return idx_ref, w_ref


def check_layout(run: Run, idx_ref):
    cfg = run.cfg
    lay = O.layout(idx_ref, cfg.E, cfg.G)
    L = run.lay
    n = lay["n_disp"]
    for name in ("expert_counts", "expert_offsets", "group_counts", "group_offsets", "pair_row", "row_pair", "row_src"):
        got = getattr(L, name).cpu().numpy()[: lay[name].size]
        assert np.array_equal(got, lay[name]), name
    assert np.array_equal(L.al.cpu().numpy()[: cfg.G * cfg.T].reshape(cfg.G, cfg.T), lay["al"]), "al"
    assert np.array_equal(L.disp_token.cpu().numpy()[:n], lay["disp_token"]), "disp_token"
    return lay
