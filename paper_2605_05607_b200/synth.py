"""Seeded synthetic workloads for the MoE-layer hot path.

This module only *draws inputs* (activations, gate weights, router biases,
expert weights) and names the workload shapes.  It holds none of the method's
arithmetic (no gating, no routing, no FFN), so both the CUDA path and the CPU
oracle may be fed from it without sharing any computation.

Shapes follow the paper's evaluation workloads (Sec. V, Table I and the
"diverse models" table: DeepSeek-V3-derived layers, GPT-OSS, Qwen3-MoE) as
restated by the five benchmark configurations; real weights or traces are not
used, every tensor is random with a fixed seed:

* ``x``       bf16 [T, d], N(0, 1)
* ``w_gate``  fp32 [d, E], N(0, std 0.02)
* ``w1, w3``  bf16 [E, d, f], N(0, variance 1/d)   (fan-in = d)
* ``w2``      bf16 [E, f, d], N(0, variance 1/f)   (fan-in = f)
* ``bias``    fp32, none | [E] (Zipf popularity: ``-s * ln(rank)`` over a seeded
  permutation of the experts) | [T, E] (locality: one seeded favourite group per
  token gets ``+boost`` on all of its experts)

Every tensor has its own generator stream ``seed * 1000 + tensor_id`` so that
changing one shape never reshuffles another tensor.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np
import torch

SCORE_SOFTMAX = 0  # softmax over the k selected keys
SCORE_SIGMOID = 1  # sigmoid(key), renormalised over the k selected


@dataclass(frozen=True)
class MoEConfig:
    name: str
    T: int
    d: int
    f: int
    E: int
    k: int
    G: int
    score_fn: int = SCORE_SOFTMAX
    bias: str = "none"        # "none" | "zipf" | "locality"
    zipf_s: float = 0.0
    boost: float = 0.0
    seed: int = 0

    @property
    def P(self) -> int:
        return self.T * self.k

    @property
    def m(self) -> int:
        return self.E // self.G

    def with_(self, **kw) -> "MoEConfig":
        return replace(self, **kw)


CONFIGS: Dict[str, MoEConfig] = {
    # tiny layer, the case the CPU oracle finishes in seconds
    "C1": MoEConfig("C1", T=256, d=512, f=1024, E=8, k=2, G=4),
    # Mixtral-shaped
    "C2": MoEConfig("C2", T=4096, d=4096, f=14336, E=8, k=2, G=8),
    # GPT-OSS-shaped, Zipf(1.1) expert popularity
    "C3": MoEConfig("C3", T=8192, d=2880, f=2880, E=128, k=4, G=8, bias="zipf", zipf_s=1.1),
    # Qwen3-MoE-shaped, per-token locality (+2.0 on one random group)
    "C4": MoEConfig("C4", T=16384, d=4096, f=1536, E=128, k=8, G=8, bias="locality", boost=2.0),
    # DeepSeek-V3-shaped, sigmoid scores; uniform (seed 0) and Zipf(1.2) (seed 1)
    "C5a": MoEConfig("C5a", T=32768, d=7168, f=2048, E=256, k=8, G=8, score_fn=SCORE_SIGMOID),
    "C5b": MoEConfig("C5b", T=32768, d=7168, f=2048, E=256, k=8, G=8, score_fn=SCORE_SIGMOID,
                     bias="zipf", zipf_s=1.2, seed=1),
}

# The paper's own evaluation shapes (Table "Model Configurations": Small / Medium / Large, the
# Large one being DeepSeek-V3's; top-k candidates 8 / 16 / 32), one GPU's share of a 32-GPU
# expert-parallel group: G = 32 logical groups, T = 4 sequences of the table's length, sigmoid
# scores as in the DeepSeek-V3 router.  The table gives no batch size: T is this build's choice.
_PAPER_SIZES = {"S": dict(T=4 * 2048, d=2048, f=512, E=64), "M": dict(T=4 * 4096, d=4096, f=1024, E=128),
                "L": dict(T=4 * 8192, d=7168, f=2048, E=256)}
PAPER_CONFIGS: Dict[str, MoEConfig] = {
    f"{size}{k}": MoEConfig(f"{size}{k}", k=k, G=32, score_fn=SCORE_SIGMOID, **dims)
    for size, dims in _PAPER_SIZES.items() for k in (8, 16, 32)
}
ALL_CONFIGS: Dict[str, MoEConfig] = {**CONFIGS, **PAPER_CONFIGS}

_TID = {"x": 1, "w_gate": 2, "w1": 3, "w3": 4, "w2": 5, "perm": 6, "fav": 7}


def _gen(cfg: MoEConfig, what: str, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed * 1000 + _TID[what])
    return g


def make_bias(cfg: MoEConfig, device="cpu") -> Optional[torch.Tensor]:
    """Router-logit bias of the workload: None, [E] or [T, E] fp32."""
    if cfg.bias == "none":
        return None
    if cfg.bias == "zipf":
        perm = torch.randperm(cfg.E, generator=_gen(cfg, "perm", "cpu"))
        rank = torch.empty(cfg.E, dtype=torch.float64)
        rank[perm] = torch.arange(1, cfg.E + 1, dtype=torch.float64)
        return (-cfg.zipf_s * torch.log(rank)).to(torch.float32).to(device)
    if cfg.bias == "locality":
        fav = torch.randint(0, cfg.G, (cfg.T,), generator=_gen(cfg, "fav", "cpu"))
        grp = torch.arange(cfg.E) // cfg.m
        b = (grp[None, :] == fav[:, None]).to(torch.float32) * cfg.boost
        return b.contiguous().to(device)
    raise ValueError(f"unknown bias kind {cfg.bias!r}")


def make_routing_inputs(cfg: MoEConfig, device="cpu") -> Dict[str, Optional[torch.Tensor]]:
    """x, w_gate and bias only (enough for routing / layout / dispatch)."""
    x = torch.randn(cfg.T, cfg.d, generator=_gen(cfg, "x", device), device=device,
                    dtype=torch.float32).to(torch.bfloat16)
    w_gate = torch.randn(cfg.d, cfg.E, generator=_gen(cfg, "w_gate", device), device=device,
                         dtype=torch.float32) * 0.02
    return {"x": x, "w_gate": w_gate.contiguous(), "bias": make_bias(cfg, device)}


def _expert_weights(cfg: MoEConfig, what: str, rows: int, cols: int, std: float, device) -> torch.Tensor:
    g = _gen(cfg, what, device)
    out = torch.empty(cfg.E, rows, cols, dtype=torch.bfloat16, device=device)
    for e in range(cfg.E):  # expert by expert: caps the fp32 staging buffer
        out[e] = (torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
    return out


def make_inputs(cfg: MoEConfig, device="cpu") -> Dict[str, Optional[torch.Tensor]]:
    """All tensors of one layer invocation."""
    t = make_routing_inputs(cfg, device)
    t["w1"] = _expert_weights(cfg, "w1", cfg.d, cfg.f, 1.0 / math.sqrt(cfg.d), device)
    t["w3"] = _expert_weights(cfg, "w3", cfg.d, cfg.f, 1.0 / math.sqrt(cfg.d), device)
    t["w2"] = _expert_weights(cfg, "w2", cfg.f, cfg.d, 1.0 / math.sqrt(cfg.f), device)
    return t


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """Raw bf16 bit patterns of a tensor as a host uint16 array (no arithmetic)."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def bits_to_bf16(a: np.ndarray, device="cpu") -> torch.Tensor:
    """Inverse of :func:`bf16_bits`."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)


def tensor_checksum(t: Optional[torch.Tensor]) -> Optional[int]:
    """Sum of the tensor's raw 16-bit words mod 2^61 - 1 (position-independent, cheap on any
    device, chunked so that a 22 GB weight tensor needs no large temporary): identifies the seeded
    inputs of a run in reports."""
    if t is None:
        return None
    words = t.contiguous().view(-1).view(torch.int16)
    total = 0
    step = 1 << 28
    for i in range(0, words.numel(), step):
        total += int((words[i:i + step].to(torch.int32) & 0xFFFF).sum(dtype=torch.int64).item())
    return total % ((1 << 61) - 1)


def sample_tokens(cfg: MoEConfig, n: int, seed: int = 12345) -> np.ndarray:
    """Deterministic token sample for full-size output checks: the first and last
    64 tokens plus a seeded choice of the rest, ascending, without repeats."""
    if n >= cfg.T:
        return np.arange(cfg.T, dtype=np.int64)
    edge = min(64, n // 4)
    rng = np.random.default_rng(seed)
    mid = rng.choice(np.arange(edge, cfg.T - edge), size=n - 2 * edge, replace=False)
    return np.unique(np.concatenate([np.arange(edge), mid, np.arange(cfg.T - edge, cfg.T)])).astype(np.int64)
