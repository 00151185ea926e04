"""Host-side logic of the multi-GPU mode: independent replicas, tokens sharded, weights replicated.

The layer's output for a token depends only on that token and the (replicated) weights, so N GPUs
run N independent copies of the path on disjoint token batches with no data-path collective.
The only cross-rank traffic is the timing barrier and a max-reduction of the measured time."""
from __future__ import annotations

from .synth import MoEConfig, make_inputs, make_routing_inputs

TOKEN_SEED_STRIDE = 7919


def rank_token_config(cfg: MoEConfig, rank: int) -> MoEConfig:
    """Configuration whose `x` stream belongs to `rank` (rank 0 keeps the base seed)."""
    return cfg if rank == 0 else cfg.with_(seed=cfg.seed + TOKEN_SEED_STRIDE * rank)


def make_rank_inputs(cfg: MoEConfig, rank: int, device="cuda"):
    """Weights, gate and bias from the base seed (identical on every rank); tokens of this rank."""
    t = make_inputs(cfg, device)
    if rank > 0:
        t["x"] = make_routing_inputs(rank_token_config(cfg, rank), device)["x"]
    return t


def max_over_ranks(value: float, dist, device) -> float:
    """Slowest rank's time (ms); `dist` is torch.distributed or None for a single process."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(cfg: MoEConfig, world: int, steps: int, elapsed_ms: float) -> float:
    """Aggregate throughput: every rank processed cfg.T tokens per step."""
    return cfg.T * world * steps / (elapsed_ms * 1e-3)
