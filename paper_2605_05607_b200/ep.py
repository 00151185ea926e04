"""Expert-parallel execution of the layer: expert group g lives on rank g (Sec. II-A of the paper:
Dispatch sends a token to the GPUs hosting its experts, Combine brings the outputs back; Sec. III-D:
one replica per destination, trimmed to its targets, outputs of one destination reduced before they
return).

Every step of the data path runs in the library's kernels; this module only sequences them and moves
the buffers between ranks (`torch.distributed.all_to_all_single`, NCCL on GPUs).  Per rank:

  send     moe_route -> moe_dispatch (G = world: the dispatched buffer xg is grouped by destination)
           -> moe_ep_pack (per dispatched row: its experts inside the destination group + gate weights)
  exchange segment g of (xg, send_idx, send_w) goes to rank g            [one row per (token, group)]
  receive  the received rows are a layer of their own: shape {T = rows, E = m, k = min(k, m), G = 1,
           sparse top-k}; moe_dispatch (layout only) -> moe_expert_ffn (local experts) -> moe_combine
           (sum per received row = the pre-reduced row of that (token, group))
  exchange the pre-reduced rows return to their senders, in the order they came
  finish   moe_ep_finish: y[t] = sum over the groups token t touched

`emulate` runs the same three phases for all ranks inside one process (the exchange becomes slicing and
concatenation); it is how the path is tested on one GPU.  Segment sizes are read back to the host once
per layer (group_counts), as any all-to-all with data-dependent splits needs.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import torch

from . import binding as B
from .synth import MoEConfig


@dataclass
class Outbox:
    """What one rank sends: rows grouped by destination and the per-destination row counts (host)."""
    rows: torch.Tensor      # [N_disp, d] bf16
    idx: torch.Tensor       # [N_disp, kk] int32, experts local to the destination group, -1 unused
    w: torch.Tensor         # [N_disp, kk] fp32
    counts: List[int]       # rows for rank 0 .. world-1


class EpRank:
    """One rank of an expert-parallel layer.  `cfg` describes the rank's share: cfg.T local tokens, all E
    experts of the layer, G = world groups; w1 / w3 / w2 hold only the m = E / G experts of this rank."""

    def __init__(self, cfg: MoEConfig, rank: int, w_gate: torch.Tensor, bias: Optional[torch.Tensor],
                 w1: torch.Tensor, w3: torch.Tensor, w2: torch.Tensor):
        assert 0 <= rank < cfg.G and w1.shape[0] == cfg.m
        self.cfg, self.rank = cfg, rank
        self.w_gate, self.bias, self.w1, self.w3, self.w2 = w_gate, bias, w1, w3, w2
        self.kk = min(cfg.k, cfg.m)
        dev = w1.device
        self.shape = B.make_shape(cfg)
        self.ws = B.alloc_workspace(self.shape, dev)
        self.lay = B.alloc_layout(self.shape)
        T, k, E, d = cfg.T, cfg.k, cfg.E, cfg.d
        cap = max(T * min(k, cfg.G), 1)
        self.logits = torch.empty(max(T * E, 1), dtype=torch.float32, device=dev)
        self.idx = torch.empty(max(T * k, 4), dtype=torch.int32, device=dev)
        self.w = torch.empty(max(T * k, 4), dtype=torch.float32, device=dev)
        self.xg = torch.empty(cap, d, dtype=torch.bfloat16, device=dev)
        self.send_idx = torch.empty(cap, self.kk, dtype=torch.int32, device=dev)
        self.send_w = torch.empty(cap, self.kk, dtype=torch.float32, device=dev)
        self.y = torch.empty(max(T, 1), d, dtype=torch.bfloat16, device=dev)
        self._recv: Dict[int, dict] = {}     # receive-side buffers by capacity bucket

    # ---- phase 1 ---------------------------------------------------------------------------
    def send_phase(self, x: torch.Tensor) -> Outbox:
        B.moe_route(self.shape, x, self.w_gate, self.bias, self.logits, self.idx, self.w, self.ws)
        B.moe_dispatch(self.shape, x, self.idx, self.lay, self.xg, self.ws)
        B.moe_ep_pack(self.shape, self.idx, self.w, self.lay, self.send_idx, self.send_w)
        counts = self.lay.group_counts[: self.cfg.G].tolist()          # device -> host: the split sizes
        n = sum(counts)
        return Outbox(self.xg[:n], self.send_idx[:n], self.send_w[:n], counts)

    # ---- phase 2 ---------------------------------------------------------------------------
    def _recv_buffers(self, R: int) -> dict:
        cap = 1 << max(int(R - 1).bit_length(), 6)
        if cap not in self._recv:
            c = self.cfg
            shape = B.MoEShape(cap, c.d, c.f, c.m, self.kk, 1, c.score_fn, B.MOE_FLAG_SPARSE_TOPK)
            dev = self.w1.device
            self._recv[cap] = {"ws": B.alloc_workspace(shape, dev), "lay": B.alloc_layout(shape),
                               "o": torch.empty(cap * self.kk, c.d, dtype=torch.bfloat16, device=dev),
                               "partial": torch.empty(cap, c.d, dtype=torch.bfloat16, device=dev)}
        return self._recv[cap]

    def recv_phase(self, rows: torch.Tensor, idx: torch.Tensor, w: torch.Tensor) -> torch.Tensor:
        """rows / idx / w: everything this rank received, senders in rank order.  Returns the pre-reduced
        rows [R, d] in the same order."""
        R = rows.shape[0]
        c = self.cfg
        buf = self._recv_buffers(R)
        shape = B.MoEShape(R, c.d, c.f, c.m, self.kk, 1, c.score_fn, B.MOE_FLAG_SPARSE_TOPK)
        if R == 0:
            return buf["partial"][:0]
        idx, w = idx.contiguous().view(-1), w.contiguous().view(-1)
        B.moe_dispatch(shape, rows, idx, buf["lay"], None, buf["ws"])         # layout only: row_src is the identity
        B.moe_expert_ffn(shape, rows, buf["lay"], w, self.w1, self.w3, self.w2, buf["o"], buf["ws"])
        B.moe_combine(shape, buf["o"], buf["lay"], idx, w, None, buf["partial"], buf["ws"])
        return buf["partial"][:R]

    # ---- phase 3 ---------------------------------------------------------------------------
    def finish_phase(self, back: torch.Tensor) -> torch.Tensor:
        B.moe_ep_finish(self.shape, back, self.lay, self.y)
        return self.y[: self.cfg.T]

    def wire_stats(self) -> Dict[str, float]:
        """Link traffic of the last forward() / send_phase() of this rank (reads two small device arrays)."""
        gc = self.lay.group_counts[: self.cfg.G].tolist()
        ec = self.lay.expert_counts[: self.cfg.E].tolist()
        return wire_stats(self.cfg, self.rank, gc, ec)

    def status(self) -> List[int]:
        return [B.moe_status(self.ws)[0]] + [B.moe_status(b["ws"])[0] for b in self._recv.values()]

    # ---- one rank per process ----------------------------------------------------------------
    def forward(self, x: torch.Tensor, group=None) -> torch.Tensor:
        import torch.distributed as dist
        out = self.send_phase(x)
        recv_counts = exchange_counts(out.counts, group)
        rows = all_to_all_rows(out.rows, out.counts, recv_counts, group)
        idx = all_to_all_rows(out.idx, out.counts, recv_counts, group)
        w = all_to_all_rows(out.w, out.counts, recv_counts, group)
        partial = self.recv_phase(rows, idx, w)
        back = all_to_all_rows(partial, recv_counts, out.counts, group)
        return self.finish_phase(back)


def wire_stats(cfg: MoEConfig, rank: int, group_counts: Sequence[int], expert_counts: Sequence[int]) -> Dict[str, float]:
    """What one rank puts on the links for one layer, from the device counters of its dispatch layout (group g lives
    on rank g; rows for the rank's own group never leave it).

    * with the per-group de-duplication / pre-reduction (Sec. III-D: one copy per destination out, one reduced row per
      destination back): `group_counts[g]` rows of d bf16 each way, plus the trimmed target list (kk local expert ids
      and gate weights per row) on the way out;
    * point to point (one copy per (token, expert) pair each way, what Sec. II-B calls redundant): the pairs whose
      expert lives in group g, i.e. the sum of `expert_counts` over that group, plus one id and weight per row.

    Returns rows and bytes for both and the share of bytes the de-duplication removes."""
    m, d = cfg.m, cfg.d
    kk = min(cfg.k, m)
    rows_dedup = sum(int(c) for g, c in enumerate(group_counts) if g != rank)
    rows_p2p = sum(int(sum(expert_counts[g * m:(g + 1) * m])) for g in range(cfg.G) if g != rank)
    row_bytes = 2 * d
    out_dedup = rows_dedup * (row_bytes + 8 * kk)
    out_p2p = rows_p2p * (row_bytes + 8)
    back_dedup, back_p2p = rows_dedup * row_bytes, rows_p2p * row_bytes
    total_dedup, total_p2p = out_dedup + back_dedup, out_p2p + back_p2p
    return {"rows_dedup": rows_dedup, "rows_point_to_point": rows_p2p,
            "bytes_out_dedup": out_dedup, "bytes_back_dedup": back_dedup,
            "bytes_out_point_to_point": out_p2p, "bytes_back_point_to_point": back_p2p,
            "bytes_removed_share": 0.0 if total_p2p == 0 else 1.0 - total_dedup / total_p2p}


def exchange_counts(send_counts: Sequence[int], group=None) -> List[int]:
    """recv_counts[s] = number of rows rank s sends to this rank."""
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    send = torch.tensor(list(send_counts), dtype=torch.int64, device=dev)
    recv = torch.empty_like(send)
    dist.all_to_all_single(recv, send, group=group)
    return recv.tolist()


def all_to_all_rows(t: torch.Tensor, send_counts: Sequence[int], recv_counts: Sequence[int], group=None) -> torch.Tensor:
    """Rows [sum(send_counts), ...] split by destination -> rows [sum(recv_counts), ...] in sender order."""
    import torch.distributed as dist
    out = torch.empty((sum(recv_counts),) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
    dist.all_to_all_single(out, t.contiguous(), output_split_sizes=list(recv_counts),
                           input_split_sizes=list(send_counts), group=group)
    return out


def emulate(ranks: Sequence[EpRank], xs: Sequence[torch.Tensor]) -> List[torch.Tensor]:
    """All ranks of an expert-parallel layer in one process, one after the other (no kernel ever waits for
    another): the exchange is slicing and concatenation.  Used to test the path on a single GPU."""
    world = len(ranks)
    outs = [r.send_phase(x) for r, x in zip(ranks, xs)]

    def segments(o: Outbox, t: torch.Tensor) -> List[torch.Tensor]:
        ends = [0]
        for c in o.counts:
            ends.append(ends[-1] + c)
        return [t[ends[g]: ends[g + 1]] for g in range(world)]

    seg = [{"rows": segments(o, o.rows), "idx": segments(o, o.idx), "w": segments(o, o.w)} for o in outs]
    partials = []
    for g, r in enumerate(ranks):
        rows = torch.cat([seg[s]["rows"][g] for s in range(world)])
        idx = torch.cat([seg[s]["idx"][g] for s in range(world)])
        w = torch.cat([seg[s]["w"][g] for s in range(world)])
        partials.append(r.recv_phase(rows, idx, w).clone())
    ys = []
    for s, r in enumerate(ranks):
        back = []
        for g in range(world):                      # what rank g reduced for sender s, in s's order
            start = sum(outs[q].counts[g] for q in range(s))
            back.append(partials[g][start: start + outs[s].counts[g]])
        ys.append(r.finish_phase(torch.cat(back)).clone())
    return ys
