"""CPU oracle for the MoE-layer hot path (gate -> top-k -> dispatch layout ->
expert SwiGLU FFN -> combine).

THIS IS TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the test-suite, the
smoke check and the benchmark's cpu_baseline / reference arm may import it.
It is deliberately plain and slow: numpy in fp64, one step per function, no
blocking, no fusion, no reordering beyond what each definition states.  It
shares no code, table or helper with the CUDA path.

What the paper fixes, and where:

* Sec. II-A ("MoE Structure and Expert Parallelism"): every token activates the
  ``topk`` experts chosen by the gate; each chosen expert runs its FFN (GEMM-1,
  GEMM-2); the ``topk`` outputs are aggregated.  Dispatch sends a token to the
  GPUs (here: logical expert groups) hosting its experts, Combine brings the
  outputs back.
* Sec. III-C (ISA extension): the reduction in Combine is un-weighted; expert i
  scales its output o_i by the gate weight w_i in GEMM-2's epilogue, so the
  plain sum  sum_i (w_i * o_i)  is the weighted result.
* Sec. III-D (switch): a target expert is routed to output port
  ``Target / #experts_per_GPU``; one replica per port, trimmed to that port's
  targets.  => expert -> group map  g(e) = e // (E // G)  and one dispatched
  copy of a token per distinct group.
* Sec. III-D (AL table, AL management, MV translation): each destination keeps
  a table  algebraic index (token id) -> layout index (row in its dense
  buffer); rows are handed out by a running counter; Combine re-uses the table
  Dispatch built because experts do not reorder tokens; a row's address is
  base + LIdx * bsize.
* Sec. IV-B (TID table): per layout block the token id it holds.

Readings taken where the paper is silent (also listed in the design notes):
linear fp32 gate; key = logit (+ bias) in one fp32 add; top-k ordered by
(key descending, expert index ascending) with IEEE comparison (-0.0 == +0.0);
weights = softmax over the k selected keys, or sigmoid(key) renormalised over
the k selected; SwiGLU experts  (silu(x W1) * (x W3)) W2 ; rows inside an
expert / group buffer in ascending token order (one legal arrival order of the
paper's counter allocation); no capacity limit, no token dropping.

Pins: every function below is pinned by tests that do not re-type its formula:
pure-Python brute force over all (token, expert) / (token, group) pairs, a
hand-worked layout example, closed forms (k = 1, equal keys, two-key softmax =
logistic), invariants, the dense-MLP special case, and the paper's printed
340 % / "nearly 50 %" traffic figures for the distinct-group counter; the backward functions
by central finite differences of the (pinned) forward and by fp64 automatic differentiation of the
dense single-expert case; the packet model by the paper's printed 80 % -> 69 %.
"""
from __future__ import annotations

from typing import Dict, Optional, Sequence

import numpy as np

SCORE_SOFTMAX = 0
SCORE_SIGMOID = 1


# --------------------------------------------------------------------------- bf16
def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Decode raw bf16 bit patterns (uint16) exactly into float64."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    with np.errstate(invalid="ignore"):           # signalling-NaN patterns stay NaN
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(v: np.ndarray) -> np.ndarray:
    """Round float64 -> bf16 (to nearest, ties to even) and return the bits."""
    f = np.ascontiguousarray(v, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32)
    # float64 -> float32 -> bf16 double rounding is avoided for the inputs used
    # here (values are produced by sums of bf16 products, far from fp32 ties).
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    out = ((u + rounding) >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(f)
    if nan.any():
        out = np.where(nan, np.uint16(0x7FC0), out)
    return out


# --------------------------------------------------------------------------- gate
def gate_logits(x_bits: np.ndarray, w_gate: np.ndarray) -> np.ndarray:
    """Sec. II-A gate network, read as a linear layer:
    logits[t, e] = sum_i x[t, i] * w_gate[i, e]  in fp64, rounded once to fp32."""
    x = bf16_to_f64(x_bits)
    w = np.asarray(w_gate, dtype=np.float32).astype(np.float64)
    return (x @ w).astype(np.float32)


def route_keys(logits: np.ndarray, bias: Optional[np.ndarray]) -> np.ndarray:
    """key = fl32(logit + bias): a single IEEE fp32 addition; bias is None,
    [E] or [T, E]."""
    logits = np.asarray(logits, dtype=np.float32)
    if bias is None:
        return logits.copy()
    b = np.asarray(bias, dtype=np.float32)
    return (logits + (b[None, :] if b.ndim == 1 else b)).astype(np.float32)


def topk_select(keys: np.ndarray, k: int) -> np.ndarray:
    """Sec. II-A "topk experts selected by the gate": per row the k largest
    keys, ordered by (key descending, expert index ascending); the lowest index
    wins a tie; -0.0 and +0.0 tie.  Returns int32 [T, k]."""
    keys = np.asarray(keys, dtype=np.float32)
    if np.isnan(keys).any():
        raise ValueError("NaN router key: routing is undefined")
    # stable ascending sort of the negated keys = descending keys, ties by index
    order = np.argsort(-keys.astype(np.float64) + 0.0, axis=1, kind="stable")
    return order[:, :k].astype(np.int32)


def gate_weights(keys: np.ndarray, idx: np.ndarray, score_fn: int) -> np.ndarray:
    """Gate weights of the selected experts, fp64, summing to 1 per token.
    score_fn 0: softmax over the k selected keys;  1: sigmoid(key) / sum."""
    sel = np.take_along_axis(np.asarray(keys, dtype=np.float32).astype(np.float64),
                             idx.astype(np.int64), axis=1)
    if score_fn == SCORE_SOFTMAX:
        z = np.exp(sel - sel[:, :1])          # sel[:, 0] is the row maximum
        return z / z.sum(axis=1, keepdims=True)
    if score_fn == SCORE_SIGMOID:
        s = 1.0 / (1.0 + np.exp(-sel))
        return s / s.sum(axis=1, keepdims=True)
    raise ValueError("score_fn must be 0 (softmax) or 1 (sigmoid)")


def route(logits: np.ndarray, bias: Optional[np.ndarray], k: int, score_fn: int):
    """keys -> (topk_idx int32 [T,k], topk_w float64 [T,k])."""
    keys = route_keys(logits, bias)
    idx = topk_select(keys, k)
    return idx, gate_weights(keys, idx, score_fn)


# --------------------------------------------------------------------------- layout
def expert_group(e, E: int, G: int):
    """Sec. III-D switch routing rule: port = target // experts_per_GPU."""
    return e // (E // G)


def layout(topk_idx: np.ndarray, E: int, G: int) -> Dict[str, np.ndarray]:
    """Canonical dispatch layout (all int32), a pure function of topk_idx.

    expert side (one AL sub-table per expert, Sec. III-D):
      expert_counts[e]   rows of expert e  (the paper's nactive[expert])
      expert_offsets[e]  exclusive prefix sum, [E] = T*k
      row_pair[r]        flat pair index t*k+j held by expert-sorted row r;
                         rows sorted by (expert, token) = stable counting sort
      pair_row[p]        inverse of row_pair
    group side (one dispatched copy per distinct (token, group)):
      group_counts[g], group_offsets[g] ([G] = N_disp)
      al[g, t]           layout index of token t inside group g, or -1
      disp_token[n]      token held by dispatched row n (TID table)
      row_src[r]         dispatched row that feeds expert row r
    """
    idx = np.asarray(topk_idx, dtype=np.int64)
    T, k = idx.shape
    if E % G:
        raise ValueError("E must be a multiple of G")
    flat = idx.reshape(-1)
    expert_counts = np.bincount(flat, minlength=E).astype(np.int64)
    expert_offsets = np.concatenate([[0], np.cumsum(expert_counts)])
    row_pair = np.argsort(flat, kind="stable")            # by expert, then pair index
    pair_row = np.empty(T * k, dtype=np.int64)
    pair_row[row_pair] = np.arange(T * k)

    grp = expert_group(idx, E, G)                          # [T, k]
    touch = np.zeros((G, T), dtype=bool)
    for j in range(k):
        touch[grp[:, j], np.arange(T)] = True
    group_counts = touch.sum(axis=1).astype(np.int64)
    group_offsets = np.concatenate([[0], np.cumsum(group_counts)])
    # running counter per group, tokens taken in ascending order
    al = np.where(touch, np.cumsum(touch, axis=1) - 1, -1)
    n_disp = int(group_offsets[G])
    disp_token = np.empty(n_disp, dtype=np.int64)
    for g in range(G):
        disp_token[group_offsets[g]:group_offsets[g + 1]] = np.nonzero(touch[g])[0]
    row_t = row_pair // k
    row_g = expert_group(flat[row_pair], E, G)
    row_src = group_offsets[row_g] + al[row_g, row_t]
    i32 = lambda a: np.ascontiguousarray(a, dtype=np.int32)
    return {
        "expert_counts": i32(expert_counts), "expert_offsets": i32(expert_offsets),
        "row_pair": i32(row_pair), "pair_row": i32(pair_row),
        "group_counts": i32(group_counts), "group_offsets": i32(group_offsets),
        "al": i32(al), "disp_token": i32(disp_token), "row_src": i32(row_src),
        "n_disp": n_disp,
    }


def dispatch(x_bits: np.ndarray, lay: Dict[str, np.ndarray]) -> np.ndarray:
    """Dispatch result: xg[n, :] = x[disp_token[n], :], a byte copy."""
    return np.ascontiguousarray(x_bits[lay["disp_token"].astype(np.int64)])


# --------------------------------------------------------------------------- experts
def expert_ffn_rows_f64(a: np.ndarray, w1: np.ndarray, w3: np.ndarray, w2: np.ndarray) -> np.ndarray:
    """One expert with float64 weights applied to rows ``a`` (float64 [n, d]):
    GEMM-1  a1 = a W1, a3 = a W3 ;  h = silu(a1) * a3 ;  GEMM-2  o = h W2."""
    a1 = a @ w1
    a3 = a @ w3
    h = a1 / (1.0 + np.exp(-a1)) * a3
    return h @ w2


def expert_ffn_rows(a: np.ndarray, w1_bits: np.ndarray, w3_bits: np.ndarray,
                    w2_bits: np.ndarray) -> np.ndarray:
    """One expert applied to rows ``a`` (float64 [n, d]), weights given as bf16 bits.
    All in fp64, no intermediate rounding."""
    return expert_ffn_rows_f64(a, bf16_to_f64(w1_bits), bf16_to_f64(w3_bits), bf16_to_f64(w2_bits))


def expert_ffn(xg_bits: np.ndarray, lay: Dict[str, np.ndarray], topk_w: Optional[np.ndarray],
               w1_bits: np.ndarray, w3_bits: np.ndarray, w2_bits: np.ndarray,
               rows: Optional[np.ndarray] = None) -> np.ndarray:
    """Expert outputs in expert-sorted row order, float64 [P, d] (or only the
    requested ``rows``).  Row r of expert e reads dispatched row row_src[r].
    With ``topk_w`` ([T, k]) the gate weight is applied here (GEMM-2 epilogue,
    Sec. III-C); with None the rows are left un-weighted."""
    off = lay["expert_offsets"].astype(np.int64)
    P = int(off[-1])
    d = xg_bits.shape[1]
    want = np.arange(P) if rows is None else np.asarray(rows, dtype=np.int64)
    out = np.zeros((want.size, d), dtype=np.float64)
    row_e = np.searchsorted(off, want, side="right") - 1
    for e in np.unique(row_e):
        sel = np.nonzero(row_e == e)[0]
        r = want[sel]
        a = bf16_to_f64(xg_bits[lay["row_src"][r].astype(np.int64)])
        o = expert_ffn_rows(a, w1_bits[e], w3_bits[e], w2_bits[e])
        if topk_w is not None:
            o = o * np.asarray(topk_w, dtype=np.float64).reshape(-1)[lay["row_pair"][r].astype(np.int64)][:, None]
        out[sel] = o
    return out


# --------------------------------------------------------------------------- combine
def combine(o: np.ndarray, lay: Dict[str, np.ndarray], topk_idx: np.ndarray,
            topk_w: Optional[np.ndarray], E: int, G: int,
            tokens: Optional[Sequence[int]] = None, o_rows: Optional[np.ndarray] = None):
    """Two-level combine (Sec. III-D reduction logic + Sec. II-A aggregation):
    pg[n] = sum of the expert rows of token t that live in group g, for the
    dispatched row n = (t, g)  (same layout as the dispatch buffer);
    y[t] = sum over the groups t touched of pg[(t, g)].

    ``o`` holds expert-sorted rows in float64: either all P rows, or (with
    ``o_rows`` = the sorted row numbers it holds) a subset.  If ``topk_w`` is
    given the rows are weighted here instead of in GEMM-2's epilogue.
    Returns (pg_n, pg, y): the dispatched-row numbers touched by the requested
    tokens (all tokens if None) in ascending order, their partial sums, and
    y [len(tokens), d]."""
    idx = np.asarray(topk_idx, dtype=np.int64)
    T, k = idx.shape
    d = o.shape[1]
    toks = np.arange(T) if tokens is None else np.asarray(tokens, dtype=np.int64)
    goff = lay["group_offsets"].astype(np.int64)
    partial: Dict[int, np.ndarray] = {}
    for t in toks:
        for j in range(k):
            g = expert_group(int(idx[t, j]), E, G)
            n = int(goff[g]) + int(lay["al"][g, t])
            r = int(lay["pair_row"][t * k + j])
            if o_rows is not None:
                r = int(np.searchsorted(o_rows, r))
            row = o[r] if topk_w is None else float(topk_w[t, j]) * o[r]
            partial[n] = partial[n] + row if n in partial else row.copy()
    pg_n = np.array(sorted(partial), dtype=np.int64)
    pg = np.stack([partial[n] for n in pg_n]) if pg_n.size else np.zeros((0, d))
    y = np.zeros((toks.size, d), dtype=np.float64)
    pos = {int(t): i for i, t in enumerate(toks)}
    for n, v in zip(pg_n, pg):
        y[pos[int(lay["disp_token"][n])]] += v
    return pg_n, pg, y


# --------------------------------------------------------------------------- whole layer
def layer(x_bits: np.ndarray, logits: np.ndarray, bias: Optional[np.ndarray],
          w1_bits, w3_bits, w2_bits, k: int, score_fn: int,
          tokens: Optional[Sequence[int]] = None):
    """Dense definition of the layer for the given tokens (all if None):
    y[t] = sum_j w[t, j] * FFN_{idx[t, j]}(x[t])  in fp64 (Sec. II-A, III-C).
    ``logits`` are the fp32 router logits to route on.  ``w*_bits`` may be any
    object indexable by expert that yields that expert's bf16 bit matrix (so
    large weight sets can be fetched slab by slab).
    Returns (tokens, idx[tokens], w[tokens], y float64 [len(tokens), d])."""
    idx, w = route(logits, bias, k, score_fn)
    T = x_bits.shape[0]
    toks = np.arange(T) if tokens is None else np.asarray(tokens, dtype=np.int64)
    y = np.zeros((toks.size, x_bits.shape[1]), dtype=np.float64)
    sel_idx = idx[toks]
    for e in np.unique(sel_idx):
        hit_t, hit_j = np.nonzero(sel_idx == e)
        a = bf16_to_f64(x_bits[toks[hit_t]])
        o = expert_ffn_rows(a, w1_bits[e], w3_bits[e], w2_bits[e])
        y[hit_t] += w[toks[hit_t], hit_j][:, None] * o
    return toks, sel_idx, w[toks], y


# --------------------------------------------------------------------------- backward
def expert_ffn_rows_backward_f64(a: np.ndarray, w1: np.ndarray, w3: np.ndarray, w2: np.ndarray, do: np.ndarray):
    """Gradients of  sum(do * o),  o = (silu(a W1) * (a W3)) W2,  with respect to a, W1, W3, W2 (the chain rule
    written out, fp64).  ``do`` is float64 [n, d].  Returns (da, dW1, dW3, dW2)."""
    a1 = a @ w1
    a3 = a @ w3
    s = 1.0 / (1.0 + np.exp(-a1))
    silu = a1 * s
    h = silu * a3
    dh = do @ w2.T
    da3 = dh * silu
    da1 = dh * a3 * (s * (1.0 + a1 * (1.0 - s)))     # d silu(u) / du = s (1 + u (1 - s))
    da = da1 @ w1.T + da3 @ w3.T
    return da, a.T @ da1, a.T @ da3, h.T @ do


def layer_backward(x_bits: np.ndarray, topk_idx: np.ndarray, topk_w: np.ndarray, w1_bits, w3_bits, w2_bits,
                   dy: np.ndarray, experts: Optional[Sequence[int]] = None):
    """Backward pass of the layer for FIXED routing (Sec. VI-A evaluates training, forward + backward): with
    y[t] = sum_j w[t, j] * FFN_{idx[t, j]}(x[t])  and the expert indices and gate weights held constant,
    the gradients of  L = sum(dy * y)  are
        dx[t]  = sum_j  w[t, j] * dFFN/da (x[t]) applied to dy[t]
        dW*[e] = sum over the pairs (t, j) with idx[t, j] = e  of  w[t, j] * (their expert-level gradient).
    ``dy`` float64 [T, d]; ``topk_w`` [T, k]; entries of ``topk_idx`` below 0 are slots not in use and contribute
    nothing.  With ``experts`` only those experts' weight gradients are formed
    (dx is then omitted).  Returns (dx [T, d] or None, {e: (dW1, dW3, dW2)}), all float64."""
    idx = np.asarray(topk_idx, dtype=np.int64)
    w = np.asarray(topk_w, dtype=np.float64)
    T = x_bits.shape[0]
    dx = np.zeros((T, x_bits.shape[1]), dtype=np.float64) if experts is None else None
    grads = {}
    for e in (np.unique(idx) if experts is None else experts):
        if e < 0:            # slot not in use (a routing table trimmed to one group's experts, Sec. III-D)
            continue
        hit_t, hit_j = np.nonzero(idx == e)
        w1, w3, w2 = bf16_to_f64(w1_bits[e]), bf16_to_f64(w3_bits[e]), bf16_to_f64(w2_bits[e])
        if hit_t.size == 0:
            grads[int(e)] = (np.zeros_like(w1), np.zeros_like(w3), np.zeros_like(w2))
            continue
        a = bf16_to_f64(x_bits[hit_t])
        do = w[hit_t, hit_j][:, None] * np.asarray(dy, dtype=np.float64)[hit_t]
        da, g1, g3, g2 = expert_ffn_rows_backward_f64(a, w1, w3, w2, do)
        if dx is not None:
            np.add.at(dx, hit_t, da)
        grads[int(e)] = (g1, g3, g2)
    return dx, grads


def gate_backward(x_bits: np.ndarray, w_gate: np.ndarray, bias: Optional[np.ndarray], topk_idx: np.ndarray,
                  score_fn: int, w1_bits, w3_bits, w2_bits, dy: np.ndarray):
    """Gradient that reaches the gate network when the SELECTION is held fixed but the gate weights are functions of
    the router keys (Sec. II-A: the gate picks the topk experts and weighs their outputs; Sec. VI-A: training).  With
        key[t, e] = x[t] . w_gate[:, e] + bias[t, e],   w[t, :] = softmax / renormalised sigmoid of key[t, topk_idx[t, :]],
        y[t] = sum_j w[t, j] * FFN_{idx[t, j]}(x[t])   and   L = sum(dy * y):
        dL/dw[t, j]   = dy[t] . FFN_{idx[t, j]}(x[t])
        dL/dkey[t, j] = softmax:  w_j (dL/dw_j - sum_i w_i dL/dw_i)
                        sigmoid:  s_j (1 - s_j) (dL/dw_j - sum_i w_i dL/dw_i) / sum_i s_i,   s = sigmoid(key)
        dL/dw_gate    = x^T . dlogits      (dlogits[t, e] = dL/dkey[t, j] at e = idx[t, j], else 0)
        dx_gate[t]    = dlogits[t] . w_gate^T          (added to the dx of ``layer_backward``).
    All in fp64; keys are formed in fp64 from the bf16 x and the fp32 gate weight (no rounding of the logits).
    Returns (dw_gate [d, E], dx_gate [T, d], dkey [T, k], dL/dw [T, k])."""
    idx = np.asarray(topk_idx, dtype=np.int64)
    x = bf16_to_f64(x_bits)
    wg = np.asarray(w_gate, dtype=np.float32).astype(np.float64)
    T, k = idx.shape
    keys = x @ wg
    if bias is not None:
        b = np.asarray(bias, dtype=np.float32).astype(np.float64)
        keys = keys + (b[None, :] if b.ndim == 1 else b)
    sel = np.take_along_axis(keys, idx, axis=1)
    if score_fn == SCORE_SOFTMAX:
        z = np.exp(sel - sel.max(axis=1, keepdims=True))
        w = z / z.sum(axis=1, keepdims=True)
    elif score_fn == SCORE_SIGMOID:
        sg = 1.0 / (1.0 + np.exp(-sel))
        ssum = sg.sum(axis=1, keepdims=True)
        w = sg / ssum
    else:
        raise ValueError("score_fn must be 0 (softmax) or 1 (sigmoid)")
    dyf = np.asarray(dy, dtype=np.float64)
    dw = np.zeros((T, k), dtype=np.float64)
    for e in np.unique(idx):
        hit_t, hit_j = np.nonzero(idx == e)
        o = expert_ffn_rows(x[hit_t], w1_bits[e], w3_bits[e], w2_bits[e])
        dw[hit_t, hit_j] = np.sum(o * dyf[hit_t], axis=1)
    centred = dw - np.sum(w * dw, axis=1, keepdims=True)
    if score_fn == SCORE_SOFTMAX:
        dkey = w * centred
    else:
        dkey = sg * (1.0 - sg) * centred / ssum
    dlogits = np.zeros_like(keys)
    np.put_along_axis(dlogits, idx, dkey, axis=1)
    return x.T @ dlogits, dlogits @ wg.T, dkey, dw


# --------------------------------------------------------------------------- traffic counters
def distinct_groups_per_token(topk_idx: np.ndarray, E: int, G: int) -> float:
    """Mean number D of distinct destination groups per token = N_disp / T."""
    lay = layout(topk_idx, E, G)
    return lay["n_disp"] / topk_idx.shape[0]


def redundancy_figures(D: float, G: int, k: Optional[int] = None) -> Dict[str, float]:
    """Traffic ratios of Sec. II-B / II-C from the mean distinct-destination
    count D of a G-GPU system:
    * allgather_useless = (G - D) / D : extra traffic when Dispatch is emulated
      by AllGather (every GPU receives every token);
    * redundant_share = (D - 1) / (2 D): share of the source<->switch link
      traffic that in-switch multicast / reduction removes (one of D copies is
      needed in the redundant direction, all D in the other);
    * ideal_speedup = 2 D / (1 + D)."""
    return {"allgather_useless": (G - D) / D,
            "redundant_share": (D - 1.0) / (2.0 * D),
            "ideal_speedup": 2.0 * D / (1.0 + D)}


# --------------------------------------------------------------------------- packet model
FLIT_BYTES = 16            # Sec. III-B: the link packet is a sequence of 16-byte flits
PACKET_DATA_FLITS = 16     # largest payload of one packet: 256 bytes
PACKET_OVERHEAD_FLITS = 4  # non-data flits per full packet over request + response; the value that makes
                           # the efficiency of plain (single-destination) transfers the paper's "ideal 80 %"
IDS_PER_EXTENSION_FLIT = 8 # Sec. III-B: eight 16-bit expert ids per target-extension flit


def payload_efficiency(transfer_bytes: int, n_targets: int) -> Dict[str, float]:
    """Payload efficiency (data flits / all transmitted flits, Sec. VI-B) of one multi-destination
    transfer of ``transfer_bytes`` under the three addressing schemes of Sec. III-A / III-B:

    * ideal: the transfer cut into packets of at most 256 bytes, each with its fixed header share;
    * explicit addressing: one destination flit per target in the request and as many again in the
      response (Sec. III-A: eight GPUs need eight destination flits both ways);
    * dynamic multimem addressing: the one multimem address stays in flit0 and the target list adds
      ceil(n_targets / 8) extension flits to the request (Sec. III-B).

    The paper gives the flit counts and the two efficiencies of its example; the fixed header share
    and the size of that example are not stated (readings, see the constants above)."""
    data = -(-int(transfer_bytes) // FLIT_BYTES)
    packets = -(-data // PACKET_DATA_FLITS)
    base = data + packets * PACKET_OVERHEAD_FLITS
    explicit = base + 2 * int(n_targets)
    dynamic = base + -(-int(n_targets) // IDS_PER_EXTENSION_FLIT)
    return {"data_flits": float(data), "ideal": data / base, "explicit": data / explicit, "dynamic": data / dynamic}
