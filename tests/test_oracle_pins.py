"""Pins for the CPU oracle: every oracle function is checked against something
other than itself - pure-Python brute force over all pairs, a hand-worked
example, closed forms, invariants, library special cases and the traffic
figures the paper prints.  No GPU involved."""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2605_05607_b200 import synth

RNG = np.random.default_rng(7)


def rand_bf16_bits(shape, scale=1.0, rng=RNG):
    t = torch.from_numpy(rng.standard_normal(shape).astype(np.float32) * scale).to(torch.bfloat16)
    return synth.bf16_bits(t)


def bf16_scalar(bits):
    """Independent scalar decode of one bf16 pattern (struct, not numpy views)."""
    import struct
    return struct.unpack("<f", struct.pack("<I", int(bits) << 16))[0]


# ---------------------------------------------------------------- bf16 codec
def test_bf16_decode_all_patterns_match_torch():
    bits = np.arange(65536, dtype=np.uint16)
    ours = O.bf16_to_f64(bits)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    both_nan = np.isnan(ours) & np.isnan(ref)
    assert np.array_equal(ours[~both_nan], ref[~both_nan])
    assert bf16_scalar(0x3FC0) == 1.5 and O.bf16_to_f64(np.array([0x3FC0], np.uint16))[0] == 1.5


def test_bf16_encode_matches_torch_rounding():
    v = RNG.standard_normal(20000) * 3.0
    v[:4] = [1.00390625, 1.01171875, -0.0, 65280.0]  # exact ties (to even) and specials
    ours = O.f64_to_bf16_bits(v)
    ref = synth.bf16_bits(torch.from_numpy(v.astype(np.float32)).to(torch.bfloat16))
    assert np.array_equal(ours, ref)


# ---------------------------------------------------------------- gate logits
def test_gate_logits_bruteforce_fsum():
    T, d, E = 5, 24, 6
    xb = rand_bf16_bits((T, d))
    wg = (RNG.standard_normal((d, E)) * 0.02).astype(np.float32)
    got = O.gate_logits(xb, wg)
    assert got.dtype == np.float32 and got.shape == (T, E)
    for t in range(T):
        for e in range(E):
            exact = math.fsum(bf16_scalar(xb[t, i]) * float(wg[i, e]) for i in range(d))
            assert got[t, e] == np.float32(exact)


def test_gate_logits_not_transposed():
    # one-hot x row picks out a row of w_gate
    d, E = 8, 3
    x = torch.zeros(2, d, dtype=torch.bfloat16)
    x[0, 5] = 1.0
    x[1, 2] = -2.0
    wg = np.arange(d * E, dtype=np.float32).reshape(d, E)
    got = O.gate_logits(synth.bf16_bits(x), wg)
    assert np.array_equal(got[0], wg[5]) and np.array_equal(got[1], -2.0 * wg[2])


# ---------------------------------------------------------------- top-k
def brute_topk(row, k):
    return sorted(range(len(row)), key=lambda e: (-float(row[e]) if row[e] != 0 else 0.0, e))[:k]


@pytest.mark.parametrize("E,k", [(4, 1), (8, 2), (16, 4), (8, 8), (33, 5)])
def test_topk_bruteforce_with_ties_everywhere(E, k):
    # keys drawn from four values, so ties are everywhere incl. the k / k+1 border
    keys = RNG.choice(np.array([-1.0, -0.0, 0.0, 0.5], np.float32), size=(64, E))
    got = O.topk_select(keys, k)
    for t in range(keys.shape[0]):
        assert list(got[t]) == brute_topk(keys[t], k)


def test_topk_crafted_rows():
    assert list(O.topk_select(np.full((1, 6), 3.0, np.float32), 3)[0]) == [0, 1, 2]
    assert list(O.topk_select(np.array([[1, 7, 2, 7, 0]], np.float32), 2)[0]) == [1, 3]
    assert list(O.topk_select(np.array([[-0.0, 0.0, -1.0]], np.float32), 2)[0]) == [0, 1]
    assert list(O.topk_select(np.array([[0.0, -0.0, 1.0]], np.float32), 3)[0]) == [2, 0, 1]
    assert list(O.topk_select(np.array([[-np.inf, np.inf, 0.0]], np.float32), 2)[0]) == [1, 2]
    with pytest.raises(ValueError):
        O.topk_select(np.array([[np.nan, 0.0]], np.float32), 1)


def test_topk_invariants_random():
    keys = RNG.standard_normal((200, 40)).astype(np.float32)
    k = 6
    idx = O.topk_select(keys, k)
    for t in range(200):
        sel = idx[t]
        assert len(set(sel)) == k
        kv = keys[t, sel]
        assert np.all(kv[:-1] >= kv[1:])
        rest = np.setdiff1d(np.arange(40), sel)
        assert np.all(keys[t, rest] <= kv[-1])


def test_route_keys_single_fp32_add():
    logits = np.array([[1e8, 1.0, 0.1]], np.float32)
    bias = np.array([1.0, 1e-8, 0.2], np.float32)
    got = O.route_keys(logits, bias)
    exp = [np.float32(np.float32(a) + np.float32(b)) for a, b in zip(logits[0], bias)]
    assert got.dtype == np.float32 and list(got[0]) == exp
    assert got[0, 0] == np.float32(1e8)  # absorbed, as fp32 addition must
    full = np.tile(bias, (1, 1))
    assert np.array_equal(O.route_keys(logits, full), got)
    assert np.array_equal(O.route_keys(logits, None), logits)


# ---------------------------------------------------------------- gate weights
def test_gate_weights_closed_forms():
    keys = RNG.standard_normal((50, 12)).astype(np.float32)
    for fn in (O.SCORE_SOFTMAX, O.SCORE_SIGMOID):
        for k in (1, 2, 5):
            idx = O.topk_select(keys, k)
            w = O.gate_weights(keys, idx, fn)
            assert np.allclose(w.sum(axis=1), 1.0, atol=1e-15)
            assert np.all(w > 0)
            if k == 1:
                assert np.all(w == 1.0)
    # equal keys -> 1/k for both score functions
    eq = np.full((3, 8), 0.75, np.float32)
    for fn in (0, 1):
        w = O.gate_weights(eq, O.topk_select(eq, 4), fn)
        assert np.allclose(w, 0.25, atol=1e-16)
    # two-key softmax is the logistic function of the key difference
    idx = O.topk_select(keys, 2)
    w = O.gate_weights(keys, idx, O.SCORE_SOFTMAX)
    for t in range(50):
        a, b = float(keys[t, idx[t, 0]]), float(keys[t, idx[t, 1]])
        assert w[t, 0] == pytest.approx(1.0 / (1.0 + math.exp(b - a)), rel=1e-14)


def test_gate_weights_bruteforce_scalar():
    keys = RNG.standard_normal((10, 9)).astype(np.float32) * 2
    idx = O.topk_select(keys, 3)
    ws = O.gate_weights(keys, idx, O.SCORE_SOFTMAX)
    wg = O.gate_weights(keys, idx, O.SCORE_SIGMOID)
    for t in range(10):
        ks = [float(keys[t, e]) for e in idx[t]]
        z = [math.exp(v) for v in ks]
        s = [1.0 / (1.0 + math.exp(-v)) for v in ks]
        for j in range(3):
            assert ws[t, j] == pytest.approx(z[j] / math.fsum(z), rel=1e-13)
            assert wg[t, j] == pytest.approx(s[j] / math.fsum(s), rel=1e-13)
    # weights follow the keys' order
    assert np.all(ws[:, :-1] >= ws[:, 1:]) and np.all(wg[:, :-1] >= wg[:, 1:])


# ---------------------------------------------------------------- layout
def brute_layout(idx, E, G):
    """Enumerate every (token, expert) and (token, group) pair in plain Python."""
    T, k = len(idx), len(idx[0])
    m = E // G
    rows = []                                     # expert-sorted rows
    for e in range(E):
        for t in range(T):
            for j in range(k):
                if idx[t][j] == e:
                    rows.append(t * k + j)
    counts = [sum(1 for t in range(T) for j in range(k) if idx[t][j] == e) for e in range(E)]
    offs = [sum(counts[:e]) for e in range(E + 1)]
    pair_row = [rows.index(p) for p in range(T * k)]
    al = [[-1] * T for _ in range(G)]
    disp = []
    gcounts = []
    for g in range(G):
        c = 0
        for t in range(T):
            if any(idx[t][j] // m == g for j in range(k)):
                al[g][t] = c
                c += 1
                disp.append(t)
        gcounts.append(c)
    goffs = [sum(gcounts[:g]) for g in range(G + 1)]
    row_src = []
    for r, p in enumerate(rows):
        t, j = divmod(p, k)
        g = idx[t][j] // m
        row_src.append(goffs[g] + al[g][t])
    return dict(expert_counts=counts, expert_offsets=offs, row_pair=rows, pair_row=pair_row,
                group_counts=gcounts, group_offsets=goffs, al=al, disp_token=disp, row_src=row_src,
                n_disp=len(disp))


def assert_layout_equal(got, exp):
    for key, val in exp.items():
        if key == "n_disp":
            assert got["n_disp"] == val
        else:
            assert got[key].dtype == np.int32, key
            assert np.array_equal(got[key], np.asarray(val, dtype=np.int32)), key


def test_layout_golden_worked_example(golden_dir):
    gold = json.load(open(os.path.join(golden_dir, "layout_worked_example.json")))
    lay = O.layout(np.array(gold["topk_idx"], np.int32), gold["E"], gold["G"])
    assert_layout_equal(lay, {k: gold[k] for k in
                              ("expert_counts", "expert_offsets", "row_pair", "pair_row", "group_counts",
                               "group_offsets", "n_disp", "al", "disp_token", "row_src")})


def random_topk(T, E, k, rng):
    return np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)


@pytest.mark.parametrize("T,E,k,G", [(1, 1, 1, 1), (7, 4, 2, 2), (13, 8, 3, 4), (9, 8, 8, 2),
                                     (20, 6, 2, 6), (20, 6, 3, 1), (40, 12, 4, 3)])
def test_layout_bruteforce(T, E, k, G):
    idx = random_topk(T, E, k, RNG)
    assert_layout_equal(O.layout(idx, E, G), brute_layout(idx.tolist(), E, G))


def test_layout_invariants_and_degenerate_groups():
    T, E, k = 300, 32, 4
    idx = random_topk(T, E, k, RNG)
    idx[:, 0] = np.where(idx[:, 0] == 5, idx[:, 0], idx[:, 0])  # keep distinct per row
    for G in (1, 4, 8, 32):
        lay = O.layout(idx, E, G)
        assert lay["expert_counts"].sum() == T * k and lay["expert_offsets"][-1] == T * k
        assert np.all(np.diff(lay["expert_offsets"]) == lay["expert_counts"])
        assert np.array_equal(np.sort(lay["row_pair"]), np.arange(T * k))
        assert np.array_equal(lay["pair_row"][lay["row_pair"]], np.arange(T * k))
        row_e = idx.reshape(-1)[lay["row_pair"]]
        assert np.all(np.diff(row_e) >= 0)
        for e in range(E):
            seg = lay["row_pair"][lay["expert_offsets"][e]:lay["expert_offsets"][e + 1]] // k
            assert np.all(np.diff(seg) > 0)               # tokens ascending, none twice
        pairs = {(t, int(e) // (E // G)) for t in range(T) for e in idx[t]}
        assert lay["n_disp"] == len(pairs) == lay["group_offsets"][-1]
        assert T <= lay["n_disp"] <= T * min(k, G)
        if G == E:
            assert lay["n_disp"] == T * k
        if G == 1:
            assert lay["n_disp"] == T and np.array_equal(lay["disp_token"], np.arange(T))
        assert np.array_equal(lay["al"] >= 0,
                              np.array([[(t, g) in pairs for t in range(T)] for g in range(G)]))
        for g in range(G):
            seg = lay["disp_token"][lay["group_offsets"][g]:lay["group_offsets"][g + 1]]
            assert np.all(np.diff(seg) > 0)
        # the dispatched row of an expert row holds that row's token
        assert np.array_equal(lay["disp_token"][lay["row_src"]], lay["row_pair"] // k)


def test_layout_empty_experts_and_k_equals_E():
    idx = np.array([[3, 1]] * 5, np.int32)                # experts 0, 2 never used
    lay = O.layout(idx, 4, 2)
    assert list(lay["expert_counts"]) == [0, 5, 0, 5]
    assert lay["n_disp"] == 10
    idx = np.array([[2, 0, 1, 3], [0, 1, 2, 3]], np.int32)
    lay = O.layout(idx, 4, 2)
    assert list(lay["expert_counts"]) == [2, 2, 2, 2] and lay["n_disp"] == 4
    with pytest.raises(ValueError):
        O.layout(idx, 4, 3)


def test_dispatch_is_byte_copy():
    T, d, E, k, G = 11, 16, 8, 3, 4
    xb = rand_bf16_bits((T, d))
    idx = random_topk(T, E, k, RNG)
    lay = O.layout(idx, E, G)
    xg = O.dispatch(xb, lay)
    assert xg.dtype == np.uint16 and xg.shape == (lay["n_disp"], d)
    b = brute_layout(idx.tolist(), E, G)
    for n, t in enumerate(b["disp_token"]):
        assert xg[n].tobytes() == xb[t].tobytes()


# ---------------------------------------------------------------- traffic figures
def closed_form_D(E, G, k):
    m = E // G
    return G * (1.0 - math.comb(E - m, k) / math.comb(E, k))


def test_distinct_group_counter_matches_closed_form_and_paper(golden_dir):
    gold = json.load(open(os.path.join(golden_dir, "paper_traffic_figures.json")))
    E, G = gold["E"], gold["G"]
    rng = np.random.default_rng(0)
    for k in (8, 16, 32):
        keys = rng.standard_normal((4096, E)).astype(np.float32)     # uniform routing
        D = O.distinct_groups_per_token(O.topk_select(keys, k), E, G)
        assert D == pytest.approx(closed_form_D(E, G, k), rel=0.01)
        fig = O.redundancy_figures(D, G)
        assert gold["redundant_share_min_k8"] <= fig["redundant_share"] < gold["redundant_share_max"]
        assert gold["ideal_speedup_min_k8"] <= fig["ideal_speedup"] < gold["ideal_speedup_max"]
        if k == 8:
            assert fig["allgather_useless"] == pytest.approx(gold["allgather_useless_k8"],
                                                             abs=gold["allgather_useless_tol"])


# ---------------------------------------------------------------- expert FFN
def test_expert_ffn_dense_special_case_vs_torch():
    # E = k = G = 1: the layer is one dense SwiGLU MLP; check against torch fp64
    n, d, f = 6, 16, 24
    xb = rand_bf16_bits((n, d))
    w1, w3, w2 = rand_bf16_bits((d, f), 0.3), rand_bf16_bits((d, f), 0.3), rand_bf16_bits((f, d), 0.3)
    got = O.expert_ffn_rows(O.bf16_to_f64(xb), w1, w3, w2)
    tx = synth.bits_to_bf16(xb).double()
    t1, t3, t2 = (synth.bits_to_bf16(w).double() for w in (w1, w3, w2))
    ref = (torch.nn.functional.silu(tx @ t1) * (tx @ t3)) @ t2
    assert np.allclose(got, ref.numpy(), rtol=1e-12, atol=1e-14)


def test_expert_ffn_python_loops_and_operand_roles():
    n, d, f = 2, 3, 4
    xb = rand_bf16_bits((n, d))
    w1, w3, w2 = rand_bf16_bits((d, f)), rand_bf16_bits((d, f)), rand_bf16_bits((f, d))
    got = O.expert_ffn_rows(O.bf16_to_f64(xb), w1, w3, w2)
    for r in range(n):
        a1 = [math.fsum(bf16_scalar(xb[r, i]) * bf16_scalar(w1[i, c]) for i in range(d)) for c in range(f)]
        a3 = [math.fsum(bf16_scalar(xb[r, i]) * bf16_scalar(w3[i, c]) for i in range(d)) for c in range(f)]
        h = [a1[c] / (1.0 + math.exp(-a1[c])) * a3[c] for c in range(f)]
        for c in range(d):
            exp = math.fsum(h[q] * bf16_scalar(w2[q, c]) for q in range(f))
            assert got[r, c] == pytest.approx(exp, rel=1e-12, abs=1e-14)
    # W2 = 0 -> 0 ; swapping W1 and W3 changes the result (silu is on the W1 branch)
    assert np.all(O.expert_ffn_rows(O.bf16_to_f64(xb), w1, w3, np.zeros_like(w2)) == 0)
    assert not np.allclose(O.expert_ffn_rows(O.bf16_to_f64(xb), w3, w1, w2), got)


def tiny_problem(T=9, d=8, f=12, E=6, k=3, G=3, seed=3):
    rng = np.random.default_rng(seed)
    xb = rand_bf16_bits((T, d), rng=rng)
    wg = (rng.standard_normal((d, E)) * 0.5).astype(np.float32)
    w1 = rand_bf16_bits((E, d, f), 0.4, rng)
    w3 = rand_bf16_bits((E, d, f), 0.4, rng)
    w2 = rand_bf16_bits((E, f, d), 0.4, rng)
    return xb, wg, w1, w3, w2


def brute_dense_layer(xb, logits, bias, w1, w3, w2, k, score_fn):
    """y[t] = sum_e M[t, e] FFN_e(x_t) over ALL experts with a k-sparse weight
    matrix M built by plain Python; shares nothing with the permutation code."""
    T, d = xb.shape
    E = logits.shape[1]
    y = np.zeros((T, d))
    for t in range(T):
        key = [float(np.float32(logits[t, e]) + (np.float32(0) if bias is None else np.float32(bias[e])))
               for e in range(E)]
        sel = sorted(range(E), key=lambda e: (-key[e], e))[:k]
        sc = [math.exp(key[e]) if score_fn == 0 else 1.0 / (1.0 + math.exp(-key[e])) for e in sel]
        M = [0.0] * E
        for e, s in zip(sel, sc):
            M[e] = s / math.fsum(sc)
        xt = [bf16_scalar(b) for b in xb[t]]
        for e in range(E):
            f = w1.shape[2]
            a1 = [math.fsum(xt[i] * bf16_scalar(w1[e, i, c]) for i in range(d)) for c in range(f)]
            a3 = [math.fsum(xt[i] * bf16_scalar(w3[e, i, c]) for i in range(d)) for c in range(f)]
            h = [a1[c] / (1.0 + math.exp(-a1[c])) * a3[c] for c in range(f)]
            for c in range(d):
                y[t, c] += M[e] * math.fsum(h[q] * bf16_scalar(w2[e, q, c]) for q in range(f))
    return y


@pytest.mark.parametrize("score_fn", [0, 1])
def test_layer_vs_dense_bruteforce(score_fn):
    xb, wg, w1, w3, w2 = tiny_problem()
    logits = O.gate_logits(xb, wg)
    bias = np.linspace(-0.3, 0.3, wg.shape[1]).astype(np.float32)
    _, _, _, y = O.layer(xb, logits, bias, w1, w3, w2, 3, score_fn)
    ref = brute_dense_layer(xb, logits, bias, w1, w3, w2, 3, score_fn)
    assert np.allclose(y, ref, rtol=1e-11, atol=1e-13)


def test_staged_path_equals_layer_and_weight_placement():
    # dispatch -> expert_ffn -> combine must reproduce layer(); weight applied in the
    # GEMM-2 epilogue or in combine gives the same sum (Sec. III-C identity)
    xb, wg, w1, w3, w2 = tiny_problem(T=17, E=8, k=4, G=4)
    E, G, k = 8, 4, 4
    logits = O.gate_logits(xb, wg)
    idx, w = O.route(logits, None, k, 0)
    lay = O.layout(idx, E, G)
    xg = O.dispatch(xb, lay)
    o_w = O.expert_ffn(xg, lay, w, w1, w3, w2)
    o_raw = O.expert_ffn(xg, lay, None, w1, w3, w2)
    pg_n, pg_a, y_a = O.combine(o_w, lay, idx, None, E, G)
    _, pg_b, y_b = O.combine(o_raw, lay, idx, w, E, G)
    _, _, _, y_ref = O.layer(xb, logits, None, w1, w3, w2, k, 0)
    assert np.array_equal(pg_n, np.arange(lay["n_disp"]))
    assert np.allclose(y_a, y_ref, rtol=1e-12, atol=1e-14)
    assert np.allclose(y_b, y_ref, rtol=1e-12, atol=1e-14)
    assert np.allclose(pg_a, pg_b, rtol=1e-12, atol=1e-14)
    # token subset / row subset variants agree with the full computation
    toks = np.array([2, 5, 16])
    rows = np.unique(lay["pair_row"].reshape(-1, k)[toks].reshape(-1))
    o_sub = O.expert_ffn(xg, lay, w, w1, w3, w2, rows=rows)
    assert np.allclose(o_sub, o_w[rows], rtol=1e-12, atol=1e-15)   # BLAS blocking differs with the row count
    _, _, y_sub = O.combine(o_sub, lay, idx, None, E, G, tokens=toks, o_rows=rows)
    assert np.allclose(y_sub, y_a[toks], rtol=1e-12, atol=1e-15)
    t2, _, _, y2 = O.layer(xb, logits, None, w1, w3, w2, k, 0, tokens=toks)
    assert np.allclose(y2, y_ref[toks], rtol=1e-12, atol=1e-14)


def test_combine_identity_experts_k1_linearity():
    T, d, E, G = 12, 10, 6, 3
    rng = np.random.default_rng(5)
    xb = rand_bf16_bits((T, d), rng=rng)
    x = O.bf16_to_f64(xb)
    for k in (1, 2, 3):
        idx = random_topk(T, E, k, rng)
        keys = rng.standard_normal((T, E)).astype(np.float32)
        w = O.gate_weights(keys, idx, 0)
        lay = O.layout(idx, E, G)
        xg = O.dispatch(xb, lay)
        o = O.bf16_to_f64(xg[lay["row_src"]])            # "identity experts": o[r] = its input row
        _, pg, y = O.combine(o, lay, idx, w, E, G)
        assert np.allclose(y, x, rtol=1e-14, atol=1e-15)  # weights sum to 1 -> combine returns x
        if k == 1:
            assert np.array_equal(y, x)                  # pure un-permute, exact
            assert np.array_equal(pg, O.bf16_to_f64(xg))
        _, pg4, y4 = O.combine(4.0 * o, lay, idx, w, E, G)
        assert np.array_equal(y4, 4.0 * y) and np.array_equal(pg4, 4.0 * pg)
    # a token whose two experts share a group: one partial row holds both terms
    idx = np.array([[0, 1]], np.int32)
    lay = O.layout(idx, 4, 2)
    o = np.array([[1.0, 2.0], [10.0, 20.0]])
    pg_n, pg, y = O.combine(o, lay, idx, None, 4, 2)
    assert lay["n_disp"] == 1 and np.array_equal(pg, [[11.0, 22.0]]) and np.array_equal(y, [[11.0, 22.0]])


def test_layer_permutation_equivariance():
    xb, wg, w1, w3, w2 = tiny_problem(T=10)
    logits = O.gate_logits(xb, wg)
    _, _, _, y = O.layer(xb, logits, None, w1, w3, w2, 2, 0)
    perm = np.random.default_rng(1).permutation(10)
    _, _, _, yp = O.layer(xb[perm], logits[perm], None, w1, w3, w2, 2, 0)
    assert np.array_equal(yp, y[perm])


# ---------------------------------------------------------------- workloads
def test_synth_is_seeded_and_shaped():
    cfg = synth.CONFIGS["C1"]
    a, b = synth.make_inputs(cfg), synth.make_inputs(cfg)
    for key in ("x", "w_gate", "w1", "w3", "w2"):
        assert torch.equal(a[key], b[key])
    assert a["x"].shape == (256, 512) and a["w1"].shape == (8, 512, 1024) and a["w2"].shape == (8, 1024, 512)
    assert a["w_gate"].dtype == torch.float32 and a["x"].dtype == torch.bfloat16
    assert abs(a["w1"].float().std().item() - 512 ** -0.5) < 2e-3
    small = synth.CONFIGS["C4"].with_(T=64)
    bias = synth.make_bias(small)
    assert bias.shape == (64, 128) and set(bias.unique().tolist()) == {0.0, 2.0}
    assert torch.all(bias.sum(dim=1) == 2.0 * 16)
    z = synth.make_bias(synth.CONFIGS["C3"])
    assert z.shape == (128,) and z.max().item() == 0.0 and z.min().item() == pytest.approx(-1.1 * math.log(128), rel=1e-6)


def test_config_dedup_statistics_match_closed_form():
    # bias-free configs route uniformly: N_disp / T ~ G (1 - C(E-m,k)/C(E,k))
    for name in ("C1", "C2"):
        cfg = synth.CONFIGS[name].with_(T=2048)
        t = synth.make_routing_inputs(cfg)
        logits = O.gate_logits(synth.bf16_bits(t["x"]), t["w_gate"].numpy())
        idx, _ = O.route(logits, None, cfg.k, cfg.score_fn)
        D = O.distinct_groups_per_token(idx, cfg.E, cfg.G)
        assert D == pytest.approx(closed_form_D(cfg.E, cfg.G, cfg.k), rel=0.03)


def test_payload_efficiency_reproduces_the_papers_printed_pair(golden_dir):
    """Sec. III-A prints one worked example of the packet model: eight targets, explicit addressing, ideal 80 % ->
    69 %.  The oracle must print the same two figures, keep the multimem-style format near the ideal, and obey the
    closed forms of the flit count (hand-computed below, not re-typed from the function)."""
    gold = json.load(open(os.path.join(golden_dir, "paper_payload_efficiency.json")))
    r = O.payload_efficiency(gold["transfer_bytes_of_the_printed_pair"], gold["n_targets"])
    assert round(r["ideal"], gold["printed_digits"]) == gold["ideal"]
    assert round(r["explicit"], gold["printed_digits"]) == gold["explicit"]
    assert r["explicit"] < r["dynamic"] < r["ideal"] and r["ideal"] - r["dynamic"] < 0.01      # "near-ideal"
    # hand count: 1280 B = 80 data flits in 5 packets -> 20 header flits; explicit +16; multimem-style +1
    assert r["data_flits"] == 80 and abs(r["explicit"] - 80 / 116) < 1e-15 and abs(r["dynamic"] - 80 / 101) < 1e-15
    # one target costs one extension flit, nine targets two; a single 16-byte flit still pays a whole header
    assert O.payload_efficiency(256, 1)["dynamic"] == 16 / 21 and O.payload_efficiency(256, 9)["dynamic"] == 16 / 22
    assert O.payload_efficiency(16, 0)["ideal"] == 1 / 5 and O.payload_efficiency(17, 0)["data_flits"] == 2
    # a token vector of the DeepSeek-V3-shaped layer (7168 bf16): the header share vanishes, all three converge
    big = O.payload_efficiency(7168 * 2, 8)
    assert big["ideal"] == 0.8 and abs(big["explicit"] - 896 / 1136) < 1e-15 and big["explicit"] < big["dynamic"] < 0.8
    # efficiency never decreases when targets are removed
    for n in range(1, 33):
        a, b = O.payload_efficiency(640, n), O.payload_efficiency(640, n - 1)
        assert a["explicit"] < b["explicit"] and a["dynamic"] <= b["dynamic"]


# ------------------------------------------------------------------------------------------------ backward
def _rand_expert(rng, n, d, f):
    return (rng.standard_normal((n, d)), rng.standard_normal((d, f)) / np.sqrt(d),
            rng.standard_normal((d, f)) / np.sqrt(d), rng.standard_normal((f, d)) / np.sqrt(f))


def test_expert_backward_against_central_finite_differences():
    """Every entry of da, dW1, dW3, dW2 of a tiny expert against a central difference of the forward (which has its
    own pins): a dropped term, a wrong sign in the derivative of silu or a transposed operand fails it."""
    rng = np.random.default_rng(3)
    a, w1, w3, w2 = _rand_expert(rng, 3, 5, 4)
    do = rng.standard_normal((3, 5))
    da, g1, g3, g2 = O.expert_ffn_rows_backward_f64(a, w1, w3, w2, do)
    loss = lambda a_, w1_, w3_, w2_: float((do * O.expert_ffn_rows_f64(a_, w1_, w3_, w2_)).sum())
    eps = 1e-6
    for arr, grad, pos in ((a, da, 0), (w1, g1, 1), (w3, g3, 2), (w2, g2, 3)):
        num = np.zeros_like(arr)
        for i in np.ndindex(arr.shape):
            args = [a, w1, w3, w2]
            hi, lo = arr.copy(), arr.copy()
            hi[i] += eps
            lo[i] -= eps
            args[pos] = hi
            up = loss(*args)
            args[pos] = lo
            num[i] = (up - loss(*args)) / (2 * eps)
        assert np.abs(num - grad).max() <= 1e-7 * max(1.0, np.abs(grad).max()), pos


def test_expert_backward_against_fp64_autograd():
    """The dense special case (one expert, every row) against torch's fp64 automatic differentiation."""
    rng = np.random.default_rng(4)
    a, w1, w3, w2 = _rand_expert(rng, 7, 12, 9)
    do = rng.standard_normal((7, 12))
    ta, t1, t3, t2 = (torch.tensor(v, dtype=torch.float64, requires_grad=True) for v in (a, w1, w3, w2))
    out = (torch.nn.functional.silu(ta @ t1) * (ta @ t3)) @ t2
    (out * torch.tensor(do)).sum().backward()
    got = O.expert_ffn_rows_backward_f64(a, w1, w3, w2, do)
    for g, t in zip(got, (ta, t1, t3, t2)):
        assert np.abs(g - t.grad.numpy()).max() <= 1e-12 * max(1.0, np.abs(g).max())


def test_layer_backward_is_the_routed_sum_of_expert_gradients():
    """layer_backward on a small routed layer: dx and the weight gradients against a finite difference of the
    oracle's own forward with the routing held fixed (tokens perturbed one coordinate at a time through the dense
    definition), plus the structural facts: experts nobody selected get zero gradients, the result is linear in
    dy, and the gate weight multiplies the expert-level gradient."""
    rng = np.random.default_rng(5)
    T, d, f, E, k = 6, 8, 8, 4, 2
    xb = O.f64_to_bf16_bits(rng.standard_normal((T, d)))
    w1b, w3b, w2b = (O.f64_to_bf16_bits(rng.standard_normal(s) * 0.4) for s in ((E, d, f), (E, d, f), (E, f, d)))
    idx = np.array([[0, 1], [1, 3], [3, 0], [0, 3], [1, 0], [3, 1]], dtype=np.int32)       # expert 2 unused
    w = rng.uniform(0.2, 0.8, size=(T, k))
    dy = rng.standard_normal((T, d))
    dx, grads = O.layer_backward(xb, idx, w, w1b, w3b, w2b, dy)

    def forward(x64):       # dense definition with the routing fixed, float64 tokens
        y = np.zeros((T, d))
        for t in range(T):
            for j in range(k):
                e = idx[t, j]
                y[t] += w[t, j] * O.expert_ffn_rows_f64(x64[t:t + 1], O.bf16_to_f64(w1b[e]), O.bf16_to_f64(w3b[e]),
                                                        O.bf16_to_f64(w2b[e]))[0]
        return y

    x64 = O.bf16_to_f64(xb)
    eps = 1e-6
    num = np.zeros_like(x64)
    for i in np.ndindex(x64.shape):
        hi, lo = x64.copy(), x64.copy()
        hi[i] += eps
        lo[i] -= eps
        num[i] = ((dy * forward(hi)).sum() - (dy * forward(lo)).sum()) / (2 * eps)
    assert np.abs(num - dx).max() <= 1e-6 * max(1.0, np.abs(dx).max())
    # expert 2 was never selected: no entry in the routed result, zeros when asked for explicitly
    assert 2 not in grads
    _, only2 = O.layer_backward(xb, idx, w, w1b, w3b, w2b, dy, experts=[2])
    assert all(not g.any() for g in only2[2])
    # weight gradient of expert 3 = sum over its pairs of w * (expert-level gradient of that row)
    g1 = np.zeros((d, f))
    for t, j in zip(*np.nonzero(idx == 3)):
        _, r1, _, _ = O.expert_ffn_rows_backward_f64(x64[t:t + 1], O.bf16_to_f64(w1b[3]), O.bf16_to_f64(w3b[3]),
                                                     O.bf16_to_f64(w2b[3]), dy[t:t + 1])
        g1 += w[t, j] * r1
    assert np.abs(g1 - grads[3][0]).max() <= 1e-12 * max(1.0, np.abs(g1).max())
    # linear in dy
    dx2, grads2 = O.layer_backward(xb, idx, w, w1b, w3b, w2b, 2.0 * dy)
    assert np.array_equal(dx2, 2.0 * dx) and np.array_equal(grads2[0][2], 2.0 * grads[0][2])


def _gate_case(rng, score_fn, k=3, with_bias=True):
    T, d, f, E = 5, 8, 6, 6
    xb = O.f64_to_bf16_bits(rng.standard_normal((T, d)))
    wg = (rng.standard_normal((d, E)) * 0.3).astype(np.float32)
    bias = (rng.standard_normal((T, E)) * 0.2).astype(np.float32) if with_bias else None
    w1b, w3b, w2b = (O.f64_to_bf16_bits(rng.standard_normal(s) * 0.4) for s in ((E, d, f), (E, d, f), (E, f, d)))
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)     # any fixed selection
    dy = rng.standard_normal((T, d))
    return xb, wg, bias, idx, w1b, w3b, w2b, dy, score_fn


def _gate_forward_loss(x64, wg64, bias, idx, w1b, w3b, w2b, dy, score_fn):
    """L = sum(dy * y) through the oracle's own forward pieces (gate_weights and expert_ffn_rows, each pinned above)
    with the selection fixed; keys in fp64 so that a difference quotient sees the perturbation."""
    keys = x64 @ wg64 + (0.0 if bias is None else bias.astype(np.float64))
    sel = np.take_along_axis(keys, idx.astype(np.int64), axis=1)
    # gate_weights rounds its keys to fp32 first; feed it per-row shifted keys is not possible, so the weights
    # come from the same definition evaluated by torch in fp64 (softmax / sigmoid are library routines there)
    ts = torch.tensor(sel, dtype=torch.float64)
    w = (torch.softmax(ts, dim=1) if score_fn == O.SCORE_SOFTMAX
         else torch.sigmoid(ts) / torch.sigmoid(ts).sum(dim=1, keepdim=True)).numpy()
    total = 0.0
    for t in range(x64.shape[0]):
        for j in range(idx.shape[1]):
            e = idx[t, j]
            o = O.expert_ffn_rows_f64(x64[t:t + 1], O.bf16_to_f64(w1b[e]), O.bf16_to_f64(w3b[e]), O.bf16_to_f64(w2b[e]))[0]
            total += w[t, j] * float(dy[t] @ o)
    return total


@pytest.mark.parametrize("score_fn", [O.SCORE_SOFTMAX, O.SCORE_SIGMOID])
def test_gate_backward_against_central_finite_differences(score_fn):
    """dL/dw_gate (every entry) and the total dL/dx (gate path + expert path) against central differences of the
    forward with the selection held fixed.  A wrong sign or a dropped renormalisation term in the softmax / sigmoid
    derivative, a transposed gate weight, or a gate path missing from dx fails it."""
    xb, wg, bias, idx, w1b, w3b, w2b, dy, _ = _gate_case(np.random.default_rng(11 + score_fn), score_fn)
    x64, wg64 = O.bf16_to_f64(xb), wg.astype(np.float64)
    dwg, dxg, dkey, dw = O.gate_backward(xb, wg, bias, idx, score_fn, w1b, w3b, w2b, dy)
    # the weights the expert path of dx needs: the oracle's own gate_weights on the fp32 keys
    keys32 = (x64 @ wg64 + bias.astype(np.float64)).astype(np.float32)
    w = O.gate_weights(keys32, idx, score_fn)
    dx_exp, _ = O.layer_backward(xb, idx, w, w1b, w3b, w2b, dy)
    loss = lambda x_, wg_: _gate_forward_loss(x_, wg_, bias, idx, w1b, w3b, w2b, dy, score_fn)
    eps = 1e-6
    num = np.zeros_like(wg64)
    for i in np.ndindex(wg64.shape):
        hi, lo = wg64.copy(), wg64.copy()
        hi[i] += eps
        lo[i] -= eps
        num[i] = (loss(x64, hi) - loss(x64, lo)) / (2 * eps)
    assert np.abs(num - dwg).max() <= 1e-6 * max(1.0, np.abs(dwg).max())
    numx = np.zeros_like(x64)
    for i in np.ndindex(x64.shape):
        hi, lo = x64.copy(), x64.copy()
        hi[i] += eps
        lo[i] -= eps
        numx[i] = (loss(hi, wg64) - loss(lo, wg64)) / (2 * eps)
    # gate_weights saw fp32-rounded keys: the expert path carries that 1e-7 relative difference
    assert np.abs(numx - (dx_exp + dxg)).max() <= 1e-5 * max(1.0, np.abs(numx).max())
    assert np.abs(dxg).max() > 1e-3 * np.abs(numx).max()          # the gate path is not negligible in this case


@pytest.mark.parametrize("score_fn", [O.SCORE_SOFTMAX, O.SCORE_SIGMOID])
def test_gate_backward_against_fp64_autograd(score_fn):
    """The same quantities from torch's fp64 automatic differentiation of a dense re-statement of the layer
    (gather of the selected keys, library softmax / sigmoid, matmul experts)."""
    xb, wg, bias, idx, w1b, w3b, w2b, dy, _ = _gate_case(np.random.default_rng(21 + score_fn), score_fn)
    tx = torch.tensor(O.bf16_to_f64(xb), requires_grad=True)
    tg = torch.tensor(wg.astype(np.float64), requires_grad=True)
    keys = tx @ tg + torch.tensor(bias.astype(np.float64))
    sel = torch.gather(keys, 1, torch.tensor(idx.astype(np.int64)))
    w = torch.softmax(sel, 1) if score_fn == O.SCORE_SOFTMAX else torch.sigmoid(sel) / torch.sigmoid(sel).sum(1, keepdim=True)
    w_const = w.detach()
    y_gate = torch.zeros(tx.shape, dtype=torch.float64)      # gradient flows through the weights only
    y_exp = torch.zeros(tx.shape, dtype=torch.float64)       # gradient flows through the experts only
    for t in range(tx.shape[0]):
        for j in range(idx.shape[1]):
            e = int(idx[t, j])
            t1, t3, t2 = (torch.tensor(O.bf16_to_f64(v[e])) for v in (w1b, w3b, w2b))
            ffn = lambda a: (torch.nn.functional.silu(a @ t1) * (a @ t3)) @ t2
            y_gate[t] = y_gate[t] + w[t, j] * ffn(tx[t:t + 1].detach())[0]
            y_exp[t] = y_exp[t] + w_const[t, j] * ffn(tx[t:t + 1])[0]
    tdy = torch.tensor(dy)
    gwg, gx_gate = torch.autograd.grad((y_gate * tdy).sum(), (tg, tx), retain_graph=True)
    dwg, dxg, dkey, dw = O.gate_backward(xb, wg, bias, idx, score_fn, w1b, w3b, w2b, dy)
    assert np.abs(dwg - gwg.numpy()).max() <= 1e-12 * max(1.0, np.abs(dwg).max())
    assert np.abs(dxg - gx_gate.numpy()).max() <= 1e-12 * max(1.0, np.abs(dxg).max())


def test_gate_backward_special_cases():
    """k = 1: the single weight is 1 whatever the key, so nothing reaches the gate.  Softmax: shifting every selected
    key of a token leaves its weights unchanged, so the key gradients of a token sum to zero.  The gate path is linear
    in dy."""
    for score_fn in (O.SCORE_SOFTMAX, O.SCORE_SIGMOID):
        xb, wg, bias, idx, w1b, w3b, w2b, dy, _ = _gate_case(np.random.default_rng(31), score_fn, k=1)
        dwg, dxg, dkey, dw = O.gate_backward(xb, wg, bias, idx, score_fn, w1b, w3b, w2b, dy)
        assert np.abs(dwg).max() <= 1e-15 and np.abs(dxg).max() <= 1e-15 and np.abs(dw).max() > 0.1
    xb, wg, bias, idx, w1b, w3b, w2b, dy, _ = _gate_case(np.random.default_rng(32), O.SCORE_SOFTMAX, k=4, with_bias=False)
    dwg, dxg, dkey, dw = O.gate_backward(xb, wg, bias, idx, O.SCORE_SOFTMAX, w1b, w3b, w2b, dy)
    assert np.abs(dkey.sum(axis=1)).max() <= 1e-14 * np.abs(dkey).max()
    dwg2, dxg2, _, _ = O.gate_backward(xb, wg, bias, idx, O.SCORE_SOFTMAX, w1b, w3b, w2b, 3.0 * dy)
    assert np.allclose(dwg2, 3.0 * dwg, rtol=1e-13, atol=0) and np.allclose(dxg2, 3.0 * dxg, rtol=1e-13, atol=0)


def test_layer_backward_ignores_slots_not_in_use():
    """A slot of topk_idx below 0 contributes nothing: the same result as pointing the slot at any expert with gate
    weight 0 (whose contribution is w * (...) = 0 term by term)."""
    rng = np.random.default_rng(41)
    T, d, f, E, k = 5, 6, 4, 3, 2
    xb = O.f64_to_bf16_bits(rng.standard_normal((T, d)))
    w1b, w3b, w2b = (O.f64_to_bf16_bits(rng.standard_normal(s) * 0.4) for s in ((E, d, f), (E, d, f), (E, f, d)))
    idx = np.array([[0, 1], [1, -1], [2, 0], [-1, -1], [1, 2]], dtype=np.int32)
    w = rng.uniform(0.2, 0.8, size=(T, k))
    dy = rng.standard_normal((T, d))
    dx, grads = O.layer_backward(xb, idx, w, w1b, w3b, w2b, dy)
    idx2, w2 = idx.copy(), w.copy()
    w2[idx < 0] = 0.0
    idx2[idx < 0] = 2
    dx2, grads2 = O.layer_backward(xb, idx2, w2, w1b, w3b, w2b, dy)
    assert np.allclose(dx, dx2, rtol=0, atol=1e-15) and not dx[3].any()
    for e in range(E):
        for a, b in zip(grads[e], grads2[e]):
            assert np.allclose(a, b, rtol=0, atol=1e-15)
