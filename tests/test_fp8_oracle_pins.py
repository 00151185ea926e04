"""Pins of the FP8 oracle against the E4M3 format's definition and the mathematics: none of them
re-types an oracle formula."""
import itertools

import numpy as np
import pytest

from oracle import fp8_oracle as F
from oracle import moe_oracle as O


def test_all_codes_follow_the_format():
    v = F.e4m3_decode(np.arange(256, dtype=np.uint8))
    assert np.isnan(v[0x7F]) and np.isnan(v[0xFF]) and np.isnan(v).sum() == 2     # no infinities, two NaNs
    pos = v[:0x7F]
    assert pos[0] == 0.0 and pos[1] == 2.0 ** -9 and pos[0x7E] == 448.0          # smallest subnormal, largest finite
    assert pos[8] == 2.0 ** -6                                                    # smallest normal
    assert np.all(np.diff(pos) > 0)                                               # strictly increasing in the code
    assert np.array_equal(v[0x80:0xFF], -pos)                                     # sign bit mirrors
    # inside a binade the spacing is 2^(e-3); each binade starts at a power of two
    for e in range(1, 16):
        block = pos[8 * e: 8 * e + 8 if e < 15 else 8 * e + 7]
        assert block[0] == 2.0 ** (e - 7)
        assert np.all(np.diff(block) == 2.0 ** (e - 10))


def test_encode_round_trips_and_breaks_ties_to_even():
    codes = np.concatenate([np.arange(0x7F), np.arange(0x81, 0xFF)]).astype(np.uint8)   # all finite, -0 aside
    vals = F.e4m3_decode(codes).astype(np.float32)
    assert np.array_equal(F.e4m3_encode(vals), codes)
    assert F.e4m3_encode(np.float32([-0.0]))[0] == 0x80
    pos = F.e4m3_decode(np.arange(0x7F, dtype=np.uint8))
    mid = ((pos[:-1] + pos[1:]) / 2).astype(np.float32)          # exactly representable in fp32
    got = F.e4m3_encode(mid)
    want = np.array([c if c % 2 == 0 else c + 1 for c in range(0x7E)], dtype=np.uint8)
    assert np.array_equal(got, want)
    # just off a midpoint goes to the nearer neighbour
    assert np.array_equal(F.e4m3_encode(np.nextafter(mid, np.float32(0))), np.arange(0x7E, dtype=np.uint8))
    assert np.array_equal(F.e4m3_encode(np.nextafter(mid, np.float32(1e9))), np.arange(1, 0x7F, dtype=np.uint8))


def test_encode_is_the_nearest_code_by_brute_force_and_saturates():
    rng = np.random.default_rng(0)
    v = np.concatenate([rng.normal(0, 1, 3000), rng.normal(0, 100, 3000), rng.uniform(-0.01, 0.01, 3000)])
    v = v.astype(np.float32)
    table = F.e4m3_decode(np.arange(256, dtype=np.uint8))
    finite = np.nonzero(~np.isnan(table))[0]
    got = F.e4m3_decode(F.e4m3_encode(v))
    for x, g in zip(v.astype(np.float64), got):
        best = np.min(np.abs(table[finite] - np.clip(x, -448, 448)))
        assert abs(g - np.clip(x, -448, 448)) == best
    big = np.float32([449, 464, 480, 1e6, np.inf, -500, -np.inf])
    assert np.array_equal(F.e4m3_decode(F.e4m3_encode(big)), [448, 448, 448, 448, 448, -448, -448])
    assert F.e4m3_encode(np.float32([np.nan]))[0] & 0x7F == 0x7F


def test_row_quantisation_properties():
    rng = np.random.default_rng(1)
    x = O.bf16_to_f64(O.f64_to_bf16_bits(rng.normal(0, 3, (64, 96))))
    x[5] = 0.0
    q, s = F.quantize_rows(x)
    assert s.dtype == np.float32 and q.dtype == np.uint8
    assert s[5] == 1.0 and not q[5].any()
    deq = F.e4m3_decode(q) * s.astype(np.float64)[:, None]
    amax = np.abs(x).max(axis=1)
    for r in range(64):
        if r == 5:
            continue
        # the largest element of a row lands on +-448
        j = int(np.argmax(np.abs(x[r])))
        assert q[r, j] & 0x7F == 0x7E
        # relative error of normal-range elements <= half a mantissa step (2^-4), tiny ones <= half the subnormal step
        err = np.abs(deq[r] - x[r])
        assert np.all(err <= np.maximum(np.abs(x[r]) * 2.0 ** -4, s[r] * 2.0 ** -10) * (1 + 1e-6))
        assert abs(s[r] - amax[r] / 448.0) <= amax[r] / 448.0 * 2.0 ** -23


def test_weight_quantisation_is_per_expert_and_output_column():
    rng = np.random.default_rng(2)
    w = rng.normal(0, 0.1, (3, 40, 24))
    q, s = F.quantize_weights(w)
    assert q.shape == (3, 24, 40) and s.shape == (3, 24)
    for e, n in itertools.product(range(3), range(24)):
        qq, ss = F.quantize_rows(w[e, :, n][None, :])
        assert np.array_equal(q[e, n], qq[0]) and s[e, n] == ss[0]


def _exact_rows(rng, rows, cols, lo=-3, hi=3):
    """Values k * 2^j with |k| <= 7 and one element of magnitude 448 * 2^(j-6) per row, so that the row
    scale is a power of two and every element is exactly representable in E4M3 after scaling."""
    j = rng.integers(lo, hi, size=rows)
    k = rng.integers(-7, 8, size=(rows, cols)).astype(np.float64)
    x = k * np.exp2(j)[:, None]
    x[np.arange(rows), rng.integers(0, cols, size=rows)] = 448.0 * np.exp2(j - 6)   # = 7 * 2^j: largest, scale 2^(j-6)
    return x


def test_exactly_representable_inputs_reduce_to_the_unquantised_ffn():
    rng = np.random.default_rng(3)
    n, d, f = 9, 32, 24
    a = _exact_rows(rng, n, d)
    w1 = _exact_rows(rng, f, d).T[None]          # [1, d, f]: every output column exact along K
    w3 = _exact_rows(rng, f, d).T[None]
    aq, sa = F.quantize_rows(a)
    w1q, s1 = F.quantize_weights(w1)
    w3q, s3 = F.quantize_weights(w3)
    assert np.array_equal(F.e4m3_decode(aq) * sa[:, None].astype(np.float64), a)
    h = F.gemm1_rows(aq, sa, w1q[0], s1[0], w3q[0], s3[0])
    a1, a3 = a @ w1[0], a @ w3[0]
    with np.errstate(over="ignore"):
        assert np.allclose(h, a1 / (1 + np.exp(-a1)) * a3, rtol=1e-13, atol=0)
    hrows = _exact_rows(rng, n, f)
    w2 = _exact_rows(rng, d, f).T[None]          # [1, f, d]
    hq, sh = F.quantize_rows(hrows)
    w2q, s2 = F.quantize_weights(w2)
    assert np.allclose(F.gemm2_rows(hq, sh, w2q[0], s2[0]), hrows @ w2[0], rtol=1e-13, atol=0)


def test_fp8_ffn_tracks_the_exact_ffn_within_the_format_error():
    """Whole FP8 FFN against the unquantised fp64 FFN of the same bf16 inputs: the error is that of
    3-bit mantissas averaged over the reductions (a few percent), never an order of magnitude."""
    rng = np.random.default_rng(4)
    T, d, f, E, k, G = 96, 64, 48, 4, 2, 2
    xb = O.f64_to_bf16_bits(rng.normal(0, 1, (T, d)))
    w1b = O.f64_to_bf16_bits(rng.normal(0, d ** -0.5, (E, d, f)))
    w3b = O.f64_to_bf16_bits(rng.normal(0, d ** -0.5, (E, d, f)))
    w2b = O.f64_to_bf16_bits(rng.normal(0, f ** -0.5, (E, f, d)))
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    lay = O.layout(idx, E, G)
    xg = O.dispatch(xb, lay)
    ref = O.expert_ffn(xg, lay, None, w1b, w3b, w2b)
    xq, sx = F.quantize_rows(O.bf16_to_f64(xg))
    w1q, s1 = F.quantize_weights(O.bf16_to_f64(w1b))
    w3q, s3 = F.quantize_weights(O.bf16_to_f64(w3b))
    w2q, s2 = F.quantize_weights(O.bf16_to_f64(w2b))
    got = F.expert_ffn_fp8(xq, sx, lay, None, w1q, s1, w3q, s3, w2q, s2)
    rel = np.abs(got - ref).sum() / np.abs(ref).sum()
    assert 5e-3 < rel < 8e-2, rel
    # a subset of rows gives the same rows
    rows = np.array([0, 5, 17, lay["expert_offsets"][2], T * k - 1])
    sub = F.expert_ffn_fp8(xq, sx, lay, None, w1q, s1, w3q, s3, w2q, s2, rows=rows)
    assert np.allclose(sub, got[rows], rtol=1e-12, atol=1e-300)
    # the gate weight multiplies the row
    w = rng.uniform(0.1, 1, (T, k))
    gw = F.expert_ffn_fp8(xq, sx, lay, w, w1q, s1, w3q, s3, w2q, s2)
    assert np.allclose(gw, got * w.reshape(-1)[lay["row_pair"]][:, None], rtol=1e-13)
