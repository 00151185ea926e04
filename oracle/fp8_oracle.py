"""CPU oracle for the FP8 form of the expert FFN (GEMM-1 + SwiGLU, GEMM-2).

THIS IS TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the test-suite and the
benchmark's baseline legs may import it.  Plain numpy, one step per function,
no blocking or reordering; it shares no code or table with the CUDA path.

What the paper fixes: Sec. V-A says only that the DeepSeek-V3 experts are
simulated with "FP8 kernels".  Format and scaling are therefore a reading,
the same on both sides:

* element format E4M3 (4 exponent bits, bias 7, 3 mantissa bits; no
  infinities; S.1111.111 is NaN; largest finite value 448; subnormals down to
  2^-9), conversion by round-to-nearest-even with saturation to +-448;
* activations: one fp32 scale per row, scale = fl32(max|row| / 448) (1 for an
  all-zero row), code = e4m3(fl32(value / scale)), both operations in fp32;
* weights: one fp32 scale per (expert, output column), same rule along K;
* GEMMs on the dequantised values, accumulation unrounded here (fp32 on the
  GPU); the product of the two scales is applied to the accumulator;
* h = silu(a1) * a3 is rounded to bf16, then quantised per row like any
  activation before GEMM-2 (the kernel writes h as bf16 and a second pass
  quantises it).

Where floating point decides a code (the scale, the division, the rounding)
the steps above are taken in fp32 exactly as stated, so that the GPU can take
the same decisions.

Pins (tests/test_fp8_oracle_pins.py): the 256 codes against the format's
closed form; encode(decode(c)) = c; ties to even at every midpoint; brute
force nearest-code search on random values; saturation; a row's largest
element always lands on +-448; exactly representable inputs make GEMM-1 /
GEMM-2 equal to the unquantised fp64 FFN.  The scaling recipe itself is this
build's choice: parity of the recipe against the paper is unpinned (the paper
gives none).
"""
from __future__ import annotations

from typing import Dict, Optional, Tuple

import numpy as np

from .moe_oracle import bf16_to_f64, f64_to_bf16_bits

E4M3_MAX = 448.0


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    """uint8 codes -> float64 values (NaN for S.1111.111)."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    exp = (c >> 3) & 0xF
    man = (c & 0x7).astype(np.float64)
    sub = man / 8.0 * 2.0 ** -6
    nor = (1.0 + man / 8.0) * np.exp2((exp - 7).astype(np.float64))
    val = np.where(exp == 0, sub, nor)
    val = np.where((c & 0x7F) == 0x7F, np.nan, val)
    return sign * val


def e4m3_encode(v: np.ndarray) -> np.ndarray:
    """float32 values -> uint8 codes: nearest finite E4M3 value, ties to the
    code with an even mantissa, magnitudes beyond 448 saturate to 448, NaN ->
    0x7F.  Written as a search over the 127 non-negative finite values."""
    v = np.asarray(v, dtype=np.float32)
    table = e4m3_decode(np.arange(0x7F, dtype=np.uint8))          # codes 0 .. 0x7E ascending
    mag = np.abs(v.astype(np.float64))
    hi = np.searchsorted(table, mag, side="left")                   # first code with value >= mag
    hi = np.clip(hi, 0, 0x7E)
    lo = np.clip(hi - 1, 0, 0x7E)
    d_hi = np.abs(table[hi] - mag)
    d_lo = np.abs(mag - table[lo])
    pick_lo = (d_lo < d_hi) | ((d_lo == d_hi) & (lo % 2 == 0))
    code = np.where(pick_lo, lo, hi)
    code = np.where(mag >= E4M3_MAX, 0x7E, code)
    code = np.where(np.isnan(v), 0x7F, code)
    return (code | np.where(np.signbit(v), 0x80, 0)).astype(np.uint8)


def quantize_rows(values: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """[R, C] values (exactly representable in fp32) -> (codes uint8 [R, C],
    scale float32 [R]).  scale = fl32(max|row| / 448), 1 for an all-zero row;
    code = e4m3(fl32(value / scale))."""
    x = np.asarray(values, dtype=np.float32)
    amax = np.max(np.abs(x), axis=1) if x.shape[1] else np.zeros(x.shape[0], np.float32)
    scale = (amax / np.float32(E4M3_MAX)).astype(np.float32)
    scale = np.where(amax == 0, np.float32(1.0), scale).astype(np.float32)
    q = (x / scale[:, None]).astype(np.float32)
    return e4m3_encode(q), scale


def quantize_weights(w: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """[E, K, N] values -> (codes uint8 [E, N, K] (K contiguous), scale float32
    [E, N]): one scale per expert and output column, taken along K."""
    w = np.asarray(w, dtype=np.float32)
    E, K, N = w.shape
    codes = np.zeros((E, N, K), dtype=np.uint8)
    scale = np.zeros((E, N), dtype=np.float32)
    for e in range(E):
        codes[e], scale[e] = quantize_rows(np.ascontiguousarray(w[e].T))
    return codes, scale


def _round_bf16(v: np.ndarray) -> np.ndarray:
    """float64 -> nearest bf16 value (ties to even), returned as float64."""
    return bf16_to_f64(f64_to_bf16_bits(np.asarray(v, dtype=np.float64)))


def gemm1_rows(aq: np.ndarray, sa: np.ndarray, w1q: np.ndarray, s1: np.ndarray, w3q: np.ndarray,
               s3: np.ndarray) -> np.ndarray:
    """GEMM-1 + SwiGLU of one expert on quantised rows: aq uint8 [n, d], sa [n];
    w1q / w3q uint8 [f, d] (K contiguous), s1 / s3 [f].  Returns h float64 [n, f]
    (unrounded)."""
    a = e4m3_decode(aq)
    a1 = (a @ e4m3_decode(w1q).T) * sa.astype(np.float64)[:, None] * s1.astype(np.float64)[None, :]
    a3 = (a @ e4m3_decode(w3q).T) * sa.astype(np.float64)[:, None] * s3.astype(np.float64)[None, :]
    with np.errstate(over="ignore"):   # exp(-a1) -> inf for very negative a1: the quotient is the correct 0
        return a1 / (1.0 + np.exp(-a1)) * a3


def gemm2_rows(hq: np.ndarray, sh: np.ndarray, w2q: np.ndarray, s2: np.ndarray) -> np.ndarray:
    """GEMM-2 of one expert on quantised rows: hq uint8 [n, f], sh [n]; w2q uint8
    [d, f], s2 [d].  Returns o float64 [n, d] (un-weighted)."""
    return (e4m3_decode(hq) @ e4m3_decode(w2q).T) * sh.astype(np.float64)[:, None] * s2.astype(np.float64)[None, :]


def expert_ffn_fp8(xq: np.ndarray, sx: np.ndarray, lay: Dict[str, np.ndarray], topk_w: Optional[np.ndarray],
                   w1q: np.ndarray, s1: np.ndarray, w3q: np.ndarray, s3: np.ndarray, w2q: np.ndarray,
                   s2: np.ndarray, rows: Optional[np.ndarray] = None, return_h: bool = False):
    """FP8 expert FFN in expert-sorted row order.  xq uint8 [rows of the
    dispatched buffer, d] with per-row scales sx; row r of expert e reads
    dispatched row row_src[r].  Steps per expert: GEMM-1 + SwiGLU (fp64 on the
    dequantised operands), h rounded to bf16, h quantised per row, GEMM-2,
    gate weight (if given).  Returns o float64 [P or len(rows), d]."""
    off = lay["expert_offsets"].astype(np.int64)
    P = int(off[-1])
    d = w2q.shape[1]
    want = np.arange(P) if rows is None else np.asarray(rows, dtype=np.int64)
    out = np.zeros((want.size, d), dtype=np.float64)
    hs = np.zeros((want.size, w1q.shape[1]), dtype=np.float64) if return_h else None
    row_e = np.searchsorted(off, want, side="right") - 1
    for e in np.unique(row_e):
        sel = np.nonzero(row_e == e)[0]
        r = want[sel]
        src = lay["row_src"][r].astype(np.int64)
        h = _round_bf16(gemm1_rows(xq[src], sx[src], w1q[e], s1[e], w3q[e], s3[e]))
        hq, sh = quantize_rows(h)
        o = gemm2_rows(hq, sh, w2q[e], s2[e])
        if topk_w is not None:
            o = o * np.asarray(topk_w, dtype=np.float64).reshape(-1)[lay["row_pair"][r].astype(np.int64)][:, None]
        out[sel] = o
        if return_h:
            hs[sel] = h
    return (out, hs) if return_h else out
