"""CPU oracle for the FP8 (W8A8) variant of the expert FFN.  TEST INFRASTRUCTURE ONLY.

The paper's kernels run W8A8 / W4A8 (Sec. 5.3); it does not say how values are scaled.  The reading taken here
(the simplest W8A8 that needs no scaling inside the MMA loop):

* storage type E4M3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; largest finite value 448; no
  infinities; subnormals down to 2^-9), conversion = nearest representable value, ties to the even code,
  saturating at +-448;
* one fp32 scale per ROW of every quantised matrix: per token row for activations (x, h), per output channel for
  weights (the rows of W_gate, W_up, W_down).  scale = amax(|row|) / 448 computed in fp32 (1 when the row is all
  zero), code = convert(fp32(value) / scale) with an fp32 division;
* a GEMM multiplies codes and applies both scales afterwards: out[r, c] = (sum_k a[r,k] w[c,k]) s_a[r] s_w[c];
* h is produced in bf16 (as in the bf16 path) and then quantised row by row; y_perm and out stay bf16.

Decisions that produce an integer code are taken in fp32, the precision the kernels use, so that codes can be
compared bit for bit; everything else is fp64.  Pins (tests/test_fp8_oracle.py): the decode table against the
format's closed form, encode against torch's float8_e4m3fn conversion (a library routine) and against hand-picked
ties, quantisation invariants, a scalar brute-force GEMM with scales, and the distance to the unquantised oracle.
"""
from __future__ import annotations

import numpy as np

from oracle import moe_oracle as orc

E4M3_MAX = 448.0


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    """uint8 codes -> fp64 values by the format definition (code 0x7F / 0xFF is NaN)."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    exp = (c >> 3) & 0xF
    man = (c & 0x7).astype(np.float64)
    normal = (1.0 + man / 8.0) * np.exp2(exp.astype(np.float64) - 7.0)
    subnormal = (man / 8.0) * 2.0 ** -6
    val = np.where(exp == 0, subnormal, normal)
    val = np.where((exp == 15) & ((c & 0x7) == 7), np.nan, val)
    return sign * val


_POSITIVE = e4m3_decode(np.arange(0, 127, dtype=np.uint8))     # codes 0..126 ascend in value: 0 .. 448


def e4m3_encode(values: np.ndarray) -> np.ndarray:
    """fp32 values -> uint8 codes: nearest representable, ties to the even code, saturating at +-448."""
    v = np.asarray(values, dtype=np.float32).astype(np.float64)
    mag = np.minimum(np.abs(v), E4M3_MAX)
    hi = np.searchsorted(_POSITIVE, mag, side="left")           # first code with value >= mag
    hi = np.clip(hi, 0, 126)
    lo = np.maximum(hi - 1, 0)
    d_lo = mag - _POSITIVE[lo]
    d_hi = _POSITIVE[hi] - mag
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    code = np.where(pick_hi, hi, lo).astype(np.uint8)
    return np.where(np.signbit(v), code | np.uint8(0x80), code).astype(np.uint8)


def quantize_rows(values: np.ndarray):
    """Row-wise quantisation.  values [rows, cols] (any float dtype holding fp32-representable numbers).
    Returns (codes uint8 [rows, cols], scales fp32 [rows])."""
    v32 = np.asarray(values, dtype=np.float32)
    amax = np.abs(v32).max(axis=1) if v32.shape[1] else np.zeros(v32.shape[0], np.float32)
    scale = np.where(amax > 0, amax / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)
    scaled = (v32 / scale[:, None]).astype(np.float32)          # fp32 division, as the kernel does
    return e4m3_encode(scaled), scale


def dequantize_rows(codes: np.ndarray, scales: np.ndarray) -> np.ndarray:
    return e4m3_decode(codes) * np.asarray(scales, dtype=np.float64)[:, None]


def scaled_gemm(a_codes, a_scales, w_codes, w_scales) -> np.ndarray:
    """out[r, c] = (sum_k a[r,k] w[c,k]) s_a[r] s_w[c] in fp64."""
    acc = e4m3_decode(a_codes) @ e4m3_decode(w_codes).T
    return acc * np.asarray(a_scales, np.float64)[:, None] * np.asarray(w_scales, np.float64)[None, :]


def round_to_bf16(v: np.ndarray) -> np.ndarray:
    """fp64 -> nearest bf16 value (ties to even), returned as fp32.  The rounding goes through fp32 first, as a
    kernel that accumulates in fp32 does."""
    u = np.asarray(v, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def expert_ffn_fp8_rows(xq, sx, wg_bits, wu_bits, wd_bits):
    """One expert on quantised rows.  xq [n,H] codes, sx [n]; weights as bf16 bit patterns (quantised here, per
    output channel).  Returns dict(h (fp64, before the bf16 rounding), h_bf16 (fp32), hq, sh, y (fp64))."""
    wgq, sg = quantize_rows(orc.bf16_to_f64(wg_bits))
    wuq, su = quantize_rows(orc.bf16_to_f64(wu_bits))
    wdq, sd = quantize_rows(orc.bf16_to_f64(wd_bits))
    g = scaled_gemm(xq, sx, wgq, sg)
    u = scaled_gemm(xq, sx, wuq, su)
    h = orc.silu(g) * u
    h_bf16 = round_to_bf16(h)
    hq, sh = quantize_rows(h_bf16)
    y = scaled_gemm(hq, sh, wdq, sd)
    return dict(h=h, h_bf16=h_bf16, hq=hq, sh=sh, y=y)


def forward_fp8(x_bits: np.ndarray, logits: np.ndarray, k: int, weights):
    """Whole layer with the FP8 expert FFN.  Routing, permutation, dispatch and combine are those of the bf16
    layer; x is quantised per token before dispatch.  Returns every intermediate."""
    E = logits.shape[1]
    ids, w = orc.topk_route(logits, k)
    counts, offsets, perm, inv_perm = orc.plan_permutation(ids, E)
    xq, sx = quantize_rows(orc.bf16_to_f64(x_bits))
    rows_tok = np.asarray(perm, dtype=np.int64) // k
    xq_perm, sx_perm = xq[rows_tok], sx[rows_tok]
    R, H = xq_perm.shape
    h = hq = y = None
    sh = np.zeros(R, dtype=np.float32)
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi == lo:
            continue
        r = expert_ffn_fp8_rows(xq_perm[lo:hi], sx_perm[lo:hi], *weights(e))
        if h is None:
            F = r["h"].shape[1]
            h = np.zeros((R, F)); hq = np.zeros((R, F), np.uint8); y = np.zeros((R, H))
        h[lo:hi], hq[lo:hi], sh[lo:hi], y[lo:hi] = r["h"], r["hq"], r["sh"], r["y"]
    out = orc.combine(y, inv_perm, w)
    return dict(topk_ids=ids, topk_w=w, counts=counts, offsets=offsets, perm=perm, inv_perm=inv_perm, xq=xq, sx=sx,
                xq_perm=xq_perm, sx_perm=sx_perm, h=h, hq=hq, sh=sh, y_perm=y, out=out)
