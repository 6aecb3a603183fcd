"""CPU oracle for the block-scaled FP8 (MXFP8) variant of the expert FFN.  TEST INFRASTRUCTURE ONLY.

The paper's kernels run W8A8 / W4A8 (Sec. 5.3) without saying how values are scaled.  This is the block-scaled
reading: the microscaling layout the Blackwell tensor pipe applies inside the MMA (scales never touch the CUDA cores).

* Elements: E4M3 codes (see ``fp8_oracle``: nearest, ties to the even code, saturating at +-448).
* Blocks: 32 consecutive elements along the contraction dimension K of a row share one scale 2^e, stored as a
  biased byte e + 127 (E8M0; 255 is never produced).  Token rows of x and h are cut along H resp. F; weight rows
  (output channels of W_gate, W_up, W_down) along their own K.
* Scale rule: e is the smallest integer with amax / 2^e <= 448, clamped to [-127, 127], where amax is the largest
  magnitude of the block in fp32; an all-zero block takes e = -127.  No element is ever clipped, and the largest one
  lands in (224, 448].  On fp32 bits this is e = q - 8 + [mantissa field > 0x600000] with q the unbiased exponent of
  amax (448 = 1.75 * 2^8), an integer decision both sides can take identically.
* code = convert(value * 2^-e): the scaling is exact (a power of two), so the only rounding is the E4M3 conversion.
* A GEMM is the plain product of the dequantised operands, out[r, c] = sum_k (a[r,k] 2^ea[r,k/32]) (w[c,k] 2^ew[c,k/32]);
  fp64 here.
* h = silu(gate) * up is quantised from its fp32 value (the GEMM's accumulator precision); y_perm and out are bf16
  on the GPU, fp64 here.

Pins (tests/test_mx_oracle.py): the scale rule against its definition (smallest e with amax 2^-e <= 448) by search,
closed-form blocks (powers of two, 448 * 2^j, just above it, zeros), no clipping and the E4M3 error bound on random
data, a scalar brute-force GEMM, and the distance to the unquantised oracle.
"""
from __future__ import annotations

import numpy as np

from oracle import fp8_oracle as f8
from oracle import moe_oracle as orc

BLOCK = 32


def block_exponents(v32: np.ndarray) -> np.ndarray:
    """Shared exponents e (int32) of the 32-element blocks along the last axis of fp32 values [rows, K]."""
    v32 = np.asarray(v32, dtype=np.float32)
    rows, K = v32.shape
    if K % BLOCK:
        raise ValueError("K must be a multiple of 32")
    amax = np.abs(v32).reshape(rows, K // BLOCK, BLOCK).max(axis=2)
    bits = amax.astype(np.float32).view(np.uint32).astype(np.int64)
    q = ((bits >> 23) & 0xFF) - 127                      # subnormal amax: exponent field 0 -> q = -127, clamped below
    e = q - 8 + ((bits & 0x7FFFFF) > 0x600000)
    return np.clip(e, -127, 127).astype(np.int32)


def quantize_rows(values: np.ndarray):
    """values [rows, K] (numbers exactly representable in fp32) -> (codes uint8 [rows, K], scale bytes uint8
    [rows, K/32] holding e + 127)."""
    v32 = np.asarray(values, dtype=np.float32)
    e = block_exponents(v32)
    scaled = np.ldexp(v32.astype(np.float64), -np.repeat(e, BLOCK, axis=1))      # exact
    return f8.e4m3_encode(scaled.astype(np.float32)), (e + 127).astype(np.uint8)


def dequantize_rows(codes: np.ndarray, scale_bytes: np.ndarray) -> np.ndarray:
    e = np.asarray(scale_bytes, dtype=np.int64) - 127
    return np.ldexp(f8.e4m3_decode(codes), np.repeat(e, BLOCK, axis=1))


def gemm(a_codes, a_scales, w_codes, w_scales) -> np.ndarray:
    """out[r, c] = sum_k dequant(a)[r, k] * dequant(w)[c, k] in fp64."""
    return dequantize_rows(a_codes, a_scales) @ dequantize_rows(w_codes, w_scales).T


def quantize_weights(wg_bits, wu_bits, wd_bits):
    """bf16 bit patterns of one expert's matrices -> ((codes, scales) for gate, up, down), rows = output channels."""
    return tuple(quantize_rows(orc.bf16_to_f64(b)) for b in (wg_bits, wu_bits, wd_bits))


def expert_ffn_rows(xq, sx, wq):
    """One expert on quantised rows.  xq [n,H] codes, sx [n,H/32]; wq from quantize_weights.
    Returns dict(h (fp64), hq, sh (h quantised from its fp32 value), y (fp64))."""
    (gq, gs), (uq, us), (dq, ds) = wq
    g = gemm(xq, sx, gq, gs)
    u = gemm(xq, sx, uq, us)
    h = orc.silu(g) * u
    hq, sh = quantize_rows(h.astype(np.float32))
    y = gemm(hq, sh, dq, ds)
    return dict(h=h, hq=hq, sh=sh, y=y)


def forward_mx(x_bits: np.ndarray, logits: np.ndarray, k: int, weights):
    """Whole layer with the block-scaled expert FFN.  Routing, permutation, dispatch and combine are those of the
    bf16 layer; x is quantised per token before dispatch.  `weights(e)` returns the bf16 bit patterns of expert e."""
    E = logits.shape[1]
    ids, w = orc.topk_route(logits, k)
    counts, offsets, perm, inv_perm = orc.plan_permutation(ids, E)
    xq, sx = quantize_rows(orc.bf16_to_f64(x_bits))
    rows_tok = np.asarray(perm, dtype=np.int64) // k
    xq_perm, sx_perm = xq[rows_tok], sx[rows_tok]
    R, H = xq_perm.shape
    h = hq = sh = y = None
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi == lo:
            continue
        r = expert_ffn_rows(xq_perm[lo:hi], sx_perm[lo:hi], quantize_weights(*weights(e)))
        if h is None:
            F = r["h"].shape[1]
            h = np.zeros((R, F)); hq = np.zeros((R, F), np.uint8); sh = np.zeros((R, F // BLOCK), np.uint8)
            y = np.zeros((R, H))
        h[lo:hi], hq[lo:hi], sh[lo:hi], y[lo:hi] = r["h"], r["hq"], r["sh"], r["y"]
    out = orc.combine(y, inv_perm, w)
    return dict(topk_ids=ids, topk_w=w, counts=counts, offsets=offsets, perm=perm, inv_perm=inv_perm, xq=xq, sx=sx,
                xq_perm=xq_perm, sx_perm=sx_perm, h=h, hq=hq, sh=sh, y_perm=y, out=out)
