"""Pins of the block-scaled FP8 (MXFP8) oracle."""
import numpy as np
import pytest

from oracle import fp8_oracle as f8
from oracle import moe_oracle as orc
from oracle import mx_oracle as mx
from paper_2607_23264_b200 import inputs


def test_scale_rule_is_the_smallest_exponent_that_avoids_clipping():
    rng = np.random.default_rng(0)
    mag = np.exp(rng.uniform(np.log(1e-30), np.log(1e30), 4000)).astype(np.float32)
    # exact boundaries too: 448 * 2^j and its neighbours
    edges = np.array([np.ldexp(448.0, j) for j in range(-60, 60)], dtype=np.float32)
    mag = np.concatenate([mag, edges, np.nextafter(edges, np.float32(np.inf)), np.nextafter(edges, np.float32(0))])
    blocks = np.zeros((mag.size, 32), dtype=np.float32)
    blocks[:, 5] = -mag                                   # sign and position do not matter
    e = mx.block_exponents(blocks)[:, 0].astype(np.int64)
    m64 = mag.astype(np.float64)
    assert (np.ldexp(m64, -e) <= 448.0).all()             # no clipping ...
    assert (np.ldexp(m64, -(e - 1)) > 448.0).all()        # ... and no smaller exponent would do


def test_closed_form_blocks():
    one = np.ones((1, 32), dtype=np.float32)
    codes, sc = mx.quantize_rows(one)
    assert int(sc[0, 0]) == 127 - 8                        # 1.0 = 256 * 2^-8
    assert (codes == 0x78).all()                           # E4M3 code of 256: exponent field 15, mantissa 0
    assert np.array_equal(mx.dequantize_rows(codes, sc), one.astype(np.float64))
    for j in (-20, -1, 0, 3, 17):
        top = np.zeros((1, 32), dtype=np.float32)
        top[0, 0] = np.ldexp(448.0, j)
        top[0, 1] = -np.ldexp(1.0, j)
        codes, sc = mx.quantize_rows(top)
        assert int(sc[0, 0]) == 127 + j and codes[0, 0] == 0x7E and codes[0, 1] == 0x80 | 0x38   # 448 and -1
        above = top.copy()
        above[0, 0] = np.nextafter(np.float32(above[0, 0]), np.float32(np.inf))
        codes, sc = mx.quantize_rows(above)
        assert int(sc[0, 0]) == 127 + j + 1 and codes[0, 0] == 0x76                               # 224 after halving
    z = np.zeros((2, 64), dtype=np.float32)
    codes, sc = mx.quantize_rows(z)
    assert (codes == 0).all() and (sc == 0).all()
    tiny = np.full((1, 32), np.float32(1e-45))            # subnormal fp32: exponent clamps at -127
    codes, sc = mx.quantize_rows(tiny)
    assert int(sc[0, 0]) == 0 and np.isfinite(mx.dequantize_rows(codes, sc)).all()
    with pytest.raises(ValueError):
        mx.block_exponents(np.zeros((1, 48), np.float32))


def test_blocks_are_independent_and_nothing_clips():
    rng = np.random.default_rng(1)
    v = (rng.standard_normal((64, 256)) * np.exp(rng.uniform(-6, 6, (64, 1)))).astype(np.float32)
    v[:, 32:64] *= 1000.0                                  # one loud block per row must not disturb the others
    codes, sc = mx.quantize_rows(v)
    dq = mx.dequantize_rows(codes, sc)
    e = sc.astype(np.int64) - 127
    scaled = np.ldexp(v.astype(np.float64), -np.repeat(e, 32, axis=1))
    assert np.abs(scaled).max() <= 448.0
    top = np.abs(scaled).reshape(64, 8, 32).max(axis=2)
    assert (top > 224.0).all()                             # the block maximum uses the top binade
    # E4M3 keeps 3 mantissa bits: relative error at most 2^-4 for values in the normal range of the scaled block
    normal = np.abs(scaled) >= 2.0 ** -6
    assert (np.abs(dq - v)[normal] <= np.abs(v.astype(np.float64))[normal] * 2.0 ** -4).all()
    # quantising one block alone gives the same codes: blocks do not interact
    c2, s2 = mx.quantize_rows(v[:, 96:128])
    assert np.array_equal(c2, codes[:, 96:128]) and np.array_equal(s2[:, 0], sc[:, 3])


def test_gemm_against_scalar_loops():
    rng = np.random.default_rng(2)
    a = rng.standard_normal((3, 64)).astype(np.float32)
    w = rng.standard_normal((4, 64)).astype(np.float32)
    aq, sa = mx.quantize_rows(a)
    wq, sw = mx.quantize_rows(w)
    got = mx.gemm(aq, sa, wq, sw)
    table = f8.e4m3_decode(np.arange(256, dtype=np.uint8))
    for r in range(3):
        for c in range(4):
            acc = 0.0
            for k in range(64):
                acc += (table[aq[r, k]] * 2.0 ** (int(sa[r, k // 32]) - 127)) * (table[wq[c, k]] * 2.0 ** (int(sw[c, k // 32]) - 127))
            assert got[r, c] == pytest.approx(acc, rel=1e-12, abs=1e-12)


def test_forward_mx_stays_close_to_the_unquantised_layer():
    cfg = inputs.random_small_config(np.random.default_rng(4), H=128, F=128, E=4, k=2, T=24)
    xb = inputs.make_x(cfg)
    logits = inputs.make_logits(cfg, xb)
    W = {e: inputs.expert_weights(cfg, e) for e in range(cfg.E)}
    ref = orc.forward(xb, logits, cfg.k, lambda e: W[e])
    got = mx.forward_mx(xb, logits, cfg.k, lambda e: W[e])
    for name in ("topk_ids", "perm", "inv_perm", "offsets"):
        assert np.array_equal(ref[name], got[name])
    rel = np.linalg.norm(got["out"] - ref["out"]) / np.linalg.norm(ref["out"])
    # quantised, but not by much: every operand carries E4M3's rounding (3 mantissa bits, about 3 % rms), which
    # does not average out of a dot product, through two GEMMs and the product silu(gate) * up
    assert 1e-3 < rel < 0.12
    # dispatch moves codes and scales together
    rows_tok = got["perm"] // cfg.k
    assert np.array_equal(got["xq_perm"], got["xq"][rows_tok]) and np.array_equal(got["sx_perm"], got["sx"][rows_tok])
