"""Pins of the FP8 (E4M3, W8A8) oracle: format table, conversion against a library and hand-picked ties,
quantisation invariants, a scalar brute-force scaled GEMM, and the distance to the unquantised oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import fp8_oracle as f8, moe_oracle as orc
from paper_2607_23264_b200 import inputs as gen


def test_decode_table_matches_the_format_definition():
    vals = f8.e4m3_decode(np.arange(256, dtype=np.uint8))
    assert vals[0] == 0.0 and vals[0x80] == 0.0 and np.signbit(vals[0x80])
    assert vals[0x01] == 2.0 ** -9 and vals[0x07] == 7 * 2.0 ** -9            # subnormals
    assert vals[0x08] == 2.0 ** -6 and vals[0x38] == 1.0 and vals[0x39] == 1.125
    assert vals[0x7E] == 448.0 and vals[0xFE] == -448.0 and math.isnan(vals[0x7F]) and math.isnan(vals[0xFF])
    pos = vals[:127]
    assert np.all(np.diff(pos) > 0), "codes 0..126 ascend"
    ref = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(np.nan_to_num(vals, nan=-1.0), np.nan_to_num(ref, nan=-1.0)), "library decode"


def test_encode_matches_library_conversion_and_tie_rules():
    rng = np.random.default_rng(0)
    v = np.concatenate([rng.standard_normal(20000) * 50, rng.standard_normal(20000) * 0.01,
                        rng.uniform(-448, 448, 20000), f8.e4m3_decode(np.arange(127, dtype=np.uint8)),
                        [1.0625, 1.1875, 2.0 ** -10, 1.5 * 2.0 ** -9, 447.9, 448.0, -448.0, 0.0]]).astype(np.float32)
    v = v[np.abs(v) <= 448.0]
    got = f8.e4m3_encode(v)
    ref = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    same = (got == ref) | ((got & 0x7F) == 0) & ((ref & 0x7F) == 0)        # signed zeros may differ in sign bit only
    assert same.all()
    # hand-picked ties: to the even code
    assert f8.e4m3_encode(np.float32([1.0625]))[0] == 0x38                  # between 1.0 (0x38) and 1.125 (0x39)
    assert f8.e4m3_encode(np.float32([1.1875]))[0] == 0x3A                  # between 1.125 (0x39) and 1.25 (0x3A)
    assert f8.e4m3_encode(np.float32([2.0 ** -10]))[0] == 0x00              # between 0 and the smallest subnormal
    # saturation (the library would produce NaN there)
    assert f8.e4m3_encode(np.float32([500.0, -1e9, 464.0]))[:].tolist() == [0x7E, 0xFE, 0x7E]
    # round trip of every finite code
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    back = f8.e4m3_encode(f8.e4m3_decode(codes).astype(np.float32))
    assert np.array_equal(back & 0x7F, codes & 0x7F)


def test_quantize_rows_invariants():
    rng = np.random.default_rng(1)
    v = (rng.standard_normal((50, 96)) * rng.uniform(1e-3, 1e3, size=(50, 1))).astype(np.float32)
    v[7] = 0.0
    q, s = f8.quantize_rows(v)
    assert q.dtype == np.uint8 and s.dtype == np.float32
    assert s[7] == 1.0 and not q[7].any(), "an all-zero row keeps scale 1 and zero codes"
    deq = f8.dequantize_rows(q, s)
    for r in range(50):
        if r == 7:
            continue
        assert np.abs(f8.e4m3_decode(q[r])).max() == 448.0, "the largest element maps to the largest code"
        assert s[r] == np.float32(np.abs(v[r]).max()) / np.float32(448.0)
        # |error| <= half a quantum: quantum = 2^(e-3) for a value in [2^e, 2^(e+1)), at least 2^-9, times the scale
        mag = np.maximum(np.abs(v[r].astype(np.float64)) / s[r], 2.0 ** -6)
        half_q = np.exp2(np.floor(np.log2(mag)) - 3) / 2 * s[r]
        assert np.all(np.abs(deq[r] - v[r]) <= half_q * 1.0001 + 1e-12)


def test_scaled_gemm_against_scalar_loops():
    rng = np.random.default_rng(2)
    a = rng.standard_normal((3, 16)).astype(np.float32)
    w = rng.standard_normal((4, 16)).astype(np.float32)
    aq, sa = f8.quantize_rows(a)
    wq, sw = f8.quantize_rows(w)
    got = f8.scaled_gemm(aq, sa, wq, sw)
    av, wv = f8.e4m3_decode(aq).tolist(), f8.e4m3_decode(wq).tolist()
    for r in range(3):
        for c in range(4):
            acc = sum(av[r][k] * wv[c][k] for k in range(16))
            assert got[r, c] == pytest.approx(acc * float(sa[r]) * float(sw[c]), rel=1e-14)
    # the quantised product tracks the exact one within the format's error
    exact = a.astype(np.float64) @ w.astype(np.float64).T
    assert np.linalg.norm(got - exact) / np.linalg.norm(exact) < 0.08


def test_fp8_layer_tracks_the_unquantised_layer():
    cfg = gen.MoEConfig("f8", T=96, H=128, F=192, E=4, k=2, seed=5, router="xWr")
    x = gen.make_x(cfg)
    logits = gen.make_logits(cfg, x)
    W = gen.stacked_weights(cfg, threads=2)
    wf = lambda e: (W[0][e], W[1][e], W[2][e])
    ref = orc.forward(x, logits, cfg.k, wf)
    q = f8.forward_fp8(x, logits, cfg.k, wf)
    for name in ("topk_ids", "counts", "offsets", "perm", "inv_perm"):
        assert np.array_equal(q[name], ref[name]), "routing does not depend on the precision of the experts"
    assert np.array_equal(f8.dequantize_rows(q["xq_perm"], q["sx_perm"]),
                          f8.dequantize_rows(q["xq"], q["sx"])[q["perm"] // cfg.k]), "dispatch moves codes and scales"
    rel = lambda a, b: np.linalg.norm(a - b) / np.linalg.norm(b)
    assert 0.005 < rel(q["h"], ref["h"]) < 0.08, "E4M3 noise: a few percent, not zero and not garbage"
    assert 0.005 < rel(q["out"], ref["out"]) < 0.08
    # bf16 rounding helper: exact on bf16 values, ties to even otherwise
    assert f8.round_to_bf16(np.float64([1.0, 1.00390625, 1.01171875])).tolist() == [1.0, 1.0, 1.015625]
