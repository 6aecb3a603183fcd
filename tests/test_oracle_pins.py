"""Pins for the CPU oracle: everything here is independent of oracle/moe_oracle.py's own arithmetic.

The paper prints no worked numbers for the MoE math, so the oracle is tied to
(a) brute-force scalar loops written out index by index, (b) numpy library
routines that the plan reduces to (stable argsort, bincount, cumsum),
(c) closed forms and hand-derived values (tests/golden/), (d) invariants.
Each pin is chosen so that a plausible slip (dropped term, wrong sign or index,
transposed operand, gate/up swapped, weight paired with the wrong expert)
fails at least one of them.
"""
import math
import os

import numpy as np
import pytest

from oracle import moe_oracle as orc
from paper_2607_23264_b200 import inputs as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f32_bits(a):
    return gen.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def bf(a):
    """Values representable in bf16, as python floats."""
    return gen.bf16_bits_to_f32(f32_bits(a)).astype(np.float64)


# ----------------------------------------------------------------------------- brute force twins

def brute_topk(logits, k):
    ids, ws = [], []
    for row in logits:
        row = [float(v) for v in row]
        order = sorted(range(len(row)), key=lambda e: (-row[e], e))[:k]
        m = max(row[e] for e in order)
        p = [math.exp(row[e] - m) for e in order]
        s = sum(p)
        ids.append(order)
        ws.append([v / s for v in p])
    return ids, ws


def brute_plan(ids, E):
    flat = [e for row in ids for e in row]
    counts = [sum(1 for e in flat if e == ex) for ex in range(E)]
    offsets = [0]
    for c in counts:
        offsets.append(offsets[-1] + c)
    perm = []
    for ex in range(E):
        perm.extend(s for s, e in enumerate(flat) if e == ex)
    inv = [0] * len(flat)
    for r, s in enumerate(perm):
        inv[s] = r
    return counts, offsets, perm, inv


def brute_layer(x, logits, k, wg, wu, wd):
    """Whole layer with scalar loops.  x[T][H]; wg,wu[E][F][H]; wd[E][H][F] as python floats."""
    T, H = len(x), len(x[0])
    F = len(wg[0])
    ids, ws = brute_topk(logits, k)
    out = [[0.0] * H for _ in range(T)]
    for t in range(T):
        for j in range(k):
            e = ids[t][j]
            hvec = []
            for f in range(F):
                g = sum(x[t][i] * wg[e][f][i] for i in range(H))
                u = sum(x[t][i] * wu[e][f][i] for i in range(H))
                hvec.append(g / (1.0 + math.exp(-g)) * u)
            for c in range(H):
                y = sum(hvec[f] * wd[e][c][f] for f in range(F))
                out[t][c] += ws[t][j] * y
    return ids, ws, out


# ----------------------------------------------------------------------------- routing

def test_topk_matches_bruteforce_with_ties():
    rng = np.random.default_rng(0)
    for _ in range(50):
        T, E = int(rng.integers(1, 9)), int(rng.integers(1, 10))
        k = int(rng.integers(1, E + 1))
        # few distinct values => many ties
        logits = rng.integers(-2, 3, size=(T, E)).astype(np.float32) * np.float32(0.5)
        ids, w = orc.topk_route(logits, k)
        bids, bw = brute_topk(logits, k)
        assert ids.tolist() == bids
        np.testing.assert_allclose(w, np.array(bw), rtol=0, atol=1e-15)


def test_topk_invariants_random():
    rng = np.random.default_rng(1)
    logits = rng.standard_normal((300, 37)).astype(np.float32)
    k = 5
    ids, w = orc.topk_route(logits, k)
    assert ids.dtype == np.int32 and w.dtype == np.float64
    for t in range(300):
        assert len(set(ids[t])) == k
        sel = logits[t, ids[t]]
        assert np.all(np.diff(sel) <= 0), "slots in descending-logit order"
        rest = np.delete(logits[t], ids[t])
        assert sel.min() >= rest.max()
    np.testing.assert_allclose(w.sum(axis=1), 1.0, atol=1e-12)
    assert np.all(np.diff(w, axis=1) <= 1e-15), "weights non-increasing in slot"
    # shift invariance of the softmax over the selected logits
    ids2, w2 = orc.topk_route(logits + np.float32(8.0), k)
    assert np.array_equal(ids, ids2)
    np.testing.assert_allclose(w, w2, atol=1e-6)  # fp32 shift rounds the logits a little
    # k = 1: weight exactly one
    ids1, w1 = orc.topk_route(logits, 1)
    assert np.all(w1 == 1.0)
    assert np.array_equal(ids1[:, 0], logits.argmax(axis=1))


def test_routing_worked_example_golden():
    """Hand-derived values: see tests/golden/routing_worked_example.txt."""
    rows = []
    with open(os.path.join(GOLDEN, "routing_worked_example.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                rows.append(line)
    assert rows[0].startswith("k=")
    k = int(rows[0][2:])
    cases = rows[1:]
    for case in cases:
        lg, ids_s, w_s = case.split("|")
        logits = np.array([[eval(v, {"ln": math.log}) for v in lg.split(",")]], dtype=np.float64)
        ids, w = orc.topk_route(logits, k)
        assert ids[0].tolist() == [int(v) for v in ids_s.split(",")]
        np.testing.assert_allclose(w[0], [float(v) for v in w_s.split(",")], atol=1e-15)


def test_plan_matches_library_routines_and_bruteforce():
    rng = np.random.default_rng(2)
    for trial in range(30):
        T, E = int(rng.integers(0, 40)), int(rng.integers(1, 9))
        k = int(rng.integers(1, E + 1))
        logits = rng.standard_normal((T, E)).astype(np.float32)
        if trial % 3 == 0 and E > 2:
            logits[:, 1] -= 100.0  # an empty expert when k is small
        ids, _ = orc.topk_route(logits, k)
        counts, offsets, perm, inv = orc.plan_permutation(ids, E)
        flat = ids.reshape(-1)
        assert np.array_equal(counts, np.bincount(flat, minlength=E))
        assert np.array_equal(offsets, np.concatenate([[0], np.cumsum(counts)]))
        assert np.array_equal(perm, np.argsort(flat, kind="stable"))
        assert counts.sum() == T * k and offsets[-1] == T * k
        assert sorted(perm.tolist()) == list(range(T * k)), "bijection"
        assert np.array_equal(inv[perm], np.arange(T * k))
        bc, bo, bp, bi = brute_plan(ids.tolist(), E)
        assert counts.tolist() == bc and offsets.tolist() == bo
        assert perm.tolist() == bp and inv.tolist() == bi
        for e in range(E):  # stable: within an expert, slots ascend
            seg = perm[offsets[e]:offsets[e + 1]]
            assert np.all(np.diff(seg) > 0)
            assert np.all(flat[seg] == e)


def test_plan_rejects_bad_ids():
    with pytest.raises(ValueError):
        orc.plan_permutation(np.array([[0, 3]]), 3)
    with pytest.raises(ValueError):
        orc.topk_route(np.zeros((2, 3), np.float32), 4)


def test_dispatch_is_a_row_gather():
    rng = np.random.default_rng(3)
    T, H, E, k = 17, 8, 5, 3
    x = rng.integers(0, 2**16, size=(T, H)).astype(np.uint16)
    ids, _ = orc.topk_route(rng.standard_normal((T, E)).astype(np.float32), k)
    _, _, perm, inv = orc.plan_permutation(ids, E)
    xp = orc.dispatch(x, perm, k)
    assert xp.dtype == np.uint16 and xp.shape == (T * k, H)
    for t in range(T):
        for j in range(k):
            assert np.array_equal(xp[inv[t * k + j]], x[t])


# ----------------------------------------------------------------------------- expert FFN

def test_silu_known_values():
    # silu(z) = z * sigmoid(z); sigmoid(1) = 0.7310585786300049, sigmoid(-1) = 0.2689414213699951
    np.testing.assert_allclose(orc.silu(np.array([0.0, 1.0, -1.0, 2.0])),
                               [0.0, 0.7310585786300049, -0.2689414213699951, 2 * 0.8807970779778823],
                               atol=1e-15)


def test_ffn_index_roles_with_one_hot_weights():
    """One-hot weights make every operand's index role visible: a transpose or a gate/up swap fails."""
    H, F = 4, 3
    x = np.array([[1.0, 2.0, -1.0, 0.5]])
    wg = np.zeros((F, H)); wu = np.zeros((F, H)); wd = np.zeros((H, F))
    wg[1, 0] = 1.0      # g_1 = x_0 = 1
    wu[1, 1] = 1.0      # u_1 = x_1 = 2
    wg[2, 2] = 1.0      # g_2 = x_2 = -1
    wu[2, 3] = 4.0      # u_2 = 4 x_3 = 2
    wd[3, 1] = 1.0      # y_3 = h_1
    wd[0, 2] = 3.0      # y_0 = 3 h_2
    h, y = orc.expert_ffn_rows(x, wg, wu, wd)
    h1 = 0.7310585786300049 * 2.0            # silu(1) * 2
    h2 = -0.2689414213699951 * 2.0           # silu(-1) * 2
    np.testing.assert_allclose(h[0], [0.0, h1, h2], atol=1e-15)
    np.testing.assert_allclose(y[0], [3 * h2, 0.0, 0.0, h1], atol=1e-15)


def _tiny_layer(seed, T=4, H=8, F=8, E=3, k=2):
    rng = np.random.default_rng(seed)
    x = f32_bits(rng.standard_normal((T, H)))
    logits = rng.standard_normal((T, E)).astype(np.float32)
    wg = f32_bits(rng.standard_normal((E, F, H)) / math.sqrt(H))
    wu = f32_bits(rng.standard_normal((E, F, H)) / math.sqrt(H))
    wd = f32_bits(rng.standard_normal((E, H, F)) / math.sqrt(F))
    return x, logits, wg, wu, wd


def test_whole_layer_matches_scalar_bruteforce():
    for seed in range(3):
        T, H, F, E, k = 4, 8, 8, 3, 2
        x, logits, wg, wu, wd = _tiny_layer(seed, T, H, F, E, k)
        res = orc.forward(x, logits, k, lambda e: (wg[e], wu[e], wd[e]))
        val = lambda b: gen.bf16_bits_to_f32(b).astype(np.float64).tolist()
        ids, ws, out = brute_layer(val(x), logits.tolist(), k, val(wg), val(wu), val(wd))
        assert res["topk_ids"].tolist() == ids
        np.testing.assert_allclose(res["topk_w"], ws, atol=1e-15)
        np.testing.assert_allclose(res["out"], out, rtol=1e-12, atol=1e-12)


def test_single_expert_k1_is_a_dense_ffn():
    """E=1, k=1: the layer is out = (silu(x Wg^T) * (x Wu^T)) Wd^T with weight 1; checked with einsum
    over explicit index letters (not the oracle's matmul calls)."""
    rng = np.random.default_rng(5)
    T, H, F = 9, 16, 24
    x = f32_bits(rng.standard_normal((T, H)))
    wg = f32_bits(rng.standard_normal((1, F, H)) / 4)
    wu = f32_bits(rng.standard_normal((1, F, H)) / 4)
    wd = f32_bits(rng.standard_normal((1, H, F)) / 5)
    res = orc.forward(x, np.zeros((T, 1), np.float32), 1, lambda e: (wg[e], wu[e], wd[e]))
    X, G, U, D = (gen.bf16_bits_to_f32(a).astype(np.float64) for a in (x, wg[0], wu[0], wd[0]))
    g = np.einsum("th,fh->tf", X, G)
    u = np.einsum("th,fh->tf", X, U)
    ref = np.einsum("tf,cf->tc", g / (1 + np.exp(-g)) * u, D)
    np.testing.assert_allclose(res["out"], ref, rtol=1e-12, atol=1e-13)
    assert np.all(res["topk_w"] == 1.0)
    assert np.array_equal(res["perm"], np.arange(T))


def test_zero_matrices_give_zero():
    x, logits, wg, wu, wd = _tiny_layer(7)
    z = np.zeros_like
    w = lambda g, u, d: (lambda e: (g[e], u[e], d[e]))
    assert np.all(orc.forward(x, logits, 2, w(wg, wu, z(wd)))["out"] == 0)
    assert np.all(orc.forward(x, logits, 2, w(z(wg), wu, wd))["out"] == 0), "silu(0) = 0"
    assert np.all(orc.forward(x, logits, 2, w(wg, z(wu), wd))["out"] == 0)


def test_identical_experts_make_routing_irrelevant():
    """All experts share weights => out[t] = FFN(x_t) whatever the routing, since weights sum to 1."""
    rng = np.random.default_rng(8)
    T, H, F, E, k = 12, 16, 16, 6, 3
    x, logits, wg, wu, wd = _tiny_layer(8, T, H, F, E, k)
    same = lambda e: (wg[0], wu[0], wd[0])
    res = orc.forward(x, logits, k, same)
    _, y = orc.expert_ffn_rows(orc.bf16_to_f64(x), *(orc.bf16_to_f64(m) for m in same(0)))
    np.testing.assert_allclose(res["out"], y, rtol=1e-12, atol=1e-12)
    res2 = orc.forward(x, rng.standard_normal((T, E)).astype(np.float32), k, same)
    np.testing.assert_allclose(res2["out"], res["out"], rtol=1e-12, atol=1e-12)


def test_scaled_down_projection_exposes_weight_expert_pairing():
    """W_down[e] = c_e W_down[0], shared gate/up => out[t] = (sum_j w_tj c_{e_tj}) FFN_0(x_t).
    A combine that pairs weights with the wrong slot/expert changes the scalar."""
    T, H, F, E, k = 10, 16, 16, 5, 3
    x, logits, wg, wu, wd = _tiny_layer(9, T, H, F, E, k)
    c = np.array([1.0, 2.0, -0.5, 4.0, 0.25])          # exact in bf16, products stay exact
    base = gen.bf16_bits_to_f32(wd[0]).astype(np.float64)
    wd_scaled = [f32_bits(c[e] * base) for e in range(E)]
    res = orc.forward(x, logits, k, lambda e: (wg[0], wu[0], wd_scaled[e]))
    _, y0 = orc.expert_ffn_rows(orc.bf16_to_f64(x), orc.bf16_to_f64(wg[0]), orc.bf16_to_f64(wu[0]), base)
    ids, ws = brute_topk(logits, k)
    scal = np.array([sum(ws[t][j] * c[ids[t][j]] for j in range(k)) for t in range(T)])
    np.testing.assert_allclose(res["out"], scal[:, None] * y0, rtol=1e-12, atol=1e-12)


def test_k1_output_is_the_chosen_expert():
    T, H, F, E = 8, 8, 16, 4
    x, logits, wg, wu, wd = _tiny_layer(10, T, H, F, E, 1)
    res = orc.forward(x, logits, 1, lambda e: (wg[e], wu[e], wd[e]))
    for t in range(T):
        e = int(np.argmax(logits[t]))
        _, y = orc.expert_ffn_rows(orc.bf16_to_f64(x[t:t + 1]), *(orc.bf16_to_f64(m[e]) for m in (wg, wu, wd)))
        np.testing.assert_allclose(res["out"][t], y[0], rtol=1e-12, atol=1e-13)


def test_combine_closed_form():
    """y rows = row index broadcast, weights given: out[t] = sum_j w_tj * inv_perm[t*k+j]."""
    T, k, H = 5, 3, 4
    inv = np.random.default_rng(11).permutation(T * k).astype(np.int32)
    y = np.repeat(np.arange(T * k, dtype=np.float64)[:, None], H, axis=1)
    w = np.random.default_rng(12).random((T, k))
    out = orc.combine(y, inv, w)
    for t in range(T):
        exp = sum(w[t, j] * float(inv[t * k + j]) for j in range(k))
        np.testing.assert_allclose(out[t], exp, rtol=1e-14)


def test_row_independence_justifies_sampled_oracle():
    cfg = gen.MoEConfig("t", T=40, H=64, F=128, E=6, k=2, seed=21, router="xWr")
    x = gen.make_x(cfg)
    logits = gen.make_logits(cfg, x)
    W = gen.stacked_weights(cfg, threads=2)
    wf = lambda e: (W[0][e], W[1][e], W[2][e])
    full = orc.forward(x, logits, cfg.k, wf)
    toks = np.array([3, 0, 39, 17])
    part = orc.forward_tokens(toks, x, logits, cfg.k, wf)
    np.testing.assert_allclose(part["out"], full["out"][toks], rtol=1e-12, atol=1e-12)
    for i, t in enumerate(toks):
        for j in range(cfg.k):
            r = part["rows"][i, j]
            assert r == full["inv_perm"][t * cfg.k + j]
            np.testing.assert_allclose(part["h"][i, j], full["h"][r], rtol=1e-12, atol=1e-12)
            np.testing.assert_allclose(part["y"][i, j], full["y_perm"][r], rtol=1e-12, atol=1e-12)


def test_config_c1_full_oracle_invariants():
    cfg = gen.CONFIGS["C1"]
    x = gen.make_x(cfg)
    logits = gen.make_logits(cfg, x)
    W = gen.stacked_weights(cfg, threads=2)
    res = orc.forward(x, logits, cfg.k, lambda e: (W[0][e], W[1][e], W[2][e]))
    assert res["counts"].sum() == cfg.R
    assert res["out"].shape == (cfg.T, cfg.H) and np.isfinite(res["out"]).all()
    # activations of order one, as the std = 1/sqrt(fan_in) reading intends
    assert 0.2 < res["out"].std() < 2.0
