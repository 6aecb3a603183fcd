"""Pins of the router oracle: the linear map against a pure-Python loop and closed forms, and the near-tie rule on
hand-made cases.  Also the bound the GPU's arithmetic rests on: two bf16 terms carry an fp32 to 2^-17."""
import numpy as np
import pytest

from oracle import moe_oracle, router_oracle
from paper_2607_23264_b200 import inputs


def _bits(a):
    return inputs.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def test_router_logits_against_triple_loop():
    rng = np.random.default_rng(0)
    T, H, E = 5, 7, 4
    xb = _bits(rng.standard_normal((T, H)))
    w = rng.standard_normal((H, E)).astype(np.float32)
    b = rng.standard_normal(E).astype(np.float32)
    got = router_oracle.router_logits(xb, w, b)
    xf = inputs.bf16_bits_to_f32(xb)
    for t in range(T):
        for e in range(E):
            acc = 0.0
            for c in range(H):
                acc += float(xf[t, c]) * float(w[c, e])
            assert got[t, e] == pytest.approx(acc + float(b[e]), rel=1e-13, abs=1e-13)


def test_router_logits_closed_forms():
    rng = np.random.default_rng(1)
    T, H = 6, 8
    xb = _bits(rng.standard_normal((T, H)))
    xf = inputs.bf16_bits_to_f32(xb).astype(np.float64)
    # identity router: logits are the activations themselves (catches a transposed operand)
    eye = np.eye(H, dtype=np.float32)
    assert np.array_equal(router_oracle.router_logits(xb, eye), xf)
    # a rectangular selector: expert e reads channel 2e (catches swapped H/E roles)
    sel = np.zeros((H, 3), dtype=np.float32)
    for e in range(3):
        sel[2 * e, e] = 1.0
    assert np.array_equal(router_oracle.router_logits(xb, sel), xf[:, [0, 2, 4]])
    # one-hot tokens read rows of W_r
    w = rng.standard_normal((H, 5)).astype(np.float32)
    onehot = _bits(np.eye(H, dtype=np.float32)[:T])
    assert np.array_equal(router_oracle.router_logits(onehot, w), w[:T].astype(np.float64))
    # zero activations leave the bias; the bias is added, not subtracted
    b = np.arange(5, dtype=np.float32)
    assert np.array_equal(router_oracle.router_logits(_bits(np.zeros((T, H))), w, b), np.tile(b.astype(np.float64), (T, 1)))
    with pytest.raises(ValueError):
        router_oracle.router_logits(xb, w.T)


def test_router_logits_match_the_generated_logits():
    # the seeded input recipe rounds the same product to fp32: an independent piece of code, same definition
    cfg = inputs.random_small_config(np.random.default_rng(3), router="xWr_zipf")
    xb = inputs.make_x(cfg)
    ref = inputs.make_logits(cfg, xb)
    got = router_oracle.router_logits(xb, inputs.make_router(cfg), inputs.zipf_log_bias(cfg.E))
    assert np.array_equal(got.astype(np.float32), ref)


def test_admissible_selection_rule():
    l = np.array([[3.0, 1.0, 1.0 + 1e-6, -2.0, 0.5]])
    exact, _ = moe_oracle.topk_route(l, 2)
    assert exact.tolist() == [[0, 2]]
    ok = router_oracle.admissible_selection
    assert ok(l, exact, 0.0).all()                       # the exact answer is admissible at any accuracy
    swapped = np.array([[0, 1]])                         # picks the near-tied neighbour instead
    assert not ok(l, swapped, 1e-7).any()                # 2*eps = 2e-7 < gap 1e-6
    assert ok(l, swapped, 5e-7).all()                    # 2*eps = 1e-6 >= gap
    assert not ok(l, np.array([[0, 4]]), 1e-3).any()     # a clearly smaller logit is never admissible
    assert not ok(l, np.array([[2, 0]]), 1e-3).any()     # wrong slot order
    assert not ok(l, np.array([[0, 0]]), 10.0).any()     # duplicate expert
    assert not ok(l, np.array([[0, 7]]), 10.0).any()     # out of range
    # per-token eps
    l2 = np.vstack([l, l])
    assert ok(l2, np.vstack([swapped, swapped]), np.array([1e-7, 5e-7])).tolist() == [False, True]


def test_perturbed_logits_always_give_admissible_selections():
    # property behind the rule: top-k of logits perturbed by at most eps is admissible at eps
    rng = np.random.default_rng(5)
    for _ in range(20):
        T, E, k = 64, int(rng.integers(2, 40)), 0
        k = int(rng.integers(1, min(E, 8) + 1))
        l = np.round(rng.standard_normal((T, E)), 2)     # coarse values: plenty of exact and near ties
        eps = 0.02
        g = l + rng.uniform(-eps, eps, size=l.shape)
        ids, _ = moe_oracle.topk_route(g, k)
        assert router_oracle.admissible_selection(l, ids, eps).all()


def test_bf16_terms_of_an_fp32():
    # the GPU's router arithmetic: W_r = t1 + t2 (+ t3); two terms leave a relative error below 2^-17, three are exact
    rng = np.random.default_rng(7)
    w = (rng.standard_normal(200000) * np.exp(rng.uniform(-20, 20, 200000))).astype(np.float32)
    t1 = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(w))
    r1 = w - t1
    t2 = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(r1))
    r2 = r1 - t2
    t3 = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(r2))
    w64 = w.astype(np.float64)
    two = t1.astype(np.float64) + t2.astype(np.float64)
    assert (np.abs(two - w64) <= 2.0 ** -17 * np.abs(w64)).all()
    assert np.array_equal(two + t3.astype(np.float64), w64)
    # and the remainders were exact fp32 subtractions
    assert np.array_equal(r1.astype(np.float64), w64 - t1.astype(np.float64))
    assert np.array_equal(r2.astype(np.float64), r1.astype(np.float64) - t2.astype(np.float64))
