"""CPU oracle for the router front end.  TEST INFRASTRUCTURE ONLY.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU legs of ``bench.py``
may import this file.  It shares no code with the CUDA path and imports
nothing from the package.

The paper keeps the router of a standard top-k MoE layer as it is (Sec. 7:
routing, placement, dependencies and bytes are unchanged) and prints no
formula for it; the workload definitions fix it as a linear map of the
token's hidden vector, optionally with a per-expert bias:

    logits[t, e] = sum_c x[t, c] * W_r[c, e]  (+ bias[e])

computed here in fp64 from the exact values of the bf16 activations and the
fp32 router matrix.  The top-k rule that follows is ``moe_oracle.topk_route``.

A GPU that computes the logits in fp32 can legitimately pick another expert
where two logits are closer than its rounding error.  ``admissible_selection``
states the rule the parity tests apply: if every computed logit is within eps
of the exact one, the j-th largest computed value is within eps of the j-th
largest exact value (order statistics are 1-Lipschitz in the sup norm), hence
the exact logit of the expert picked for slot j lies within 2*eps of the exact
j-th largest logit.  A selection that breaks this cannot come from logits that
accurate.

Pins (tests/test_router_oracle.py): a pure-Python triple loop on tiny shapes,
closed forms (identity router, one-hot tokens, zero activations leave the
bias), and hand-made near-tie cases for the admissibility rule.
"""
from __future__ import annotations

import numpy as np


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp64 exactly."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def router_logits(x_bits: np.ndarray, w_router: np.ndarray, bias=None) -> np.ndarray:
    """logits[T,E] in fp64 from x[T,H] (bf16 bits) and W_r[H,E] (fp32), plus bias[E] if given."""
    x = bf16_to_f64(x_bits)
    w = np.asarray(w_router).astype(np.float64)
    if x.ndim != 2 or w.ndim != 2 or x.shape[1] != w.shape[0]:
        raise ValueError("need x[T,H] and W_r[H,E]")
    logits = x @ w
    if bias is not None:
        b = np.asarray(bias).astype(np.float64)
        if b.shape != (w.shape[1],):
            raise ValueError("need bias[E]")
        logits = logits + b[None, :]
    return logits


def admissible_selection(logits64: np.ndarray, ids: np.ndarray, eps) -> np.ndarray:
    """Per token: could `ids` be the ordered top-k of logits that are within eps of `logits64`?

    ids[T,k] must hold distinct experts per token; slot j must satisfy
    |logits64[t, ids[t,j]] - (j-th largest of logits64[t])| <= 2*eps[t].  `eps` is a scalar or one value per
    token.  Returns a boolean array [T].
    """
    l64 = np.asarray(logits64, dtype=np.float64)
    ids = np.asarray(ids, dtype=np.int64)
    T, k = ids.shape
    eps = np.broadcast_to(np.asarray(eps, dtype=np.float64), (T,))
    ok = np.ones(T, dtype=bool)
    ranked = -np.sort(-l64, axis=1)[:, :k]                      # exact order statistics, descending
    picked = np.take_along_axis(l64, np.clip(ids, 0, l64.shape[1] - 1), axis=1)
    ok &= (np.abs(picked - ranked) <= 2.0 * eps[:, None]).all(axis=1)
    srt = np.sort(ids, axis=1)
    ok &= (srt[:, 1:] != srt[:, :-1]).all(axis=1) if k > 1 else True
    ok &= ((ids >= 0) & (ids < l64.shape[1])).all(axis=1)
    return ok
