"""CPU oracle for the expert-parallel MoE forward at EP=1.  TEST INFRASTRUCTURE ONLY.

Only ``tests/``, ``__graft_entry__.smoke()`` and the ``cpu_baseline`` /
``--impl reference`` legs of ``bench.py`` may import this file.  It shares no
code with the CUDA path and imports nothing from the package; it takes plain
numpy arrays.

What it computes is the plain definition of the layer, in fp64, with no
blocking, fusion or intermediate rounding:

* the EP problem statement (paper Sec. 2.2): every token's hidden vector is
  sent to the experts its router picked (Dispatch), each expert applies its
  feed-forward block, and the expert outputs are returned to the token's owner
  and summed with the router weights (Combine);
* the expert block is two linear layers, "Linear-1" then "Linear-2"
  (Sec. 4.3); Linear-1 produces twice the intermediate width (the
  ``2 h_inter`` of the lead-knee formula, App. A.2), i.e. a gated unit: a gate
  half and an up half, merged as silu(gate) * up;
* routing, placement, dependencies and bytes are those of a standard top-k
  router: the paper changes none of them (Sec. 7, "MoE communication").

Readings taken where the paper is silent (the workload definitions fix them):
top-k picks the k largest logits, ties to the lower expert index, slots in
descending-logit order; the combine weights are a softmax over the k selected
logits; rows of the expert-contiguous buffer are ordered by expert, and inside
an expert by ascending flat slot index t*k+j (a stable counting sort).

Pins (tests/test_oracle_*.py): brute-force triple loops on tiny shapes,
numpy.argsort(kind="stable") / bincount / cumsum for the plan, closed forms
(E=1,k=1 dense FFN; identical experts; scaled down-projections; zero
matrices), invariants (bijection, counts sum to T*k, weights sum to 1) and
row independence.  No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp64 exactly."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


# ----------------------------------------------------------------------------
# S1: routing plan
# ----------------------------------------------------------------------------

def topk_route(logits: np.ndarray, k: int):
    """Top-k expert ids and renormalised softmax weights per token.

    ids[t, j] = expert with the j-th largest logit of token t (ties: lower id);
    w[t, j]   = exp(l_j - m) / sum_j' exp(l_j' - m) over the k selected logits.
    """
    l64 = np.asarray(logits).astype(np.float64)
    T, E = l64.shape
    if not (1 <= k <= E):
        raise ValueError("need 1 <= k <= E")
    # A stable sort of the negated logits lists experts by (descending logit, ascending id).
    order = np.argsort(-l64, axis=1, kind="stable")
    ids = order[:, :k].astype(np.int32)
    sel = np.take_along_axis(l64, ids.astype(np.int64), axis=1)
    m = sel.max(axis=1, keepdims=True) if T else sel
    p = np.exp(sel - m)
    w = p / p.sum(axis=1, keepdims=True)
    return ids, w


def plan_permutation(ids: np.ndarray, E: int):
    """Per-expert counts, exclusive offsets and the stable slot permutation.

    Flat slot s = t*k + j goes to sorted row offsets[e] + (number of earlier
    slots s' < s routed to the same expert e).  perm[row] = s, inv_perm[s] = row.
    """
    flat = np.asarray(ids, dtype=np.int64).reshape(-1)
    R = flat.size
    if R and (flat.min() < 0 or flat.max() >= E):
        raise ValueError("expert id out of range")
    counts = np.zeros(E, dtype=np.int32)
    for e in flat:
        counts[e] += 1
    offsets = np.zeros(E + 1, dtype=np.int32)
    for e in range(E):
        offsets[e + 1] = offsets[e] + counts[e]
    cursor = offsets[:-1].astype(np.int64).copy()
    perm = np.empty(R, dtype=np.int32)
    inv_perm = np.empty(R, dtype=np.int32)
    for s in range(R):
        e = flat[s]
        row = cursor[e]
        cursor[e] += 1
        perm[row] = s
        inv_perm[s] = row
    return counts, offsets, perm, inv_perm


# ----------------------------------------------------------------------------
# S2: dispatch
# ----------------------------------------------------------------------------

def dispatch(x: np.ndarray, perm: np.ndarray, k: int) -> np.ndarray:
    """x_perm[row, :] = x[perm[row] div k, :]  (works on bit patterns or values)."""
    return np.asarray(x)[np.asarray(perm, dtype=np.int64) // k]


# ----------------------------------------------------------------------------
# S3 + S4: expert feed-forward
# ----------------------------------------------------------------------------

def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def expert_ffn_rows(x_rows: np.ndarray, wg: np.ndarray, wu: np.ndarray, wd: np.ndarray):
    """One expert on a block of rows, fp64.  x_rows[n,H]; wg,wu[F,H]; wd[H,F] (fp64 values).

    g = x Wg^T ; u = x Wu^T ; h = silu(g) * u ; y = h Wd^T.   Returns (h[n,F], y[n,H]).
    """
    g = x_rows @ wg.T
    u = x_rows @ wu.T
    h = silu(g) * u
    y = h @ wd.T
    return h, y


def expert_ffn(x_perm_bits: np.ndarray, offsets: np.ndarray, weights):
    """Grouped expert FFN over the expert-contiguous buffer.

    ``weights(e)`` returns expert e's (W_gate[F,H], W_up[F,H], W_down[H,F]) as
    bf16 bit patterns.  Returns (h[R,F], y[R,H]) in fp64, nothing rounded.
    """
    R, H = x_perm_bits.shape
    E = len(offsets) - 1
    h_all = y_all = None
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi == lo:
            continue
        wg, wu, wd = (bf16_to_f64(w) for w in weights(e))
        h, y = expert_ffn_rows(bf16_to_f64(x_perm_bits[lo:hi]), wg, wu, wd)
        if h_all is None:
            h_all = np.zeros((R, h.shape[1]), dtype=np.float64)
            y_all = np.zeros((R, H), dtype=np.float64)
        h_all[lo:hi] = h
        y_all[lo:hi] = y
    if h_all is None:
        F = weights(0)[0].shape[0] if E else 0
        h_all = np.zeros((R, F), dtype=np.float64)
        y_all = np.zeros((R, H), dtype=np.float64)
    return h_all, y_all


# ----------------------------------------------------------------------------
# S5: combine
# ----------------------------------------------------------------------------

def combine(y_perm: np.ndarray, inv_perm: np.ndarray, w: np.ndarray) -> np.ndarray:
    """out[t, :] = sum_j w[t, j] * y_perm[inv_perm[t*k + j], :]   (fp64)."""
    T, k = w.shape
    rows = np.asarray(inv_perm, dtype=np.int64).reshape(T, k)
    out = np.zeros((T, y_perm.shape[1]), dtype=np.float64)
    for j in range(k):
        out += w[:, j:j + 1] * y_perm[rows[:, j]]
    return out


# ----------------------------------------------------------------------------
# S6: whole layer, and the row-sampled form used at full size
# ----------------------------------------------------------------------------

def forward(x_bits: np.ndarray, logits: np.ndarray, k: int, weights):
    """Whole layer.  Returns a dict with every intermediate (indices int32, values fp64)."""
    E = logits.shape[1]
    ids, w = topk_route(logits, k)
    counts, offsets, perm, inv_perm = plan_permutation(ids, E)
    x_perm = dispatch(x_bits, perm, k)
    h, y = expert_ffn(x_perm, offsets, weights)
    out = combine(y, inv_perm, w)
    return dict(topk_ids=ids, topk_w=w, counts=counts, offsets=offsets, perm=perm,
                inv_perm=inv_perm, x_perm=x_perm, h=h, y_perm=y, out=out)


def forward_tokens(tokens, x_bits: np.ndarray, logits: np.ndarray, k: int, weights):
    """The layer's output for a subset of tokens only.

    A token's output depends on its own row of x, its own routing and the
    expert weights, never on other tokens, so this equals the corresponding
    rows of ``forward``.  The routing plan is still computed for all tokens
    (it is cheap), so that ``rows`` are positions in the full sorted buffer.

    Returns dict(tokens, rows[n,k], h[n,k,F], y[n,k,H], out[n,H]) plus the full plan.
    """
    tokens = np.asarray(tokens, dtype=np.int64)
    E = logits.shape[1]
    ids, w = topk_route(logits, k)
    counts, offsets, perm, inv_perm = plan_permutation(ids, E)
    n, H = tokens.size, x_bits.shape[1]
    rows = inv_perm.astype(np.int64).reshape(-1, k)[tokens]
    h_out = y_out = None
    out = np.zeros((n, H), dtype=np.float64)
    x64 = bf16_to_f64(x_bits[tokens])
    sel_ids = ids[tokens]
    for e in np.unique(sel_ids):
        ii, jj = np.nonzero(sel_ids == e)
        wg, wu, wd = (bf16_to_f64(m) for m in weights(int(e)))
        h, y = expert_ffn_rows(x64[ii], wg, wu, wd)
        if h_out is None:
            h_out = np.zeros((n, k, h.shape[1]), dtype=np.float64)
            y_out = np.zeros((n, k, H), dtype=np.float64)
        h_out[ii, jj] = h
        y_out[ii, jj] = y
    for j in range(k):
        if y_out is not None:
            out += w[tokens][:, j:j + 1] * y_out[:, j]
    return dict(tokens=tokens, rows=rows, h=h_out, y=y_out, out=out, topk_ids=ids, topk_w=w,
                counts=counts, offsets=offsets, perm=perm, inv_perm=inv_perm)
