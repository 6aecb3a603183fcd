"""Block-scaled FP8 (MXFP8) experts on the GPU against the oracle.

Codes and scale bytes are integer decisions taken in fp32 on both sides: compared bit for bit (x, the weights, the
dispatched rows, and h re-quantised by the oracle from the GPU's own fp32 h).  The GEMMs are compared on identical
quantised operands (fp32 accumulation and bf16 output rounding only), and the whole layer in norm against the fully
independent oracle, where a last-bit difference in h can move an E4M3 code by one step."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as orc
from oracle import mx_oracle as mx
from paper_2607_23264_b200 import binding, inputs as gen
from moe_testlib import DEV, TOL_FRO, TOL_OUT, Layer, assert_out_close, bits_to_dev, dev_bf16_to_f64, rel_fro

pytestmark = pytest.mark.gpu


def words_to_bytes(words: torch.Tensor, rows: int) -> np.ndarray:
    """scale words [K/128][rows] (device) -> scale bytes [rows, K/32] as the oracle orders them."""
    w = words.cpu().numpy().view(np.uint8).reshape(-1, rows, 4)
    return np.ascontiguousarray(w.transpose(1, 0, 2)).reshape(rows, -1)


def bytes_to_words(b: np.ndarray) -> torch.Tensor:
    rows, nb = b.shape
    w = np.ascontiguousarray(b.reshape(rows, nb // 4, 4).transpose(1, 0, 2)).reshape(nb // 4, rows * 4)
    return torch.from_numpy(w.view(np.uint32).reshape(nb // 4, rows).copy().view(np.int32)).to(DEV)


def quantize_on_gpu(ctx, t_bf16: torch.Tensor):
    rows, cols = t_bf16.shape
    codes = torch.full((rows, cols), 0x7F, dtype=torch.uint8, device=DEV)
    words = torch.full((cols // 128, rows), -1, dtype=torch.int32, device=DEV)
    ctx.moe_quantize_rows_mx(t_bf16, rows, cols, codes, words)
    torch.cuda.synchronize()
    return codes, words


class MxLayer:
    def __init__(self, cfg):
        self.cfg = cfg
        self.L = Layer(cfg)
        L, E, F, H = self.L, cfg.E, cfg.F, cfg.H
        self.q = {}
        for name, t, rows, cols in (("gate", L.w_gate, E * F, H), ("up", L.w_up, E * F, H), ("down", L.w_down, E * H, F)):
            self.q[name] = quantize_on_gpu(L.ctx, t.view(rows, cols))

        self._wq = {}

    def oracle_weights(self, e):
        if e not in self._wq:
            self._wq[e] = mx.quantize_weights(*self.L.weights(e))
        return self._wq[e]


def out_from_gpu_codes(ws, lay, tokens, cfg, ids, w, inv_perm, oracle_weights, rows_of_tokens=None):
    """The oracle's Linear-2 and combine run on the GPU's own h codes (read from the fused call's workspace) for the
    given tokens: isolates the arithmetic after h from quantisation decisions that a last-bit difference in h flips."""
    F, H, k = cfg.F, cfg.H, cfg.k
    toks = np.arange(tokens) if isinstance(tokens, int) else np.asarray(tokens)
    n_rows = int(inv_perm.size)
    hq = ws[lay["hq"]:lay["hq"] + n_rows * F].view(n_rows, F)
    sfh = ws[lay["sfh"]:lay["sfh"] + 4 * (F // 128) * n_rows].view(torch.int32).view(F // 128, n_rows)
    rows = inv_perm.reshape(-1, k)[toks].astype(np.int64)
    rows_dev = torch.from_numpy(rows.reshape(-1)).to(DEV)
    codes = hq[rows_dev].cpu().numpy().reshape(len(toks), k, F)
    w8 = sfh[:, rows_dev].cpu().numpy().view(np.uint8).reshape(F // 128, len(toks) * k, 4)
    scales = np.ascontiguousarray(w8.transpose(1, 0, 2)).reshape(len(toks), k, F // 32)
    ref = np.zeros((len(toks), H))
    w_down = {}                                   # expert -> dequantised W_down [H, F], widened once
    for i, t in enumerate(toks):
        for j in range(k):
            e = int(ids[t, j])
            if e not in w_down:
                w_down[e] = mx.dequantize_rows(*oracle_weights(e)[2])
            ref[i] += w[t, j] * (mx.dequantize_rows(codes[i, j:j + 1], scales[i, j:j + 1]) @ w_down[e].T)[0]
    return ref


def small_cfg(T, H, F, E, k, seed, router="xWr"):
    return gen.MoEConfig(name="mx", T=T, H=H, F=F, E=E, k=k, seed=seed, router=router)


@pytest.mark.parametrize("rows,cols", [(1, 128), (37, 256), (300, 1024)])
def test_quantize_rows_mx_bits(rows, cols):
    rng = np.random.default_rng(rows)
    v = (rng.standard_normal((rows, cols)) * np.exp(rng.uniform(-8, 8, (rows, 1)))).astype(np.float32)
    v[0, :32] = 0.0                                               # an all-zero block
    if rows > 2:
        v[2, 32:64] = np.float32(448.0) * np.float32(2.0) ** rng.integers(-5, 5, 32)   # exact boundary values
    bits = gen.f32_to_bf16_bits(v)
    ctx = binding.Context(8, 128, 128, 2, 1)
    codes, words = quantize_on_gpu(ctx, bits_to_dev(bits))
    ref_c, ref_s = mx.quantize_rows(gen.bf16_bits_to_f32(bits))
    assert np.array_equal(codes.cpu().numpy(), ref_c)
    assert np.array_equal(words_to_bytes(words, rows), ref_s)


@pytest.mark.parametrize("T,H,F,E,k,router", [
    (64, 128, 128, 4, 2, "xWr"),        # one K stage per GEMM; one Linear-1 tile of 128 h columns; Linear-2 tile wider than H
    (300, 512, 384, 8, 2, "xWr"),       # several row blocks per expert, ragged tails, whole column tiles
    (129, 256, 640, 16, 4, "xWr_zipf"), # skewed: empty experts, experts of one row
    (5, 384, 256, 6, 6, "xWr"),         # k = E, five rows per expert
    (70, 128, 128, 1024, 32, "xWr"),    # the boundary's largest E and k
])
@pytest.mark.parametrize("swapped", [True, False], ids=["swapped_small_experts", "128_row_tiles_only"])
def test_expert_ffn_mx_parity(T, H, F, E, k, router, swapped, monkeypatch):
    """Experts of at most 64 rows run with swapped operands by default (h quantised with a warp-wide block maximum);
    the development knob switches that off, and both ways must give the oracle's codes and values."""
    if not swapped:
        monkeypatch.setenv("MOE_TUNING", "x.mx_swap_rows=0")
    cfg = small_cfg(T, H, F, E, k, seed=T + H, router=router)
    M = MxLayer(cfg)
    L, ctx = M.L, M.L.ctx
    L.plan()
    ref = mx.forward_mx(L.x_bits, L.logits, k, L.weights)
    R = cfg.R
    # x: quantise and dispatch on the GPU, bit for bit
    xq, sfx = quantize_on_gpu(ctx, L.x)
    assert np.array_equal(xq.cpu().numpy(), ref["xq"]) and np.array_equal(words_to_bytes(sfx, T), ref["sx"])
    xq_perm = torch.full((R, H), 0x7F, dtype=torch.uint8, device=DEV)
    sfx_perm = torch.full((H // 128, R), -1, dtype=torch.int32, device=DEV)
    ctx.moe_dispatch_mx(xq, sfx, L.inv_perm, xq_perm, sfx_perm)
    torch.cuda.synchronize()
    assert np.array_equal(xq_perm.cpu().numpy(), ref["xq_perm"])
    assert np.array_equal(words_to_bytes(sfx_perm, R), ref["sx_perm"])
    # weights: the GPU's codes are the oracle's
    for e in (0, E - 1):
        (gq, gs), (uq, us), (dq, ds) = M.oracle_weights(e)
        assert np.array_equal(M.q["gate"][0][e * F:(e + 1) * F].cpu().numpy(), gq)
        assert np.array_equal(words_to_bytes(M.q["down"][1], E * H)[e * H:(e + 1) * H], ds)
    # the two GEMMs
    hq = torch.full((R, F), 0x7F, dtype=torch.uint8, device=DEV)
    sfh = torch.full((F // 128, R), -1, dtype=torch.int32, device=DEV)
    y = L.nan_bf16(R, H)
    h_dbg = torch.full((R, F), float("nan"), device=DEV)
    ctx.moe_expert_ffn_mx(xq_perm, sfx_perm, L.offsets, *M.q["gate"], *M.q["up"], *M.q["down"], hq, sfh, y, h_dbg)
    torch.cuda.synchronize()
    L.check_device_status()
    h_gpu = h_dbg.cpu().numpy()
    assert np.isfinite(h_gpu).all()
    assert rel_fro(h_gpu.astype(np.float64), ref["h"]) <= TOL_FRO
    # h's codes and scales are the oracle's quantisation of the GPU's own fp32 h
    req_c, req_s = mx.quantize_rows(h_gpu)
    assert np.array_equal(hq.cpu().numpy(), req_c)
    assert np.array_equal(words_to_bytes(sfh, R), req_s)
    # Linear-2 on the GPU's own codes
    y_gpu = dev_bf16_to_f64(y)
    assert np.isfinite(y_gpu).all()
    offsets = L.offsets.cpu().numpy()
    y_ref = np.zeros((R, H))
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi > lo:
            dq, ds = M.oracle_weights(e)[2]
            y_ref[lo:hi] = mx.gemm(req_c[lo:hi], req_s[lo:hi], dq, ds)
    assert rel_fro(y_gpu, y_ref) <= TOL_FRO
    assert_out_close(y_gpu, y_ref, "Linear-2 on the GPU's codes")
    # and against the fully independent oracle, in norm
    assert rel_fro(y_gpu, ref["y_perm"]) <= 2e-2


def test_fused_forward_mx_and_sampled_rows_at_full_k():
    # C2's hidden size with two experts: K loops of 32 and 11 stages (the 4-stage ring wraps many times), 11 column
    # tiles of Linear-1 (1408 = 11 * 128 h columns), 16 of Linear-2 (4096 = 16 * 256)
    cfg = small_cfg(1024, 4096, 1408, 2, 2, seed=9)
    M = MxLayer(cfg)
    L, ctx = M.L, M.L.ctx
    lay = ctx.workspace_layout_mx()
    ws = torch.empty(lay["total"], dtype=torch.uint8, device=DEV)
    out = L.nan_bf16(cfg.T, cfg.H)
    ctx.moe_fused_forward_mx(L.x, L.d_logits, *M.q["gate"], *M.q["up"], *M.q["down"], out, ws)
    torch.cuda.synchronize()
    L.check_device_status()
    assert ctx.moe_last_launch_count() == 8
    out_gpu = dev_bf16_to_f64(out)
    assert np.isfinite(out_gpu).all()
    # oracle on a sample of tokens (rows are independent)
    ids, w = orc.topk_route(L.logits, cfg.k)
    counts, offsets, perm, inv_perm = orc.plan_permutation(ids, cfg.E)
    rng = np.random.default_rng(0)
    toks = np.sort(rng.choice(cfg.T, 48, replace=False))
    xq, sx = mx.quantize_rows(orc.bf16_to_f64(L.x_bits[toks]))
    wq = {e: M.oracle_weights(e) for e in range(cfg.E)}
    ref = np.zeros((len(toks), cfg.H))
    for i, t in enumerate(toks):
        for j in range(cfg.k):
            r = mx.expert_ffn_rows(xq[i:i + 1], sx[i:i + 1], wq[int(ids[t, j])])
            ref[i] += w[t, j] * r["y"][0]
    assert rel_fro(out_gpu[toks], ref) <= 2e-2
    # and element by element against the oracle's Linear-2 + combine of the GPU's own h codes
    own = out_from_gpu_codes(ws, lay, toks, cfg, ids, w, inv_perm, lambda e: wq[e])
    assert_out_close(out_gpu[toks], own, "mx out on the GPU's h codes")
    # the plan in the workspace is the bf16 path's plan
    got_perm = ws[lay["perm"]:lay["perm"] + 4 * cfg.R].view(torch.int32).cpu().numpy()
    assert np.array_equal(got_perm, perm)
    # determinism
    out2 = L.nan_bf16(cfg.T, cfg.H)
    ctx.moe_fused_forward_mx(L.x, L.d_logits, *M.q["gate"], *M.q["up"], *M.q["down"], out2, ws)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))


def test_expert_ffn_mx_random_layers(monkeypatch):
    """The same checks on random layers, with and without swapped-operand tiles for the small experts."""
    rng = np.random.default_rng(14)
    for trial in range(6):
        E = int(rng.integers(1, 5)) if trial % 2 else int(rng.integers(5, 30))
        k = int(rng.integers(1, min(E, 8) + 1))
        monkeypatch.delenv("MOE_TUNING", raising=False)
        test_expert_ffn_mx_parity(int(rng.integers(1, 2500)), 128 * int(rng.integers(1, 5)), 128 * int(rng.integers(1, 6)),
                                  E, k, "xWr_zipf" if trial % 3 == 0 else "xWr", trial % 4 != 3, monkeypatch)


def test_mx_rejects_shapes_it_cannot_tile():
    ctx = binding.Context(16, 192, 128, 2, 1)       # H is not a multiple of 128
    t = torch.zeros(64, dtype=torch.uint8, device=DEV)
    with pytest.raises(binding.MoeError) as e:
        ctx.moe_dispatch_mx(t, t, t, t, t)
    assert e.value.code == 2
    with pytest.raises(binding.MoeError) as e:
        ctx.workspace_layout_mx()
    assert e.value.code == 2
    with pytest.raises(binding.MoeError) as e:
        ctx.moe_quantize_rows_mx(t, 1, 96, t, t)
    assert e.value.code == 1


def test_mx_smaller_batches_on_one_context():
    # a context created for T tokens runs any smaller batch (and an empty one) through the block-scaled path
    cfg = small_cfg(96, 256, 256, 4, 2, seed=21)
    M = MxLayer(cfg)
    L, ctx = M.L, M.L.ctx
    ws = torch.empty(ctx.workspace_layout_mx()["total"], dtype=torch.uint8, device=DEV)
    for tokens in (96, 33, 1, 0):
        ctx.moe_set_active_tokens(tokens)
        out = L.nan_bf16(max(tokens, 1), cfg.H)
        ctx.moe_fused_forward_mx(L.x[:tokens].contiguous() if tokens else L.x, L.d_logits[:tokens].contiguous() if tokens
                                 else L.d_logits, *M.q["gate"], *M.q["up"], *M.q["down"], out, ws)
        torch.cuda.synchronize()
        L.check_device_status()
        if tokens == 0:
            assert ctx.moe_last_launch_count() == 0
            continue
        ref = mx.forward_mx(L.x_bits[:tokens], L.logits[:tokens], cfg.k, L.weights)
        got = dev_bf16_to_f64(out)[:tokens]
        assert np.isfinite(got).all()
        # element by element against the oracle run on the GPU's own h codes; in norm against the independent oracle,
        # from 33 tokens on (over the 256 outputs of a single token one flipped E4M3 code of h is a visible share)
        lay = ctx.workspace_layout_mx()
        own = out_from_gpu_codes(ws, lay, tokens, cfg, ref["topk_ids"], ref["topk_w"], ref["inv_perm"], M.oracle_weights)
        assert_out_close(got, own, f"mx out, {tokens} tokens")
        if tokens >= 33:
            assert rel_fro(got, ref["out"]) <= 2e-2
    ctx.moe_set_active_tokens(cfg.T)
