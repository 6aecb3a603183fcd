"""GPU parity of the two FP8 variants (per-row scales, block scales) at the full workload sizes, in the launch
configuration bench.py times (CTA pairs at 2048 rows per expert on C2; 256 experts with swapped-operand tiles and
empty experts on C3; K = 14336 and K = 7168 mainloops).

Same decomposition as the small-shape tests: every decision that produces a code or a scale is compared bit for
bit, each GEMM is compared with the oracle run on identical quantised operands (the GPU's own h codes for
Linear-2), and the layer output with the oracle's combine of those rows.  What makes it affordable is sampling in
both directions: rows stratified over every 128-row block of the chosen experts (so every tile class is hit) and,
per row, output columns stratified over every 128-column block of both GEMMs; the oracle then only has to quantise
the weight rows of those columns.  The end-to-end norm against the fully independent oracle (its own h, its own
codes) needs whole weight matrices and stays with the small-shape tests."""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

from oracle import fp8_oracle as f8, moe_oracle as orc, mx_oracle as mx
from paper_2607_23264_b200 import inputs as gen
from moe_testlib import DEV, TOL_FRO, Layer, assert_out_close, assert_rows_close, dev_bf16_to_f64

pytestmark = pytest.mark.gpu


def block_columns(n, rng, block=128):
    """First, last and one seeded-random column of every `block`-wide slice of range(n)."""
    cols = []
    for b0 in range(0, n, block):
        b1 = min(b0 + block, n)
        cols += [b0, b1 - 1, int(rng.integers(b0, b1))]
    return np.unique(np.array(cols, dtype=np.int64))


class Sample:
    """Oracle plan, chosen experts, stratified rows and columns, and the tokens whose output is checked."""

    def __init__(self, cfg, n_out_tokens, n_extra_experts):
        self.cfg = cfg
        rng = np.random.default_rng(cfg.seed + 500)
        self.x_bits = gen.make_x(cfg)
        self.logits = gen.make_logits(cfg, self.x_bits)
        self.ids, self.w = orc.topk_route(self.logits, cfg.k)
        self.counts, self.offsets, self.perm, self.inv_perm = orc.plan_permutation(self.ids, cfg.E)
        self.out_tokens = np.sort(rng.choice(cfg.T, size=n_out_tokens, replace=False))
        nonempty = np.flatnonzero(self.counts > 0)
        if cfg.E <= 16:
            chosen = set(nonempty.tolist())
        else:   # the experts of the output tokens, the largest ones, and a seeded pick of the others
            chosen = set(self.ids[self.out_tokens].reshape(-1).tolist())
            chosen.update(nonempty[np.argsort(-self.counts[nonempty], kind="stable")[:4]].tolist())
            chosen.update(rng.permutation(nonempty)[:n_extra_experts].tolist())
        self.experts = sorted(chosen)
        rows = set(self.inv_perm.reshape(cfg.T, cfg.k)[self.out_tokens].reshape(-1).tolist())
        for e in self.experts:                       # every 128-row block of a chosen expert, its first and last row
            lo, hi = int(self.offsets[e]), int(self.offsets[e + 1])
            rows.update([lo, hi - 1])
            rows.update(int(rng.integers(b0, min(b0 + 128, hi))) for b0 in range(lo, hi, 128))
        self.rows = np.array(sorted(rows), dtype=np.int64)
        self.row_expert = np.searchsorted(self.offsets, self.rows, side="right") - 1
        self.row_token = self.perm[self.rows].astype(np.int64) // cfg.k
        assert set(self.row_expert.tolist()) <= chosen
        self.h_cols = block_columns(cfg.F, rng)      # Linear-1 tiles are 128 h columns wide
        self.y_cols = block_columns(cfg.H, rng)      # Linear-2 tiles are two 128-row weight boxes wide

    def rows_of(self, e):
        return np.flatnonzero(self.row_expert == e)

    def out_reference(self, y_ref):
        """The oracle's combine over the sampled columns: y_ref[i] is row self.rows[i] on self.y_cols."""
        pos = {int(r): i for i, r in enumerate(self.rows)}
        ref = np.zeros((len(self.out_tokens), len(self.y_cols)))
        for n, t in enumerate(self.out_tokens):
            for j in range(self.cfg.k):
                ref[n] += self.w[t, j] * y_ref[pos[int(self.inv_perm[t * self.cfg.k + j])]]
        return ref


def gather_rows(t2d, rows):
    return t2d[torch.from_numpy(rows).to(DEV)].cpu().numpy()


def check_plan(S, ws, lay):
    R, cfg = S.cfg.R, S.cfg

    def sl(name, count, dtype):
        nbytes = count * torch.empty((), dtype=dtype).element_size()
        return ws[lay[name]:lay[name] + nbytes].view(dtype)

    for name, ref, count in (("topk_ids", S.ids, R), ("counts", S.counts, cfg.E), ("offsets", S.offsets, cfg.E + 1),
                             ("perm", S.perm, R), ("inv_perm", S.inv_perm, R)):
        assert np.array_equal(sl(name, count, torch.int32).cpu().numpy(), np.asarray(ref).reshape(-1)), name
    return sl


FP8_CASES = [("C2", 24, 0), ("C3", 6, 12)]


@pytest.mark.parametrize("name,n_out,n_extra", FP8_CASES, ids=[c[0] for c in FP8_CASES])
def test_fused_forward_fp8_full_size_sampled(name, n_out, n_extra):
    cfg = gen.CONFIGS[name]
    S = Sample(cfg, n_out, n_extra)
    L = Layer(cfg, keep_experts=set(S.experts), x_bits=S.x_bits, logits=S.logits)
    ctx = L.ctx
    wq = {}
    for wname, w in (("gate", L.w_gate), ("up", L.w_up), ("down", L.w_down)):
        E, r, c = w.shape
        codes = torch.empty((E * r, c), dtype=torch.uint8, device=DEV)
        scales = torch.empty((E * r,), dtype=torch.float32, device=DEV)
        ctx.moe_quantize_rows(w.view(E * r, c), E * r, c, codes, scales)
        wq[wname] = (codes, scales)
    torch.cuda.synchronize()
    del L.w_gate, L.w_up, L.w_down
    lay = ctx.workspace_layout_fp8()
    ws = torch.empty(lay["total"], dtype=torch.uint8, device=DEV)
    out = L.nan_bf16(cfg.T, cfg.H)
    ctx.moe_fused_forward_fp8(L.x, L.d_logits, *wq["gate"], *wq["up"], *wq["down"], out, ws)
    torch.cuda.synchronize()
    L.check_device_status()
    sl = check_plan(S, ws, lay)
    R, H, F = cfg.R, cfg.H, cfg.F

    # x: codes and scales of the sampled rows' tokens, before and after dispatch
    xq_ref, sx_ref = f8.quantize_rows(orc.bf16_to_f64(S.x_bits[S.row_token]))
    tok = torch.from_numpy(S.row_token).to(DEV)
    assert np.array_equal(sl("xq", cfg.T * H, torch.uint8).view(cfg.T, H)[tok].cpu().numpy(), xq_ref), "xq"
    assert np.array_equal(sl("sx", cfg.T, torch.float32)[tok].cpu().numpy(), sx_ref), "sx"
    assert np.array_equal(gather_rows(sl("xq_perm", R * H, torch.uint8).view(R, H), S.rows), xq_ref), "xq_perm"
    assert np.array_equal(gather_rows(sl("sx_perm", R, torch.float32).view(R, 1), S.rows)[:, 0], sx_ref), "sx_perm"

    h_gpu = dev_bf16_to_f64(sl("h", R * F, torch.bfloat16).view(R, F)[torch.from_numpy(S.rows).to(DEV)])
    hq_gpu = gather_rows(sl("hq", R * F, torch.uint8).view(R, F), S.rows)
    sh_gpu = gather_rows(sl("sh", R, torch.float32).view(R, 1), S.rows)[:, 0]
    y_gpu = dev_bf16_to_f64(sl("y_perm", R * H, torch.bfloat16).view(R, H)[torch.from_numpy(S.rows).to(DEV)])
    # h is quantised from the GPU's own bf16 h: the oracle's quantisation of those rows must give the same codes
    want_hq, want_sh = f8.quantize_rows(h_gpu.astype(np.float32))
    assert np.array_equal(sh_gpu, want_sh) and np.array_equal(hq_gpu, want_hq), "hq / sh"

    h_ref = np.zeros((len(S.rows), len(S.h_cols)))
    y_ref = np.zeros((len(S.rows), len(S.y_cols)))

    def one_expert(e):
        idx = S.rows_of(e)
        g, u, d = L.weights(e)
        gq, sg = f8.quantize_rows(orc.bf16_to_f64(g[S.h_cols]))
        uq, su = f8.quantize_rows(orc.bf16_to_f64(u[S.h_cols]))
        dq, sd = f8.quantize_rows(orc.bf16_to_f64(d[S.y_cols]))
        # the GPU's weight codes and scales of those rows are the oracle's
        for wname, cols, q, s, per in (("gate", S.h_cols, gq, sg, F), ("up", S.h_cols, uq, su, F), ("down", S.y_cols, dq, sd, H)):
            at = torch.from_numpy(e * per + cols).to(DEV)
            assert np.array_equal(wq[wname][0][at].cpu().numpy(), q), f"W_{wname}[{e}] codes"
            assert np.array_equal(wq[wname][1][at].cpu().numpy(), s), f"W_{wname}[{e}] scales"
        gg = f8.scaled_gemm(xq_ref[idx], sx_ref[idx], gq, sg)
        uu = f8.scaled_gemm(xq_ref[idx], sx_ref[idx], uq, su)
        h_ref[idx] = orc.silu(gg) * uu
        y_ref[idx] = f8.scaled_gemm(hq_gpu[idx], sh_gpu[idx], dq, sd)      # Linear-2 on the GPU's own codes

    with ThreadPoolExecutor(max_workers=8) as pool:
        list(pool.map(one_expert, S.experts))
    assert_rows_close(h_gpu[:, S.h_cols], h_ref, f"fp8 h[{name}]")
    assert_rows_close(y_gpu[:, S.y_cols], y_ref, f"fp8 y_perm[{name}]")
    out_np = dev_bf16_to_f64(out)
    assert np.isfinite(out_np).all(), "every token row must be written"
    assert_out_close(out_np[S.out_tokens][:, S.y_cols], S.out_reference(y_ref), f"fp8 out[{name}]")


MX_CASES = [("C2", 24, 0), ("C3", 6, 12)]


def words_to_bytes(words_rows: np.ndarray) -> np.ndarray:
    """scale words [K/128, n] (int32, one column per row) -> scale bytes [n, K/32] in the oracle's order."""
    w = np.ascontiguousarray(words_rows).view(np.uint8).reshape(words_rows.shape[0], words_rows.shape[1], 4)
    return np.ascontiguousarray(w.transpose(1, 0, 2)).reshape(words_rows.shape[1], -1)


@pytest.mark.parametrize("name,n_out,n_extra", MX_CASES, ids=[c[0] for c in MX_CASES])
def test_mx_path_full_size_sampled(name, n_out, n_extra):
    cfg = gen.CONFIGS[name]
    S = Sample(cfg, n_out, n_extra)
    L = Layer(cfg, keep_experts=set(S.experts), x_bits=S.x_bits, logits=S.logits)
    ctx = L.ctx
    T, R, H, F, E = cfg.T, cfg.R, cfg.H, cfg.F, cfg.E
    wq = {}
    for wname, w in (("gate", L.w_gate), ("up", L.w_up), ("down", L.w_down)):
        _, r, c = w.shape
        codes = torch.empty((E * r, c), dtype=torch.uint8, device=DEV)
        words = torch.empty((c // 128, E * r), dtype=torch.int32, device=DEV)
        ctx.moe_quantize_rows_mx(w.view(E * r, c), E * r, c, codes, words)
        wq[wname] = (codes, words)
    torch.cuda.synchronize()
    del L.w_gate, L.w_up, L.w_down
    rows_dev = torch.from_numpy(S.rows).to(DEV)

    # the path call by call, so that the fp32 h the GPU quantises can be read back
    L.plan()
    xq = torch.empty((T, H), dtype=torch.uint8, device=DEV)
    sfx = torch.empty((H // 128, T), dtype=torch.int32, device=DEV)
    ctx.moe_quantize_rows_mx(L.x, T, H, xq, sfx)
    xq_perm = torch.empty((R, H), dtype=torch.uint8, device=DEV)
    sfx_perm = torch.empty((H // 128, R), dtype=torch.int32, device=DEV)
    ctx.moe_dispatch_mx(xq, sfx, L.inv_perm, xq_perm, sfx_perm)
    hq = torch.empty((R, F), dtype=torch.uint8, device=DEV)
    sfh = torch.empty((F // 128, R), dtype=torch.int32, device=DEV)
    y = L.nan_bf16(R, H)
    h_dbg = torch.full((R, F), float("nan"), device=DEV)
    ctx.moe_expert_ffn_mx(xq_perm, sfx_perm, L.offsets, *wq["gate"], *wq["up"], *wq["down"], hq, sfh, y, h_dbg)
    out_steps = L.nan_bf16(T, H)
    ctx.moe_combine(y, L.inv_perm, L.topk_w, out_steps)
    torch.cuda.synchronize()
    L.check_device_status()
    assert np.array_equal(L.perm.cpu().numpy(), S.perm) and np.array_equal(L.offsets.cpu().numpy(), S.offsets)

    xq_ref, sx_ref = mx.quantize_rows(orc.bf16_to_f64(S.x_bits[S.row_token]))
    tok = torch.from_numpy(S.row_token).to(DEV)
    assert np.array_equal(xq[tok].cpu().numpy(), xq_ref), "xq"
    assert np.array_equal(words_to_bytes(sfx[:, tok].cpu().numpy()), sx_ref), "x scale bytes"
    assert np.array_equal(xq_perm[rows_dev].cpu().numpy(), xq_ref), "xq_perm"
    assert np.array_equal(words_to_bytes(sfx_perm[:, rows_dev].cpu().numpy()), sx_ref), "dispatched scale bytes"

    h_gpu = h_dbg[rows_dev].cpu().numpy()
    assert np.isfinite(h_gpu).all()
    hq_gpu = hq[rows_dev].cpu().numpy()
    sh_gpu = words_to_bytes(sfh[:, rows_dev].cpu().numpy())
    want_hq, want_sh = mx.quantize_rows(h_gpu)       # the oracle's quantisation of the GPU's own fp32 h
    assert np.array_equal(sh_gpu, want_sh) and np.array_equal(hq_gpu, want_hq), "hq / h scale bytes"
    y_gpu = dev_bf16_to_f64(y[rows_dev])
    del h_dbg

    h_ref = np.zeros((len(S.rows), len(S.h_cols)))
    y_ref = np.zeros((len(S.rows), len(S.y_cols)))

    def one_expert(e):
        idx = S.rows_of(e)
        g, u, d = L.weights(e)
        (gq, gs), (uq, us), (dq, ds) = (mx.quantize_rows(orc.bf16_to_f64(m)) for m in (g[S.h_cols], u[S.h_cols], d[S.y_cols]))
        for wname, cols, q, s, per in (("gate", S.h_cols, gq, gs, F), ("up", S.h_cols, uq, us, F), ("down", S.y_cols, dq, ds, H)):
            at = torch.from_numpy(e * per + cols).to(DEV)
            assert np.array_equal(wq[wname][0][at].cpu().numpy(), q), f"W_{wname}[{e}] codes"
            assert np.array_equal(words_to_bytes(wq[wname][1][:, at].cpu().numpy()), s), f"W_{wname}[{e}] scale bytes"
        gg = mx.gemm(xq_ref[idx], sx_ref[idx], gq, gs)
        uu = mx.gemm(xq_ref[idx], sx_ref[idx], uq, us)
        h_ref[idx] = orc.silu(gg) * uu
        y_ref[idx] = mx.gemm(hq_gpu[idx], sh_gpu[idx], dq, ds)             # Linear-2 on the GPU's own codes

    with ThreadPoolExecutor(max_workers=8) as pool:
        list(pool.map(one_expert, S.experts))
    assert_rows_close(h_gpu[:, S.h_cols].astype(np.float64), h_ref, f"mx h[{name}]")
    assert_rows_close(y_gpu[:, S.y_cols], y_ref, f"mx y_perm[{name}]")
    out_np = dev_bf16_to_f64(out_steps)
    assert np.isfinite(out_np).all(), "every token row must be written"
    assert_out_close(out_np[S.out_tokens][:, S.y_cols], S.out_reference(y_ref), f"mx out[{name}]")

    # the fused entry point runs the same kernels on the same inputs: its output is the step-by-step one, bit for bit
    del xq, sfx, xq_perm, sfx_perm, hq, sfh, y
    lay = ctx.workspace_layout_mx()
    ws = torch.empty(lay["total"], dtype=torch.uint8, device=DEV)
    out = L.nan_bf16(T, H)
    ctx.moe_fused_forward_mx(L.x, L.d_logits, *wq["gate"], *wq["up"], *wq["down"], out, ws)
    torch.cuda.synchronize()
    L.check_device_status()
    check_plan(S, ws, lay)
    assert torch.equal(out.view(torch.int16), out_steps.view(torch.int16)), "fused MXFP8 forward differs from its steps"
