"""GPU parity of the FP8 (E4M3, W8A8) variant against oracle/fp8_oracle.py: quantised codes and scales bit for
bit, expert activations and the layer output within tolerance."""
import numpy as np
import pytest
import torch

from oracle import fp8_oracle as f8, moe_oracle as orc
from paper_2607_23264_b200 import binding, inputs as gen
from moe_testlib import DEV, TOL_FRO, Layer, assert_out_close, bits_to_dev, dev_bf16_to_f64, rel_fro

pytestmark = pytest.mark.gpu

CASES = [
    gen.MoEConfig("f8_small", T=300, H=256, F=384, E=5, k=2, seed=91, router="xWr"),
    gen.MoEConfig("f8_skew", T=700, H=128, F=256, E=24, k=4, seed=92, router="xWr_zipf"),
    gen.MoEConfig("f8_dense", T=2600, H=384, F=512, E=2, k=2, seed=93, router="xWr"),      # CTA-pair kernel
    # about 1000 rows per expert in two launches: below the CTA-pair threshold, so 256-row tiles on both accumulators,
    # with a short swapped-operand or 128-row tile at the end of each expert
    gen.MoEConfig("f8_wide", T=3000, H=512, F=1024, E=6, k=2, seed=94, router="xWr"),
    gen.MoEConfig("f8_limits", T=70, H=128, F=128, E=1024, k=32, seed=95, router="xWr"),   # the boundary's largest E and k
]


def quantize_on_gpu(ctx, t_bf16):
    rows, cols = t_bf16.shape
    codes = torch.empty((rows, cols), dtype=torch.uint8, device=DEV)
    scales = torch.empty((rows,), dtype=torch.float32, device=DEV)
    ctx.moe_quantize_rows(t_bf16, rows, cols, codes, scales)
    return codes, scales


def test_quantize_rows_bit_exact():
    ctx = binding.Context(8, 128, 128, 2, 1)
    rng = np.random.default_rng(3)
    for rows, cols in [(1, 8), (37, 264), (300, 14336), (5, 128)]:
        v = (rng.standard_normal((rows, cols)) * rng.uniform(1e-3, 50, size=(rows, 1))).astype(np.float32)
        if rows > 2:
            v[1] = 0.0                                   # an all-zero row
            v[2, :] = np.float32(2.0 ** -20)             # constant row: every element is the row maximum
        bits = gen.f32_to_bf16_bits(v)
        codes, scales = quantize_on_gpu(ctx, bits_to_dev(bits))
        torch.cuda.synchronize()
        want_q, want_s = f8.quantize_rows(gen.bf16_bits_to_f32(bits))
        assert np.array_equal(scales.cpu().numpy(), want_s), "scales"
        assert np.array_equal(codes.cpu().numpy(), want_q), "codes"


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
def test_fused_forward_fp8_parity(cfg):
    L = Layer(cfg)
    ctx = L.ctx
    ref = f8.forward_fp8(L.x_bits, L.logits, cfg.k, L.weights)
    # weights are quantised on the GPU (per output channel) and must match the oracle's codes and scales exactly
    wq = {}
    for name, w in (("gate", L.w_gate), ("up", L.w_up), ("down", L.w_down)):
        E, r, c = w.shape
        wq[name] = quantize_on_gpu(ctx, w.view(E * r, c))
    torch.cuda.synchronize()
    for e in (0, cfg.E - 1):
        g, u, d = L.weights(e)
        for name, bits in (("gate", g), ("up", u), ("down", d)):
            q, s = f8.quantize_rows(orc.bf16_to_f64(bits))
            rows = bits.shape[0]
            assert np.array_equal(wq[name][0][e * rows:(e + 1) * rows].cpu().numpy(), q), f"W_{name}[{e}] codes"
            assert np.array_equal(wq[name][1][e * rows:(e + 1) * rows].cpu().numpy(), s), f"W_{name}[{e}] scales"

    lay = ctx.workspace_layout_fp8()
    ws = torch.empty(lay["total"], dtype=torch.uint8, device=DEV)
    ws.fill_(0xFF)
    out = L.nan_bf16(cfg.T, cfg.H)
    for _ in range(2):
        ctx.moe_fused_forward_fp8(L.x, L.d_logits, wq["gate"][0], wq["gate"][1], wq["up"][0], wq["up"][1],
                                  wq["down"][0], wq["down"][1], out, ws)
    torch.cuda.synchronize()
    L.check_device_status()
    assert ctx.moe_last_launch_count() == 9
    R = cfg.R

    def sl(name, count, dtype):
        nbytes = count * torch.empty((), dtype=dtype).element_size()
        return ws[lay[name]:lay[name] + nbytes].view(dtype)

    for name, count in (("topk_ids", R), ("counts", cfg.E), ("offsets", cfg.E + 1), ("perm", R), ("inv_perm", R)):
        assert np.array_equal(sl(name, count, torch.int32).cpu().numpy(), np.asarray(ref[name]).reshape(-1)), name
    # activations: codes and scales bit for bit
    assert np.array_equal(sl("xq", cfg.T * cfg.H, torch.uint8).cpu().numpy().reshape(cfg.T, cfg.H), ref["xq"])
    assert np.array_equal(sl("sx", cfg.T, torch.float32).cpu().numpy(), ref["sx"])
    assert np.array_equal(sl("xq_perm", R * cfg.H, torch.uint8).cpu().numpy().reshape(R, cfg.H), ref["xq_perm"])
    assert np.array_equal(sl("sx_perm", R, torch.float32).cpu().numpy(), ref["sx_perm"])
    # h before quantisation (bf16), against the oracle's fp64 h
    h = dev_bf16_to_f64(sl("h", R * cfg.F, torch.bfloat16)).reshape(R, cfg.F)
    assert rel_fro(h, ref["h"]) <= TOL_FRO
    # hq: the GPU quantises ITS h (bf16, fp32-accumulated); re-quantising that h with the oracle must give its codes
    hq = sl("hq", R * cfg.F, torch.uint8).cpu().numpy().reshape(R, cfg.F)
    sh = sl("sh", R, torch.float32).cpu().numpy()
    want_hq, want_sh = f8.quantize_rows(h.astype(np.float32))
    assert np.array_equal(sh, want_sh) and np.array_equal(hq, want_hq)
    # Linear-2 on the GPU's own hq: isolates its arithmetic from quantisation decisions that flipped upstream
    y = dev_bf16_to_f64(sl("y_perm", R * cfg.H, torch.bfloat16)).reshape(R, cfg.H)
    y_ref_own = np.zeros_like(y)
    for e in range(cfg.E):
        lo, hi = int(ref["offsets"][e]), int(ref["offsets"][e + 1])
        if hi > lo:
            dq, sd = f8.quantize_rows(orc.bf16_to_f64(L.weights(e)[2]))
            y_ref_own[lo:hi] = f8.scaled_gemm(hq[lo:hi], sh[lo:hi], dq, sd)
    assert rel_fro(y, y_ref_own) <= TOL_FRO
    # the output against the oracle's combine of those rows: the bf16 path's elementwise bound
    out_np = dev_bf16_to_f64(out)
    assert_out_close(out_np, orc.combine(y_ref_own, ref["inv_perm"], ref["topk_w"]), f"fp8 out[{cfg.name}]")
    # end to end against the fully independent oracle (its own h, its own codes): where the GPU's bf16 h and the
    # oracle's differ in the last bit, an E4M3 code can flip and move that element of h by one step (up to 7 % of
    # the row maximum), so single outputs may leave the elementwise bound; the norms must still agree
    assert rel_fro(y, ref["y_perm"]) <= 2e-2
    assert rel_fro(out_np, ref["out"]) <= 2e-2
    # and the FP8 layer stays within E4M3 noise of the bf16 layer
    full = orc.forward(L.x_bits, L.logits, cfg.k, L.weights)
    assert rel_fro(dev_bf16_to_f64(out), full["out"]) < 0.08


def test_fp8_kernel_choices_give_the_same_bits(monkeypatch):
    """On a layer of many-row experts Linear-1 runs as CTA pairs by default; the single-CTA kernel everywhere
    (debug_flags bit 4), CTA pairs for both GEMMs (bit 3) and 128-row tiles only give the same output bits."""
    cfg = CASES[2]
    assert cfg.R // cfg.E >= 1024
    outs = []
    for env, flags in ((None, 0), (None, 16), (None, 8), ("x.wide_tiles=0", 16), ("x.fp8_pair_phases=3", 0)):
        if env is None:
            monkeypatch.delenv("MOE_TUNING", raising=False)
        else:
            monkeypatch.setenv("MOE_TUNING", env)
        L = Layer(cfg)                       # the context reads the variable when it is created
        ctx = L.ctx
        wq = []
        for w in (L.w_gate, L.w_up, L.w_down):
            E, r, c = w.shape
            wq.extend(quantize_on_gpu(ctx, w.view(E * r, c)))
        ws = torch.empty(ctx.workspace_layout_fp8()["total"], dtype=torch.uint8, device=DEV)
        out = L.nan_bf16(cfg.T, cfg.H)
        ctx.moe_fused_forward_fp8(L.x, L.d_logits, *wq, out, ws, tuning=binding.make_tuning(debug_flags=flags))
        torch.cuda.synchronize()
        L.check_device_status()
        outs.append(out)
    for o in outs[1:]:
        assert torch.equal(o.view(torch.int16), outs[0].view(torch.int16))


def test_fused_forward_fp8_random_layers():
    """The same checks on random layers: ragged and empty experts, one to thousands of rows per expert."""
    rng = np.random.default_rng(8)
    for trial in range(6):
        E = int(rng.integers(1, 5)) if trial % 2 else int(rng.integers(5, 30))
        cfg = gen.random_small_config(rng, T=int(rng.integers(1, 3000)), E=E, k=int(rng.integers(1, min(E, 8) + 1)),
                                      H=128 * int(rng.integers(1, 5)), F=128 * int(rng.integers(1, 5)),
                                      router="xWr_zipf" if trial % 3 == 0 else "xWr")
        test_fused_forward_fp8_parity(cfg)


def test_fp8_rejects_unsupported_requests():
    ctx = binding.Context(16, 192, 128, 2, 1)          # H not a multiple of 128
    with pytest.raises(binding.MoeError) as ei:
        ctx.workspace_layout_fp8()
    assert ei.value.code == 2
    ctx = binding.Context(16, 128, 128, 2, 1)
    z = torch.zeros(64 * 1024, dtype=torch.uint8, device=DEV)
    f = z.view(torch.float32)
    with pytest.raises(binding.MoeError) as ei:        # interleaved schedule is bf16-only
        ctx.moe_fused_forward_fp8(z, f, z, f, z, f, z, f, z, z, tuning=binding.make_tuning(1, 0, 1, schedule=1))
    assert ei.value.code == 7
    with pytest.raises(binding.MoeError) as ei:
        ctx.moe_quantize_rows(z, 4, 12, z, f)          # cols not a multiple of 8
    assert ei.value.code == 1
