"""GPU parity: every C-ABI call against the CPU oracle on the same seeded inputs (small sizes, full
element-by-element comparison).  Indices bit-exact; values within the stated tolerances."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as orc
from paper_2607_23264_b200 import binding, inputs as gen
from moe_testlib import (DEV, TOL_FRO, Layer, assert_out_close, assert_plan_matches, bits_to_dev, dev_bf16_to_f64,
                         dev_to_bits, rel_fro)

pytestmark = pytest.mark.gpu

# Small layers spanning several 128-row tiles, ragged tails, empty experts and N tails (F=192, H=320).
SMALL = [
    gen.CONFIGS["C1"],
    gen.MoEConfig("ragged", T=333, H=320, F=192, E=5, k=2, seed=11, router="xWr"),
    gen.MoEConfig("k1", T=200, H=128, F=128, E=3, k=1, seed=12, router="xWr"),
    gen.MoEConfig("one_expert", T=300, H=64, F=64, E=1, k=1, seed=13, router="xWr"),
    gen.MoEConfig("k_eq_E", T=50, H=128, F=256, E=4, k=4, seed=14, router="xWr"),
    gen.MoEConfig("skewed", T=700, H=256, F=128, E=40, k=4, seed=15, router="xWr_zipf"),
    gen.MoEConfig("tiny_T", T=3, H=64, F=64, E=16, k=2, seed=16, router="iid"),
    gen.MoEConfig("deep_k", T=130, H=1024, F=1088, E=6, k=3, seed=17, router="xWr"),
]
IDS = [c.name for c in SMALL]


def oracle_for(layer: Layer) -> dict:
    return orc.forward(layer.x_bits, layer.logits, layer.cfg.k, layer.weights)


@pytest.mark.parametrize("cfg", SMALL, ids=IDS)
def test_plan_routing_bit_exact(cfg):
    L = Layer(cfg, upload_weights=False)
    L.plan()
    ids, w = orc.topk_route(L.logits, cfg.k)
    counts, offsets, perm, inv = orc.plan_permutation(ids, cfg.E)
    assert_plan_matches(L, dict(topk_ids=ids, topk_w=w, counts=counts, offsets=offsets, perm=perm, inv_perm=inv))


def test_plan_routing_ties_and_wide_experts():
    """Logits with many exact ties (tie-break to the lower index) and E beyond one warp's width."""
    rng = np.random.default_rng(5)
    for (T, E, k) in [(97, 8, 3), (260, 256, 8), (64, 1000, 32), (33, 31, 31)]:
        cfg = gen.MoEConfig("ties", T=T, H=64, F=64, E=E, k=k, seed=0, router="iid")
        logits = (rng.integers(-3, 4, size=(T, E)) * 0.25).astype(np.float32)
        L = Layer(cfg, upload_weights=False, logits=logits)
        L.plan()
        ids, w = orc.topk_route(logits, k)
        counts, offsets, perm, inv = orc.plan_permutation(ids, E)
        assert_plan_matches(L, dict(topk_ids=ids, topk_w=w, counts=counts, offsets=offsets, perm=perm, inv_perm=inv))


@pytest.mark.parametrize("cfg", SMALL, ids=IDS)
def test_dispatch_bit_exact(cfg):
    L = Layer(cfg, upload_weights=False)
    ids, _ = orc.topk_route(L.logits, cfg.k)
    _, _, perm, inv = orc.plan_permutation(ids, cfg.E)
    x_perm = L.nan_bf16(cfg.R + 1, cfg.H)          # one canary row after the buffer
    L.ctx.moe_dispatch(L.x, torch.from_numpy(inv).to(DEV), x_perm)
    torch.cuda.synchronize()
    got = dev_to_bits(x_perm)
    assert np.array_equal(got[:cfg.R], orc.dispatch(L.x_bits, perm, cfg.k))
    assert np.all(got[cfg.R] == got[cfg.R, 0]) and np.isnan(gen.bf16_bits_to_f32(got[cfg.R, :1]))[0], "canary row"


@pytest.mark.parametrize("cfg", SMALL, ids=IDS)
def test_expert_ffn_parity(cfg):
    L = Layer(cfg)
    ref = oracle_for(L)
    x_perm = bits_to_dev(ref["x_perm"])
    offsets = torch.from_numpy(ref["offsets"]).to(DEV)
    h = L.nan_bf16(cfg.R + 1, cfg.F)
    y = L.nan_bf16(cfg.R + 1, cfg.H)
    h32 = torch.full((cfg.R, cfg.F), float("nan"), dtype=torch.float32, device=DEV)
    L.ctx.moe_expert_ffn(x_perm, offsets, L.w_gate, L.w_up, L.w_down, h, y, h_fp32_debug=h32)
    torch.cuda.synchronize()
    L.check_device_status()
    assert L.ctx.moe_last_launch_count() in (1, 2)      # tiny layers run both GEMMs in one launch
    h32_np = h32.cpu().numpy().astype(np.float64)
    assert np.isfinite(h32_np).all(), "every row of h belongs to an expert and must be written"
    assert rel_fro(h32_np, ref["h"]) <= TOL_FRO
    h_np, y_np = dev_bf16_to_f64(h), dev_bf16_to_f64(y)
    assert np.isnan(h_np[cfg.R]).all() and np.isnan(y_np[cfg.R]).all(), "canary rows must stay untouched"
    assert rel_fro(h_np[:cfg.R], ref["h"]) <= TOL_FRO
    assert rel_fro(y_np[:cfg.R], ref["y_perm"]) <= TOL_FRO
    # per expert too, so that a small expert cannot hide behind a large one
    for e in range(cfg.E):
        lo, hi = ref["offsets"][e], ref["offsets"][e + 1]
        if hi > lo:
            assert rel_fro(y_np[lo:hi], ref["y_perm"][lo:hi]) <= 2 * TOL_FRO, f"expert {e}"


@pytest.mark.parametrize("cfg", SMALL, ids=IDS)
def test_combine_parity(cfg):
    L = Layer(cfg, upload_weights=False)
    rng = np.random.default_rng(cfg.seed)
    y_bits = gen.f32_to_bf16_bits(rng.standard_normal((cfg.R, cfg.H)).astype(np.float32))
    ids, w = orc.topk_route(L.logits, cfg.k)
    _, _, _, inv = orc.plan_permutation(ids, cfg.E)
    w32 = w.astype(np.float32)
    out = L.nan_bf16(cfg.T, cfg.H)
    L.ctx.moe_combine(bits_to_dev(y_bits), torch.from_numpy(inv).to(DEV), torch.from_numpy(w32).to(DEV), out)
    torch.cuda.synchronize()
    ref = orc.combine(orc.bf16_to_f64(y_bits), inv, w32.astype(np.float64))
    got = dev_bf16_to_f64(out)
    # fp32 accumulation of k terms then one bf16 rounding: relative error about 2^-9
    np.testing.assert_allclose(got, ref, rtol=2.0 ** -8, atol=1e-6)


@pytest.mark.parametrize("cfg", SMALL, ids=IDS)
def test_fused_forward_parity(cfg):
    L = Layer(cfg)
    ref = oracle_for(L)
    lay = L.ctx.workspace_layout()
    ws = torch.empty(lay["total"], dtype=torch.uint8, device=DEV)
    ws.fill_(0xFF)
    out = L.nan_bf16(cfg.T, cfg.H)
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws)
    torch.cuda.synchronize()
    L.check_device_status()
    assert L.ctx.moe_last_launch_count() in (6, 7)

    def sl(name, count, dtype):
        nbytes = count * torch.empty((), dtype=dtype).element_size()
        return ws[lay[name]:lay[name] + nbytes].view(dtype)

    R = cfg.R
    for name, count in (("topk_ids", R), ("counts", cfg.E), ("offsets", cfg.E + 1), ("perm", R), ("inv_perm", R)):
        got = sl(name, count, torch.int32).cpu().numpy()
        assert np.array_equal(got, np.asarray(ref[name]).reshape(-1)), name
    assert np.abs(sl("topk_w", R, torch.float32).cpu().numpy() - ref["topk_w"].reshape(-1)).max() <= 1e-6
    assert np.array_equal(dev_to_bits(sl("x_perm", R * cfg.H, torch.bfloat16)).reshape(R, cfg.H), ref["x_perm"])
    assert rel_fro(dev_bf16_to_f64(sl("h", R * cfg.F, torch.bfloat16)).reshape(R, cfg.F), ref["h"]) <= TOL_FRO
    assert rel_fro(dev_bf16_to_f64(sl("y_perm", R * cfg.H, torch.bfloat16)).reshape(R, cfg.H), ref["y_perm"]) <= TOL_FRO
    assert_out_close(dev_bf16_to_f64(out), ref["out"], f"out[{cfg.name}]")

    # determinism: a second run is bitwise identical
    out2 = L.nan_bf16(cfg.T, cfg.H)
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out2, ws)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))


def test_fused_forward_host_matches_device_path():
    cfg = SMALL[1]
    L = Layer(cfg)
    ws = torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
    out = L.nan_bf16(cfg.T, cfg.H)
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws)
    x_host = torch.from_numpy(L.x_bits.view(np.int16)).pin_memory()
    logits_host = torch.from_numpy(L.logits).pin_memory()
    out_host = torch.zeros((cfg.T, cfg.H), dtype=torch.int16).pin_memory()
    L.ctx.moe_fused_forward_host(x_host, logits_host, L.w_gate, L.w_up, L.w_down, out_host, ws)
    torch.cuda.synchronize()
    assert np.array_equal(out_host.numpy().view(np.uint16), dev_to_bits(out))


def test_pipelined_host_calls_match_device_path():
    """Five pipelined host-buffer steps on different batches: every out_host equals the device-resident result."""
    cfg = SMALL[1]
    L = Layer(cfg)
    ws = torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
    rng = np.random.default_rng(9)
    xs, lgs, outs, want = [], [], [], []
    for i in range(5):
        xb = np.roll(L.x_bits, 7 * i, axis=0).copy()
        lg = gen.make_logits(cfg, xb)
        out = L.nan_bf16(cfg.T, cfg.H)
        L.ctx.moe_fused_forward(bits_to_dev(xb), torch.from_numpy(lg).to(DEV), L.w_gate, L.w_up, L.w_down, out, ws)
        torch.cuda.synchronize()
        want.append(dev_to_bits(out))
        xs.append(torch.from_numpy(xb.view(np.int16)).pin_memory())
        lgs.append(torch.from_numpy(lg).pin_memory())
        outs.append(torch.zeros((cfg.T, cfg.H), dtype=torch.int16).pin_memory())
    for i in range(5):
        L.ctx.moe_fused_forward_host_pipelined(xs[i], lgs[i], L.w_gate, L.w_up, L.w_down, outs[i], ws)
    L.ctx.moe_host_pipeline_flush()
    torch.cuda.synchronize()
    for i in range(5):
        assert np.array_equal(outs[i].numpy().view(np.uint16), want[i]), f"step {i}"
    L.check_device_status()


def test_pacing_points_are_bitwise_identical():
    """Store pacing reorders stores in time only: all 20 sweep points give the same bits."""
    cfg = gen.MoEConfig("pace", T=2400, H=512, F=1024, E=4, k=2, seed=31, router="xWr")   # large enough for two launches
    L = Layer(cfg)
    ws = torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
    base = L.nan_bf16(cfg.T, cfg.H)
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, base, ws)
    torch.cuda.synchronize()
    ref = orc.forward(L.x_bits, L.logits, cfg.k, L.weights)
    assert_out_close(dev_bf16_to_f64(base), ref["out"], "pacing baseline")
    points = [(b, 0, 1) for b in (1, 2, 4, 8, 16)] + [(b, 1, ik) for b in (1, 2, 4, 8, 16) for ik in (1, 2, 4)]
    assert len(points) == 20
    for pairs in (0, 8):                       # the single-CTA kernel, then the CTA-pair kernel (forced)
        for b, mode, ik in points:
            out = L.nan_bf16(cfg.T, cfg.H)
            L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws,
                                    tuning=binding.make_tuning(b, mode, ik, debug_flags=pairs))
            torch.cuda.synchronize()
            assert torch.equal(out.view(torch.int16), base.view(torch.int16)), (pairs, b, mode, ik)
    L.check_device_status()
    # in a CTA pair both CTAs pace their stores on the leader's MMA progress: with a gap after every store tile the
    # hold counter (trace field 7) moves in leaders (even CTAs) and peers (odd CTAs) that drained a tile
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws,
                            tuning=binding.make_tuning(1, 1, 4, debug_flags=8 | 1))
    torch.cuda.synchronize()
    tr = L.ctx.moe_get_ffn_trace()
    drained = tr[1][:, 5] > 0
    assert drained[0::2].any() and drained[1::2].any()
    held = tr[1][:, 7] > 0
    assert held[0::2][drained[0::2]].any(), "no leader CTA held a store"
    assert held[1::2][drained[1::2]].any(), "no peer CTA held a store: the peer drains unpaced"
    # a burst as large as a whole tile still inserts gaps, because the count runs across tiles: 8 store tiles are the two
    # accumulators of one 256-row Linear-1 tile, so a CTA that drains a second tile holds before its ninth store
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws,
                            tuning=binding.make_tuning(8, 1, 4, debug_flags=16 | 1))
    torch.cuda.synchronize()
    tr = L.ctx.moe_get_ffn_trace()
    assert (tr[0][:, 6] >= 2).any() and (tr[0][:, 7] > 0).any(), "a burst of 8 store tiles never held a store"
    L.check_device_status()


def test_environment_override_of_the_default_tuning(monkeypatch):
    """MOE_TUNING, read by moe_create, replaces the tuning of calls that pass none; an explicit tuning wins; a string
    the parser rejects makes moe_create fail."""
    cfg = gen.MoEConfig("env", T=2000, H=512, F=1024, E=6, k=2, seed=33, router="xWr")   # large enough for two launches
    base_layer = Layer(cfg)
    ws = torch.empty(base_layer.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
    base = base_layer.nan_bf16(cfg.T, cfg.H)
    # the built-in default runs the two GEMMs as two launches (7 kernels); the override asks for the interleaved order,
    # which runs them as one launch (6 kernels)
    base_layer.ctx.moe_fused_forward(base_layer.x, base_layer.d_logits, base_layer.w_gate, base_layer.w_up,
                                     base_layer.w_down, base, ws, tuning=binding.make_tuning(debug_flags=16))
    torch.cuda.synchronize()
    assert base_layer.ctx.moe_last_launch_count() == 7
    monkeypatch.setenv("MOE_TUNING", "schedule=1,lead=4,x.some_development_knob=0")
    L = Layer(cfg)
    out = L.nan_bf16(cfg.T, cfg.H)
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws)
    torch.cuda.synchronize()
    assert L.ctx.moe_last_launch_count() == 6, "the environment's schedule was not used"
    assert torch.equal(out.view(torch.int16), base.view(torch.int16))
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws,
                            tuning=binding.make_tuning(debug_flags=16))
    torch.cuda.synchronize()
    assert L.ctx.moe_last_launch_count() == 7, "an explicit tuning must win over the environment"
    L.check_device_status()
    monkeypatch.setenv("MOE_TUNING", "burst=3")
    with pytest.raises(binding.MoeError) as ei:
        binding.Context(cfg.T, cfg.H, cfg.F, cfg.E, cfg.k)
    assert ei.value.code == 1


def test_development_knobs_do_not_change_values(monkeypatch):
    """The development knobs of MOE_TUNING choose between ways of computing the same tiles (256-row tiles on or off or
    in one GEMM only, swapped operands up to 128 rows, 16-row boxes of A for larger tiles, L2 priorities off, register
    stores, the four-stage ring for tiny experts, one launch per GEMM on fine-grained layers, the CTA-pair kernel): every
    setting gives the bits of the default, on a layer of many-row experts, on a skewed one (250 rows per expert on
    average, experts of a few rows beside experts of a thousand: its GEMMs run as two launches each by default) and on a
    decode-like one."""
    settings = ("x.wide_tiles=0", "x.wide_tiles=2", "x.wide_phases=1", "x.wide_phases=2", "x.small_a=64,x.swap_rows=128",
                "x.small_a=0,x.swap_rows=16", "x.cache_hints=0", "x.bulk_stores=0", "x.small_ring=0", "x.split_sizes=0", "flags=8")
    for cfg in (gen.MoEConfig("knobs_dense", T=2000, H=512, F=1024, E=6, k=2, seed=91, router="xWr"),
                gen.MoEConfig("knobs_skew", T=1500, H=512, F=512, E=24, k=4, seed=92, router="xWr_zipf"),
                # a few rows per expert, two launches: the six-stage ring of 16-row A boxes
                gen.MoEConfig("knobs_decode", T=32, H=512, F=512, E=128, k=4, seed=93, router="xWr")):
        monkeypatch.delenv("MOE_TUNING", raising=False)
        base_layer = Layer(cfg)
        ws = torch.empty(base_layer.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
        base = base_layer.nan_bf16(cfg.T, cfg.H)
        base_layer.ctx.moe_fused_forward(base_layer.x, base_layer.d_logits, base_layer.w_gate, base_layer.w_up,
                                         base_layer.w_down, base, ws)
        torch.cuda.synchronize()
        assert_out_close(dev_bf16_to_f64(base), oracle_for(base_layer)["out"], f"out[{cfg.name}]")
        for setting in settings:
            monkeypatch.setenv("MOE_TUNING", setting)
            L = Layer(cfg)
            out = L.nan_bf16(cfg.T, cfg.H)
            L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws)
            torch.cuda.synchronize()
            L.check_device_status()
            assert torch.equal(out.view(torch.int16), base.view(torch.int16)), (cfg.name, setting)


def test_debug_check_refuses_non_finite_logits(monkeypatch):
    """Non-finite logits violate the routing contract and are not tested on the device; the debug entry
    x.check_logits=1 of MOE_TUNING tests them on the host and returns MOE_ERR_BAD_ROUTING before any launch."""
    cfg = gen.MoEConfig("nan", T=96, H=128, F=128, E=8, k=2, seed=35, router="xWr")
    monkeypatch.setenv("MOE_TUNING", "x.check_logits=1")
    L = Layer(cfg)
    L.plan()                                         # finite logits pass
    assert_plan_matches(L, oracle_for(L))
    for bad in (float("nan"), float("inf"), float("-inf")):
        logits = L.d_logits.clone()
        logits[17, 3] = bad
        with pytest.raises(binding.MoeError) as ei:
            L.ctx.moe_plan_routing(logits, L.topk_ids, L.topk_w, L.counts, L.offsets, L.perm, L.inv_perm)
        assert ei.value.code == 4
        ws = torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
        with pytest.raises(binding.MoeError) as ei:
            L.ctx.moe_fused_forward(L.x, logits, L.w_gate, L.w_up, L.w_down, L.nan_bf16(cfg.T, cfg.H), ws)
        assert ei.value.code == 4
        assert L.ctx.moe_last_launch_count() == 0
    monkeypatch.delenv("MOE_TUNING")
    L2 = Layer(cfg)                                  # without the entry nothing is tested (and nothing synchronises)
    logits = L2.d_logits.clone()
    logits[0, 0] = float("inf")
    L2.ctx.moe_plan_routing(logits, L2.topk_ids, L2.topk_w, L2.counts, L2.offsets, L2.perm, L2.inv_perm)
    torch.cuda.synchronize()


@pytest.mark.parametrize("cfg", [SMALL[0], SMALL[1], SMALL[5], SMALL[7],
                                 gen.MoEConfig("waves", T=1500, H=512, F=512, E=6, k=2, seed=51, router="xWr")],
                         ids=lambda c: c.name)
def test_schedules_are_bitwise_identical(cfg):
    """Expert-Wave as two launches, Expert-Wave as one launch with ready counters, and the interleaved order
    (Algorithm 1) for several leads compute the same bits: only the order of tiles changes."""
    L = Layer(cfg)
    lay = L.ctx.workspace_layout()
    ws = torch.empty(lay["total"], dtype=torch.uint8, device=DEV)
    base = L.nan_bf16(cfg.T, cfg.H)
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, base, ws)
    torch.cuda.synchronize()
    assert L.ctx.moe_last_launch_count() in (6, 7)
    ref = oracle_for(L)
    assert_out_close(dev_bf16_to_f64(base), ref["out"], f"out[{cfg.name}]")
    R = cfg.R
    h_base = ws[lay["h"]:lay["h"] + R * cfg.F * 2].clone()
    variants = [binding.make_tuning(1, 0, 1, debug_flags=2)] + \
               [binding.make_tuning(1, 0, 1, schedule=1, dep_lead_D=D) for D in (0, 1, 2, 7, 1000)] + \
               [binding.make_tuning(2, 1, 2, schedule=1, dep_lead_D=1)]
    for tn in variants:
        ws[lay["h"]:lay["h"] + R * cfg.F * 2].fill_(0xFF)          # stale h must not be read before it is rewritten
        out = L.nan_bf16(cfg.T, cfg.H)
        for _ in range(2):                                          # twice: the ready counters re-arm themselves
            L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws, tuning=tn)
        torch.cuda.synchronize()
        assert L.ctx.moe_last_launch_count() == 6
        what = (tn.schedule, tn.dep_lead_D, tn.debug_flags)
        assert torch.equal(ws[lay["h"]:lay["h"] + R * cfg.F * 2], h_base), what
        assert torch.equal(out.view(torch.int16), base.view(torch.int16)), what
    L.check_device_status()


@pytest.mark.parametrize("cfg", [SMALL[1], SMALL[3], SMALL[5], SMALL[7],
                                 gen.MoEConfig("pairs", T=3000, H=512, F=640, E=3, k=2, seed=81, router="xWr"),
                                 gen.MoEConfig("pair_tails", T=1500, H=1024, F=512, E=4, k=2, seed=82, router="xWr"),
                                 gen.MoEConfig("pair_tails_skew", T=2200, H=512, F=256, E=8, k=2, seed=83,
                                               router="xWr_zipf")],
                         ids=lambda c: c.name)
def test_cta_pair_kernel_matches_single_cta_kernel(cfg):
    """The cta_group::2 variant (256-row tiles over a cluster of two CTAs), forced on, gives the same bits as the
    single-CTA kernel, ragged and empty experts and odd block counts included."""
    L = Layer(cfg)
    lay = L.ctx.workspace_layout()
    ws = torch.empty(lay["total"], dtype=torch.uint8, device=DEV)
    base = L.nan_bf16(cfg.T, cfg.H)
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, base, ws,
                            tuning=binding.make_tuning(1, 0, 1, debug_flags=16))       # single-CTA kernel
    torch.cuda.synchronize()
    assert_out_close(dev_bf16_to_f64(base), oracle_for(L)["out"], f"out[{cfg.name}]")
    R = cfg.R
    h_base = ws[lay["h"]:lay["h"] + R * cfg.F * 2].clone()
    y_base = ws[lay["y_perm"]:lay["y_perm"] + R * cfg.H * 2].clone()
    for tn in (binding.make_tuning(1, 0, 1, debug_flags=8), binding.make_tuning(2, 1, 1, debug_flags=8 | 1)):
        ws[lay["h"]:lay["h"] + R * cfg.F * 2].fill_(0xFF)
        ws[lay["y_perm"]:lay["y_perm"] + R * cfg.H * 2].fill_(0xFF)
        out = L.nan_bf16(cfg.T, cfg.H)
        L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws, tuning=tn)
        torch.cuda.synchronize()
        L.check_device_status()
        assert torch.equal(ws[lay["h"]:lay["h"] + R * cfg.F * 2], h_base), "h"
        assert torch.equal(ws[lay["y_perm"]:lay["y_perm"] + R * cfg.H * 2], y_base), "y_perm"
        assert torch.equal(out.view(torch.int16), base.view(torch.int16))


def test_zero_tokens_is_a_no_op():
    ctx = binding.Context(0, 128, 128, 4, 2)
    counts = torch.full((4,), -1, dtype=torch.int32, device=DEV)
    offsets = torch.full((5,), -1, dtype=torch.int32, device=DEV)
    ctx.moe_plan_routing(None, None, None, counts, offsets, None, None)
    ctx.moe_dispatch(None, None, None)
    ctx.moe_combine(None, None, None, None)
    ctx.moe_expert_ffn(None, None, None, None, None, None, None)
    torch.cuda.synchronize()
    assert counts.eq(0).all() and offsets.eq(0).all()


def test_host_side_errors_are_synchronous():
    cfg = SMALL[0]
    L = Layer(cfg, upload_weights=False)
    ws = torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
    out = L.nan_bf16(cfg.T, cfg.H)
    w = torch.zeros(8, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(binding.MoeError) as ei:       # workspace too small
        L.ctx.moe_fused_forward(L.x, L.d_logits, w, w, w, out, ws[:4096])
    assert ei.value.code == 3
    with pytest.raises(binding.MoeError) as ei:       # misaligned pointer
        L.ctx.moe_dispatch(L.x.view(-1)[1:], L.inv_perm, out)
    assert ei.value.code == 1
    with pytest.raises(binding.MoeError) as ei:       # null pointer
        L.ctx.moe_combine(None, L.inv_perm, L.topk_w, out)
    assert ei.value.code == 1
    for bad in (binding.make_tuning(3, 0, 1), binding.make_tuning(1, 2, 1), binding.make_tuning(1, 1, 3),
                binding.make_tuning(1, 0, 1, dep_lead_D=1)):
        with pytest.raises(binding.MoeError) as ei:
            L.ctx.moe_fused_forward(L.x, L.d_logits, w, w, w, out, ws, tuning=bad)
        assert ei.value.code == 1
    with pytest.raises(binding.MoeError) as ei:       # unknown schedule
        L.ctx.moe_fused_forward(L.x, L.d_logits, w, w, w, out, ws, tuning=binding.make_tuning(1, 0, 1, schedule=2))
    assert ei.value.code == 7
    with pytest.raises(binding.MoeError) as ei:
        binding.Context(8, 100, 128, 4, 2)
    assert ei.value.code == 2
    torch.cuda.synchronize()
    L.check_device_status()


def test_kernel_times_of_back_to_back_calls():
    """The library keeps the per-kernel events of the last 32 timed calls, so a run of calls is timed per kernel without a
    host synchronisation in between; each call's kernel times sum to no more than the time between the calls' ends."""
    cfg = gen.MoEConfig("ring", T=2000, H=512, F=512, E=6, k=2, seed=62, router="xWr")
    L = Layer(cfg)
    ws = torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
    out = L.nan_bf16(cfg.T, cfg.H)
    step = lambda: L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws)
    for _ in range(3):
        step()
    n = 5
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
    L.ctx.moe_set_kernel_timing(True)
    assert all(v == -1 for v in L.ctx.moe_get_kernel_times_back(0)), "enabling clears the ring"
    marks[0].record()
    for i in range(n):
        step()
        marks[i + 1].record()
    torch.cuda.synchronize()
    per = [L.ctx.moe_get_kernel_times_back(b) for b in range(n)]      # per[0] = the last call
    assert all(len(ms) == 7 and all(v > 0 for v in ms) for ms in per)
    for b in range(n):
        step_ms = marks[n - 1 - b].elapsed_time(marks[n - b])
        assert sum(per[b]) <= step_ms * 1.02 + 0.01, (b, per[b], step_ms)
    assert per[0] == L.ctx.moe_get_kernel_times()
    assert all(v == -1 for v in L.ctx.moe_get_kernel_times_back(n)), "a slot no call has used reads -1"
    for bad in (-1, binding.TIMING_SLOTS):
        with pytest.raises(binding.MoeError) as ei:
            L.ctx.moe_get_kernel_times_back(bad)
        assert ei.value.code == 1
    L.ctx.moe_set_kernel_timing(False)
    L.check_device_status()


def test_ffn_trace_and_kernel_times():
    """Measurement aids: per-kernel event times and the per-CTA wait counters of the grouped GEMMs."""
    cfg = gen.MoEConfig("traced", T=4000, H=512, F=384, E=6, k=2, seed=61, router="xWr")   # two launches
    L = Layer(cfg)
    ws = torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
    out = L.nan_bf16(cfg.T, cfg.H)
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws)
    L.ctx.moe_set_kernel_timing(True)
    out2 = L.nan_bf16(cfg.T, cfg.H)
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out2, ws,
                            tuning=binding.make_tuning(1, 1, 2, debug_flags=1 | 16))     # single-CTA kernel, traced
    ms = L.ctx.moe_get_kernel_times()
    L.ctx.moe_set_kernel_timing(False)
    assert len(ms) == 7 and all(0 < v < 100 for v in ms)
    tr = L.ctx.moe_get_ffn_trace()
    assert tr.shape[0] == 2 and tr.shape[2] == len(binding.TRACE_FIELDS) == 12
    # every tile is processed exactly once.  A two-launch run of the single-CTA kernel cuts experts with more than 128
    # rows into 256-row blocks (one tile on both accumulators each, the last one possibly a 128-row or swapped tile)
    # and takes smaller experts as one block
    counts = L.ctx_counts = ws[L.ctx.workspace_layout()["counts"]:][: 4 * cfg.E].view(torch.int32).cpu().numpy()
    assert (counts > 128).all()
    mblocks = int(((counts + 255) // 256).sum())
    assert tr[0, :, 6].sum() == mblocks * ((cfg.F + 127) // 128)
    assert tr[1, :, 6].sum() == mblocks * ((cfg.H + 255) // 256)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16)), "tracing must not change values"
    # the same launches as one launch with ready counters work on 128-row blocks (and give the same bits)
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out2, ws,
                            tuning=binding.make_tuning(1, 0, 1, debug_flags=1 | 2))
    tr = L.ctx.moe_get_ffn_trace()
    blocks128 = int(((counts + 127) // 128).sum())
    assert tr[0, :, 6].sum() == blocks128 * ((cfg.F + 127) // 128 + (cfg.H + 255) // 256)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16)), "256-row tiles must not change values"
    # the CTA-pair kernel works on 256-row blocks; only the leader of a pair counts tiles
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out2, ws,
                            tuning=binding.make_tuning(1, 0, 1, debug_flags=1 | 8))
    tr = L.ctx.moe_get_ffn_trace()
    pblocks = int(((counts + 255) // 256).sum())
    assert tr[0, :, 6].sum() == pblocks * ((cfg.F + 127) // 128)
    assert tr[1, :, 6].sum() == pblocks * ((cfg.H + 255) // 256)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
    L.check_device_status()


def test_expired_wait_is_reported_not_hung():
    """Failure path without a GPU fault: the host asks Linear-1 to withhold its ready counts, so every bounded
    Linear-2 wait runs out; the kernel must unwind by itself, report MOE_ERR_TIMEOUT in the status word, and the
    context must stay usable (the next run is correct)."""
    import time
    cfg = gen.MoEConfig("drill", T=600, H=256, F=256, E=4, k=2, seed=71, router="xWr")
    L = Layer(cfg)
    ws = torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
    out = L.nan_bf16(cfg.T, cfg.H)
    t0 = time.time()
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws,
                            tuning=binding.make_tuning(1, 0, 1, debug_flags=4))
    code, detail = L.ctx.moe_last_device_status()          # synchronises
    assert time.time() - t0 < 10.0, "the drill must end by itself"
    assert code == 6, "MOE_ERR_TIMEOUT expected"
    assert detail >> 16 == 3 and (detail & 0xFFFF) in (1, 2, 3, 4, 5, 6, 7, 8), "kernel 3 (one launch), some role"
    assert L.ctx.moe_last_device_status() == (0, 0), "reading the status clears it"
    # the same context computes correctly afterwards: scheduler and ready counters were re-armed
    for tn in (None, binding.make_tuning(1, 0, 1, schedule=1, dep_lead_D=2)):
        L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws, tuning=tn)
        torch.cuda.synchronize()
        assert_out_close(dev_bf16_to_f64(out), oracle_for(L)["out"], "after the drill")
    L.check_device_status()


def test_random_small_layers_property():
    """Property tier: random small layers (ragged loads, empty experts, k up to 4, E up to 11) through every
    schedule and kernel variant; indices bit-exact, output within tolerance, variants bitwise equal."""
    rng = np.random.default_rng(2026)
    for trial in range(16):
        cfg = gen.random_small_config(rng)
        L = Layer(cfg)
        ref = oracle_for(L)
        lay = L.ctx.workspace_layout()
        ws = torch.empty(lay["total"], dtype=torch.uint8, device=DEV)
        outs = []
        for tn in (None, binding.make_tuning(1, 0, 1, debug_flags=8), binding.make_tuning(1, 0, 1, debug_flags=16),
                   binding.make_tuning(1, 0, 1, schedule=1, dep_lead_D=1 + trial % 3)):
            out = L.nan_bf16(cfg.T, cfg.H)
            L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws, tuning=tn)
            torch.cuda.synchronize()
            outs.append(out)
        what = f"trial {trial}: {cfg}"
        perm = ws[lay["perm"]:lay["perm"] + 4 * cfg.R].view(torch.int32).cpu().numpy()
        assert np.array_equal(perm, ref["perm"]), what
        assert_out_close(dev_bf16_to_f64(outs[0]), ref["out"], what)
        for o in outs[1:]:
            assert torch.equal(o.view(torch.int16), outs[0].view(torch.int16)), what
        L.check_device_status()


def test_random_mid_size_layers_property():
    """Random layers of up to 5000 tokens on few or many experts: several hundred to a few thousand rows per expert
    (256-row tiles on both accumulators, the merged order of many-row and few-row experts, swapped-operand remainders),
    through the default path, the CTA-pair kernel, the interleaved schedule and a paced store; all bitwise equal."""
    rng = np.random.default_rng(77)
    for trial in range(10):
        few = trial % 2 == 0
        E = int(rng.integers(1, 5)) if few else int(rng.integers(5, 40))
        cfg = gen.random_small_config(rng, T=int(rng.integers(1500, 5000)), E=E, k=int(rng.integers(1, min(E, 8) + 1)),
                                      H=64 * int(rng.integers(1, 9)), F=64 * int(rng.integers(1, 9)),
                                      router="xWr" if few else "xWr_zipf")
        L = Layer(cfg)
        ref = oracle_for(L)
        lay = L.ctx.workspace_layout()
        ws = torch.empty(lay["total"], dtype=torch.uint8, device=DEV)
        outs = []
        for tn in (None, binding.make_tuning(1, 0, 1, debug_flags=8),
                   binding.make_tuning(1, 0, 1, schedule=1, dep_lead_D=1 + trial % 3),
                   binding.make_tuning([2, 4, 8, 16][trial % 4], 1, [1, 2, 4][trial % 3])):
            out = L.nan_bf16(cfg.T, cfg.H)
            L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws, tuning=tn)
            torch.cuda.synchronize()
            outs.append(out)
        what = f"trial {trial}: {cfg}"
        perm = ws[lay["perm"]:lay["perm"] + 4 * cfg.R].view(torch.int32).cpu().numpy()
        assert np.array_equal(perm, ref["perm"]), what
        assert_out_close(dev_bf16_to_f64(outs[0]), ref["out"], what)
        for o in outs[1:]:
            assert torch.equal(o.view(torch.int16), outs[0].view(torch.int16)), what
        L.check_device_status()


def test_largest_expert_count_and_top_k():
    """E = 1024 experts and k = 32, the limits of the boundary: most experts hold no or a few rows, every kernel
    variant (default, CTA pairs, one launch, interleaved) gives the default's bits and the oracle's values."""
    cfg = gen.MoEConfig("limits", T=70, H=128, F=128, E=1024, k=32, seed=301, router="xWr")
    L = Layer(cfg)
    ref = oracle_for(L)
    lay = L.ctx.workspace_layout()
    ws = torch.empty(lay["total"], dtype=torch.uint8, device=DEV)
    outs = []
    for tn in (None, binding.make_tuning(1, 0, 1, debug_flags=8), binding.make_tuning(1, 0, 1, debug_flags=2),
               binding.make_tuning(1, 0, 1, schedule=1, dep_lead_D=2)):
        out = L.nan_bf16(cfg.T, cfg.H)
        L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws, tuning=tn)
        torch.cuda.synchronize()
        outs.append(out)
    for name in ("counts", "offsets", "perm", "inv_perm"):
        n = {"counts": cfg.E, "offsets": cfg.E + 1}.get(name, cfg.R)
        got = ws[lay[name]:lay[name] + 4 * n].view(torch.int32).cpu().numpy()
        assert np.array_equal(got, np.asarray(ref[name]).reshape(-1)), name
    assert_out_close(dev_bf16_to_f64(outs[0]), ref["out"], "E=1024, k=32")
    for o in outs[1:]:
        assert torch.equal(o.view(torch.int16), outs[0].view(torch.int16))
    L.check_device_status()


def test_smaller_batches_on_one_context():
    """A context created for T tokens serves any smaller batch (moe_set_active_tokens), with a workspace sized once."""
    cfg = gen.MoEConfig("varT", T=900, H=256, F=384, E=6, k=2, seed=101, router="xWr")
    L = Layer(cfg)
    ws = torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)      # sized for the creation shape
    for tokens in (900, 1, 137, 512, 0, 900):
        L.ctx.moe_set_active_tokens(tokens)
        assert L.ctx.workspace_bytes() <= ws.numel()
        out = L.nan_bf16(max(tokens, 1), cfg.H)
        L.ctx.moe_fused_forward(L.x[:tokens].contiguous() if tokens else L.x, L.d_logits[:tokens].contiguous() if tokens
                                else L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws)
        torch.cuda.synchronize()
        if tokens:
            ref = orc.forward(L.x_bits[:tokens], L.logits[:tokens], cfg.k, L.weights)
            assert_out_close(dev_bf16_to_f64(out[:tokens]), ref["out"], f"{tokens} tokens")
    with pytest.raises(binding.MoeError):
        L.ctx.moe_set_active_tokens(901)
    L.check_device_status()


def test_fused_forward_replays_from_a_cuda_graph():
    """The layer makes no host synchronisation and no allocation, so a stream capture records it and the graph
    replays it on new input values in the same buffers."""
    cfg = SMALL[5]
    L = Layer(cfg)
    ws = torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
    out = L.nan_bf16(cfg.T, cfg.H)
    x_buf, lg_buf = L.x.clone(), L.d_logits.clone()
    L.ctx.moe_fused_forward(x_buf, lg_buf, L.w_gate, L.w_up, L.w_down, out, ws)      # warm-up outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        graph.capture_begin()
        L.ctx.moe_fused_forward(x_buf, lg_buf, L.w_gate, L.w_up, L.w_down, out, ws, stream=side)
        graph.capture_end()
    torch.cuda.synchronize()
    xb = np.roll(L.x_bits, 5, axis=0).copy()
    lg = gen.make_logits(cfg, xb)
    x_buf.copy_(bits_to_dev(xb))
    lg_buf.copy_(torch.from_numpy(lg).to(DEV))
    out.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    ref = orc.forward(xb, lg, cfg.k, L.weights)
    assert_out_close(dev_bf16_to_f64(out), ref["out"], "graph replay")
    L.check_device_status()


def test_plan_from_external_topk_and_bad_ids():
    """Expert ids chosen by the caller (any router): the plan equals the oracle's plan for those ids; an id out of
    range is reported in the status word and cannot write out of bounds."""
    rng = np.random.default_rng(17)
    T, E, k = 777, 33, 5
    ids = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)      # not sorted by any score
    ctx = binding.Context(T, 64, 64, E, k)
    i32 = dict(dtype=torch.int32, device=DEV)
    d_ids = torch.from_numpy(ids).to(DEV)
    checked = torch.full((T, k), -1, **i32)
    counts, offsets = torch.full((E,), -1, **i32), torch.full((E + 1,), -1, **i32)
    perm, inv = torch.full((T * k + 1,), -7, **i32), torch.full((T * k + 1,), -7, **i32)
    ctx.moe_plan_routing_from_topk(d_ids, checked, counts, offsets, perm, inv)
    torch.cuda.synchronize()
    c, o, p, ip = orc.plan_permutation(ids, E)
    assert np.array_equal(checked.cpu().numpy(), ids)
    assert np.array_equal(counts.cpu().numpy(), c) and np.array_equal(offsets.cpu().numpy(), o)
    assert np.array_equal(perm[:-1].cpu().numpy(), p) and np.array_equal(inv[:-1].cpu().numpy(), ip)
    assert perm[-1].item() == -7 and inv[-1].item() == -7, "canaries"
    assert ctx.moe_last_device_status() == (0, 0)
    bad = ids.copy()
    bad[5, 2] = E + 3
    ctx.moe_plan_routing_from_topk(torch.from_numpy(bad).to(DEV), checked, counts, offsets, perm, inv)
    code, detail = ctx.moe_last_device_status()
    assert code == 4 and detail == 5 * k + 2, "MOE_ERR_BAD_ROUTING with the offending slot"
    assert checked[5, 2].item() == 0 and int(offsets[-1]) == T * k and perm[-1].item() == -7


def test_wide_router_and_large_batch_plans():
    """The limits of the routing plan: E = 1024 with k = 32 through the whole layer, and a 65536-token batch."""
    cfg = gen.MoEConfig("wide", T=40, H=64, F=64, E=1024, k=32, seed=111, router="iid")
    L = Layer(cfg)
    ws = torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
    out = L.nan_bf16(cfg.T, cfg.H)
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws)
    torch.cuda.synchronize()
    L.check_device_status()
    assert_out_close(dev_bf16_to_f64(out), oracle_for(L)["out"], "E=1024, k=32")
    big = gen.MoEConfig("bigT", T=65536, H=64, F=64, E=256, k=8, seed=112, router="iid")
    logits = gen.make_logits(big, None)
    Lb = Layer(big, upload_weights=False, logits=logits, x_bits=np.zeros((1, 64), np.uint16))
    Lb.plan()
    ids, w = orc.topk_route(logits, big.k)
    c, o, p, ip = orc.plan_permutation(ids, big.E)
    assert_plan_matches(Lb, dict(topk_ids=ids, topk_w=w, counts=c, offsets=o, perm=p, inv_perm=ip))
