"""GPU parity at the full workload sizes, in the launch configuration bench.py times.

The routing plan and the dispatch copy are compared in full (they are cheap for the oracle).  The
expert FFN and the output are compared on sampled tokens: a token's output depends only on its own row,
its routing and the weights (pinned by test_row_independence_justifies_sampled_oracle), so the oracle
computes exactly those rows one by one."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as orc
from paper_2607_23264_b200 import inputs as gen
from paper_2607_23264_b200 import binding
from moe_testlib import (DEV, Layer, assert_out_close, assert_rows_close, dev_bf16_to_f64, dev_to_bits,
                         stratified_tokens)

pytestmark = pytest.mark.gpu


def run_sampled(cfg, n_random):
    x_bits = gen.make_x(cfg)
    logits = gen.make_logits(cfg, x_bits)
    ids, w = orc.topk_route(logits, cfg.k)
    counts, offsets, perm, inv = orc.plan_permutation(ids, cfg.E)
    plan = dict(topk_ids=ids, topk_w=w, counts=counts, offsets=offsets, perm=perm, inv_perm=inv)
    toks, strat_rows = stratified_tokens(cfg, plan, n_random, seed=cfg.seed + 100)
    L = Layer(cfg, keep_experts=set(), x_bits=x_bits, logits=logits)

    lay = L.ctx.workspace_layout()
    ws = torch.empty(lay["total"], dtype=torch.uint8, device=DEV)
    out = L.nan_bf16(cfg.T, cfg.H)
    for _ in range(2):
        L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws)
    torch.cuda.synchronize()
    L.check_device_status()

    R = cfg.R

    def sl(name, count, dtype):
        nbytes = count * torch.empty((), dtype=dtype).element_size()
        return ws[lay[name]:lay[name] + nbytes].view(dtype)

    for name, count in (("topk_ids", R), ("counts", cfg.E), ("offsets", cfg.E + 1), ("perm", R), ("inv_perm", R)):
        assert np.array_equal(sl(name, count, torch.int32).cpu().numpy(), np.asarray(plan[name]).reshape(-1)), name
    assert np.abs(sl("topk_w", R, torch.float32).cpu().numpy() - w.reshape(-1)).max() <= 1e-6
    x_perm = dev_to_bits(sl("x_perm", R * cfg.H, torch.bfloat16)).reshape(R, cfg.H)
    assert np.array_equal(x_perm, orc.dispatch(x_bits, perm, cfg.k)), "x_perm"
    del x_perm

    stream = gen.WeightStream(cfg, np.unique(ids[toks]))     # regenerates the experts the sample touches
    ref = orc.forward_tokens(toks, x_bits, logits, cfg.k, stream)
    stream.close()
    # the checked rows (all k rows of every sampled token) leave no 128-row block of any expert out: every tile of
    # both launches, each half of a CTA-pair tile and every swapped-operand tile included, holds a compared row
    checked = np.zeros(R, dtype=bool)
    checked[ref["rows"].reshape(-1)] = True
    assert checked[strat_rows].all()
    for e in range(cfg.E):
        for b0 in range(int(offsets[e]), int(offsets[e + 1]), 128):
            assert checked[b0:min(b0 + 128, int(offsets[e + 1]))].any(), f"block at row {b0} of expert {e} unsampled"
        if offsets[e + 1] > offsets[e]:
            assert checked[offsets[e]] and checked[offsets[e + 1] - 1]
    rows = torch.from_numpy(ref["rows"].reshape(-1)).to(DEV)
    h_dev = sl("h", R * cfg.F, torch.bfloat16).view(R, cfg.F)[rows]
    y_dev = sl("y_perm", R * cfg.H, torch.bfloat16).view(R, cfg.H)[rows]
    assert_rows_close(dev_bf16_to_f64(h_dev), ref["h"].reshape(-1, cfg.F), f"h[{cfg.name}]")
    assert_rows_close(dev_bf16_to_f64(y_dev), ref["y"].reshape(-1, cfg.H), f"y_perm[{cfg.name}]")
    out_np = dev_bf16_to_f64(out)
    assert np.isfinite(out_np).all(), "every token row must be written"
    assert_out_close(out_np[toks], ref["out"], f"out[{cfg.name}] on {len(toks)} sampled tokens")

    # the interleaved order (Algorithm 1, one launch with ready counters) must give the same bits at full size
    out1 = L.nan_bf16(cfg.T, cfg.H)
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out1, ws,
                            tuning=binding.make_tuning(1, 0, 1, schedule=1, dep_lead_D=8))
    torch.cuda.synchronize()
    L.check_device_status()
    assert torch.equal(out1.view(torch.int16), out.view(torch.int16)), "schedule 1 differs from schedule 0"
    return L, plan


def test_c2_mixtral_like_sampled():
    cfg = gen.CONFIGS["C2"]
    _, plan = run_sampled(cfg, n_random=32)
    c = plan["counts"]
    assert c.min() > 0.8 * cfg.R / cfg.E and c.max() < 1.2 * cfg.R / cfg.E, "near-uniform expert loads"


def test_c2_layer_at_2048_tokens_runs_256_row_tiles():
    """The Mixtral-like layer at a serving batch of 2048 tokens: about 512 rows per expert, too few for CTA pairs, so
    the single-CTA kernel runs it and cuts every expert into 256-row tiles on both accumulators (the rows sampled in
    every 128-row block fall into both halves of every such tile)."""
    import dataclasses
    cfg = dataclasses.replace(gen.CONFIGS["C2"], name="C2@T=2048", T=2048)
    L, plan = run_sampled(cfg, n_random=16)
    c = plan["counts"]
    assert c.min() > 256 and c.max() < 1024, "several 128-row blocks per expert, fewer than the CTA-pair threshold"
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, L.nan_bf16(cfg.T, cfg.H),
                            torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV),
                            tuning=binding.make_tuning(debug_flags=1))
    tr = L.ctx.moe_get_ffn_trace()
    wide_blocks = int(((c + 255) // 256).sum())
    assert tr[0, :, 6].sum() == wide_blocks * (cfg.F // 128), "Linear-1 ran one tile per 256-row block and column tile"


def test_c3_deepseek_like_sampled():
    cfg = gen.CONFIGS["C3"]
    _, plan = run_sampled(cfg, n_random=16)
    c = plan["counts"]
    assert (c == 0).sum() > 0 and c.max() > 8 * cfg.R / cfg.E, "skewed loads with empty experts"


def test_c4_decode_like_full():
    cfg = gen.CONFIGS["C4"]
    # every token is sampled: the oracle runs the whole (45 GFLOP) layer
    x_bits = gen.make_x(cfg)
    logits = gen.make_logits(cfg, x_bits)
    ids, w = orc.topk_route(logits, cfg.k)
    counts, offsets, perm, inv = orc.plan_permutation(ids, cfg.E)
    assert np.median(counts) <= 3, "most experts get 0-3 rows"
    L = Layer(cfg, keep_experts=set(), x_bits=x_bits, logits=logits)
    ws = torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
    out = L.nan_bf16(cfg.T, cfg.H)
    L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws)
    torch.cuda.synchronize()
    L.check_device_status()
    stream = gen.WeightStream(cfg, np.unique(ids))
    ref = orc.forward_tokens(np.arange(cfg.T), x_bits, logits, cfg.k, stream)
    stream.close()
    assert_out_close(dev_bf16_to_f64(out), ref["out"], "out[C4]")
