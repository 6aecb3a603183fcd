"""Router front end on the GPU against the oracle: logits within the fp32-accumulation bound, the selection
bit-exact on the logits the GPU computed and admissible with respect to the exact logits, the plan bit-exact."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle, router_oracle
from paper_2607_23264_b200 import binding, inputs as gen
from moe_testlib import DEV, TOL_W, Layer, assert_out_close, bits_to_dev, dev_bf16_to_f64, dev_to_bits

pytestmark = pytest.mark.gpu

# |logit_gpu - logit_fp64| <= TOL_LOGIT * (1 + |logit|): the products are exact; what is left is the tensor pipe's
# fp32 accumulation over 2H/16 instructions per K split (addends are aligned and truncated, not rounded to nearest, so
# the error grows with the length: about 6e-5 at H = 7168), the bits below the second bf16 term of W_r (relative
# 2^-17 per weight, about 5e-6 on a logit) and the fp32 sums of the split partials and the bias.
TOL_LOGIT = 1e-4


class RouterCase:
    def __init__(self, T, H, E, k, seed, bias=False, F=64):
        self.cfg = gen.MoEConfig(name="router", T=T, H=H, F=F, E=E, k=k, seed=seed, router="xWr")
        self.x_bits = gen.make_x(self.cfg)
        self.w_router = gen.make_router(self.cfg)
        self.bias = gen.zipf_log_bias(E).astype(np.float32) if bias else None
        self.ctx = binding.Context(T, H, F, E, k)
        self.x = bits_to_dev(self.x_bits)
        self.d_w = torch.from_numpy(self.w_router).to(DEV)
        self.d_bias = torch.from_numpy(self.bias).to(DEV) if bias else None
        self.w_split = torch.zeros(self.ctx.router_weight_bytes() // 2, dtype=torch.bfloat16, device=DEV)
        self.scratch = torch.full((max(self.ctx.router_scratch_bytes(), 16) // 4,), float("nan"), device=DEV)
        self.ctx.moe_router_prepare(self.d_w, self.w_split)
        i32 = dict(dtype=torch.int32, device=DEV)
        R = T * k
        self.logits = torch.full((T, E), float("nan"), device=DEV)
        self.topk_ids = torch.full((T, k), -1, **i32)
        self.topk_w = torch.full((T, k), float("nan"), device=DEV)
        self.counts = torch.full((E,), -1, **i32)
        self.offsets = torch.full((E + 1,), -1, **i32)
        self.perm = torch.full((R,), -1, **i32)
        self.inv_perm = torch.full((R,), -1, **i32)

    def route(self, want_logits=True):
        self.ctx.moe_route_tokens(self.x, self.w_split, self.d_bias, self.scratch, self.logits if want_logits else None,
                                  self.topk_ids, self.topk_w, self.counts, self.offsets, self.perm, self.inv_perm)
        torch.cuda.synchronize()
        code, detail = self.ctx.moe_last_device_status()
        assert code == 0, (code, detail)

    def check(self):
        cfg = self.cfg
        exact = router_oracle.router_logits(self.x_bits, self.w_router, self.bias)
        g = self.logits.cpu().numpy()
        assert np.isfinite(g).all()
        err = np.abs(g.astype(np.float64) - exact)
        worst = float((err / (TOL_LOGIT * (1.0 + np.abs(exact)))).max())
        assert worst <= 1.0, f"logits: max err / bound = {worst:.3f}"
        # the selection is an integer decision taken on the GPU's own fp32 logits: bit-exact against the oracle on them
        ids_ref, w_ref = moe_oracle.topk_route(g, cfg.k)
        ids = self.topk_ids.cpu().numpy()
        assert np.array_equal(ids, ids_ref)
        assert np.abs(self.topk_w.cpu().numpy().astype(np.float64) - w_ref).max() <= TOL_W
        counts, offsets, perm, inv_perm = moe_oracle.plan_permutation(ids_ref, cfg.E)
        assert np.array_equal(self.counts.cpu().numpy(), counts)
        assert np.array_equal(self.offsets.cpu().numpy(), offsets)
        assert np.array_equal(self.perm.cpu().numpy(), perm)
        assert np.array_equal(self.inv_perm.cpu().numpy(), inv_perm)
        # and with respect to the exact logits it is what logits this accurate can give
        eps = err.max(axis=1)
        assert router_oracle.admissible_selection(exact, ids, eps).all()
        ids_exact, _ = moe_oracle.topk_route(exact, cfg.k)
        flipped = int((ids != ids_exact).any(axis=1).sum())
        assert flipped <= max(1, cfg.T // 100), f"{flipped} of {cfg.T} tokens route differently from the fp64 logits"
        return flipped, float(err.max())


def _np_split(w_router, EpT):
    H, E = w_router.shape
    w = np.zeros((EpT, H), dtype=np.float32)
    w[:E] = w_router.T
    terms = []
    rem = w
    for _ in range(2):
        b = gen.f32_to_bf16_bits(rem)
        terms.append(b)
        rem = rem - gen.bf16_bits_to_f32(b)
    return np.stack(terms)


@pytest.mark.parametrize("T,H,E", [(5, 64, 3), (40, 192, 17), (16, 128, 128), (33, 256, 130), (9, 64, 300)])
def test_router_prepare_bits(T, H, E):
    c = RouterCase(T, H, E, 1, seed=11)
    torch.cuda.synchronize()
    EpT = c.ctx.router_weight_bytes() // (2 * H * 2)
    assert EpT >= E and EpT % 16 == 0
    got = dev_to_bits(c.w_split).reshape(2, EpT, H)
    assert np.array_equal(got, _np_split(c.w_router, EpT))


@pytest.mark.parametrize("T,H,E,k,bias", [
    (128, 256, 8, 2, False),       # the tiny layer
    (1, 64, 2, 1, False),          # one token, one K block
    (127, 192, 3, 3, True),        # ragged row tile, k = E
    (129, 320, 17, 4, True),       # two row tiles, second nearly empty
    (300, 512, 64, 8, False),
    (257, 448, 130, 6, True),      # two column tiles, second ragged
    (515, 1024, 256, 8, True),
    (64, 256, 300, 32, False),     # three column tiles, k = 32
    (2000, 128, 40, 5, True),      # more row tiles than a K split can use
])
def test_route_tokens_parity(T, H, E, k, bias):
    c = RouterCase(T, H, E, k, seed=T + E, bias=bias)
    c.route()
    c.check()


def test_route_tokens_is_deterministic_and_matches_plan_routing():
    c = RouterCase(700, 512, 96, 4, seed=3, bias=True)
    c.route()
    first = [t.clone() for t in (c.logits, c.topk_ids, c.topk_w, c.perm)]
    for _ in range(3):
        c.route()
        for a, b in zip(first, (c.logits, c.topk_ids, c.topk_w, c.perm)):
            assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    # moe_plan_routing on the returned logits gives the same plan bit for bit
    ids2, w2 = torch.empty_like(c.topk_ids), torch.empty_like(c.topk_w)
    counts2, offsets2 = torch.empty_like(c.counts), torch.empty_like(c.offsets)
    perm2, inv2 = torch.empty_like(c.perm), torch.empty_like(c.inv_perm)
    c.ctx.moe_plan_routing(c.logits, ids2, w2, counts2, offsets2, perm2, inv2)
    torch.cuda.synchronize()
    assert torch.equal(ids2, c.topk_ids) and torch.equal(w2.view(torch.int32), c.topk_w.view(torch.int32))
    assert torch.equal(counts2, c.counts) and torch.equal(offsets2, c.offsets)
    assert torch.equal(perm2, c.perm) and torch.equal(inv2, c.inv_perm)
    # logits_out is optional
    c.topk_ids.fill_(-1)
    c.route(want_logits=False)
    assert torch.equal(c.topk_ids, first[1])


@pytest.mark.parametrize("name,T,H,E,k,bias", [("C2", 8192, 4096, 8, 2, False), ("C3", 4096, 7168, 256, 8, True)])
def test_route_tokens_full_size(name, T, H, E, k, bias):
    c = RouterCase(T, H, E, k, seed=1 if name == "C2" else 2, bias=bias)
    c.route()
    flipped, worst = c.check()
    print(f"{name}: {flipped} tokens differ from the fp64 selection, max |dlogit| = {worst:.2e}")


def test_fused_forward_routed_matches_fused_forward_on_the_same_logits():
    cfg = gen.CONFIGS["C1"]
    layer = Layer(cfg)
    ctx = layer.ctx
    w_router = gen.make_router(cfg)
    d_w = torch.from_numpy(w_router).to(DEV)
    w_split = torch.zeros(ctx.router_weight_bytes() // 2, dtype=torch.bfloat16, device=DEV)
    scratch = torch.empty(ctx.router_scratch_bytes() // 4, device=DEV)
    ctx.moe_router_prepare(d_w, w_split)
    ws = torch.empty(ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
    out = layer.nan_bf16(cfg.T, cfg.H)
    ctx.moe_fused_forward_routed(layer.x, w_split, None, layer.w_gate, layer.w_up, layer.w_down, out, ws, scratch)
    torch.cuda.synchronize()
    layer.check_device_status()
    # the logits the router used, through the stand-alone call
    logits = torch.empty((cfg.T, cfg.E), device=DEV)
    ctx.moe_route_tokens(layer.x, w_split, None, scratch, logits, layer.topk_ids, layer.topk_w, layer.counts,
                         layer.offsets, layer.perm, layer.inv_perm)
    out2 = layer.nan_bf16(cfg.T, cfg.H)
    ctx.moe_fused_forward(layer.x, logits, layer.w_gate, layer.w_up, layer.w_down, out2, ws)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
    ref = moe_oracle.forward(layer.x_bits, logits.cpu().numpy(), cfg.k, layer.weights)
    assert_out_close(dev_bf16_to_f64(out), ref["out"], "routed forward")


def test_router_argument_errors():
    c = RouterCase(64, 128, 8, 2, seed=5)
    small = torch.empty(4, device=DEV)
    with pytest.raises(binding.MoeError) as e:
        c.ctx.moe_route_tokens(c.x, c.w_split, None, small, None, c.topk_ids, c.topk_w, c.counts, c.offsets, c.perm,
                               c.inv_perm)
    assert e.value.code == 3
    with pytest.raises(binding.MoeError) as e:
        c.ctx.moe_route_tokens(None, c.w_split, None, c.scratch, None, c.topk_ids, c.topk_w, c.counts, c.offsets,
                               c.perm, c.inv_perm)
    assert e.value.code == 1
    with pytest.raises(binding.MoeError) as e:
        c.ctx.moe_router_prepare(None, c.w_split)
    assert e.value.code == 1
    # an empty batch writes zero counts and offsets and launches nothing
    c.ctx.moe_set_active_tokens(0)
    c.ctx.moe_route_tokens(c.x, c.w_split, None, c.scratch, None, c.topk_ids, c.topk_w, c.counts, c.offsets, c.perm,
                           c.inv_perm)
    torch.cuda.synchronize()
    assert int(c.counts.abs().sum()) == 0 and int(c.offsets.abs().sum()) == 0
    assert c.ctx.moe_last_launch_count() == 0


def test_router_smaller_batches_on_one_context():
    c = RouterCase(300, 256, 24, 3, seed=17, bias=True)
    c.route()
    full_ids = c.topk_ids.clone()
    full_logits = c.logits.clone()
    for tokens in (129, 128, 7):
        c.ctx.moe_set_active_tokens(tokens)
        c.topk_ids.fill_(-1)
        c.logits.fill_(float("nan"))
        c.ctx.moe_route_tokens(c.x, c.w_split, c.d_bias, c.scratch, c.logits, c.topk_ids, c.topk_w, c.counts, c.offsets,
                               c.perm, c.inv_perm)
        torch.cuda.synchronize()
        code, _ = c.ctx.moe_last_device_status()
        assert code == 0
        # rows are independent and the K split is the same for every batch size here (H = 256 has four K blocks,
        # which caps the split at 4), so the first `tokens` tokens get the same logit bits as in the full batch
        ids = c.topk_ids.view(-1)[: tokens * 3].view(tokens, 3)
        assert torch.equal(ids, full_ids[:tokens])
        lg = c.logits.view(-1)[: tokens * 24].view(tokens, 24)
        assert torch.equal(lg.view(torch.int32), full_logits[:tokens].view(torch.int32))
        counts, offsets, perm, inv_perm = moe_oracle.plan_permutation(ids.cpu().numpy(), 24)
        assert np.array_equal(c.counts.cpu().numpy(), counts)
        assert np.array_equal(c.perm.cpu().numpy()[: tokens * 3], perm)
    c.ctx.moe_set_active_tokens(300)
