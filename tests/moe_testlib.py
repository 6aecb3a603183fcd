"""Shared helpers of the GPU parity tests: upload seeded inputs, call the C ABI, compare with the oracle."""
from __future__ import annotations

import numpy as np
import torch

from paper_2607_23264_b200 import binding, inputs as gen

# Acceptance bars (stated by the workload definition): indices bit-exact; routing weights |d| <= 1e-6;
# bf16 outputs max|gpu-ref| <= 2e-2 (1+|ref|); intermediate activations relative Frobenius error <= 5e-3.
TOL_W = 1e-6
TOL_OUT = 2e-2
TOL_FRO = 5e-3

DEV = "cuda:0"


def bits_to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor on the device (same bytes)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(DEV).view(torch.bfloat16)


def dev_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def dev_bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return gen.bf16_bits_to_f32(dev_to_bits(t)).astype(np.float64)


def rel_fro(a: np.ndarray, ref: np.ndarray) -> float:
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(a - ref) / den) if den > 0 else float(np.linalg.norm(a))


def assert_out_close(got: np.ndarray, ref: np.ndarray, what: str):
    err = np.abs(got - ref)
    bound = TOL_OUT * (1.0 + np.abs(ref))
    worst = float((err / bound).max()) if err.size else 0.0
    assert worst <= 1.0, f"{what}: max |gpu-ref| / (2e-2 (1+|ref|)) = {worst:.3f}"


class Layer:
    """A layer's inputs on host and device plus device buffers for every intermediate."""

    def __init__(self, cfg: gen.MoEConfig, keep_experts=None, upload_weights=True, logits=None, x_bits=None):
        self.cfg = cfg
        T, H, F, E, k = cfg.T, cfg.H, cfg.F, cfg.E, cfg.k
        self.x_bits = gen.make_x(cfg) if x_bits is None else x_bits
        self.logits = gen.make_logits(cfg, self.x_bits) if logits is None else logits
        self.kept = {}
        self.ctx = binding.Context(T, H, F, E, k)
        self.x = bits_to_dev(self.x_bits)
        self.d_logits = torch.from_numpy(self.logits).to(DEV)
        if upload_weights:
            self.w_gate = torch.empty((E, F, H), dtype=torch.bfloat16, device=DEV)
            self.w_up = torch.empty((E, F, H), dtype=torch.bfloat16, device=DEV)
            self.w_down = torch.empty((E, H, F), dtype=torch.bfloat16, device=DEV)

            def sink(e, g, u, d):
                self.w_gate[e].copy_(torch.from_numpy(g.view(np.int16)).view(torch.bfloat16))
                self.w_up[e].copy_(torch.from_numpy(u.view(np.int16)).view(torch.bfloat16))
                self.w_down[e].copy_(torch.from_numpy(d.view(np.int16)).view(torch.bfloat16))
                if keep_experts is None or e in keep_experts:
                    self.kept[e] = (g, u, d)

            gen.for_each_expert(cfg, sink)
        R = cfg.R
        i32 = dict(dtype=torch.int32, device=DEV)
        self.topk_ids = torch.full((T, k), -1, **i32)
        self.topk_w = torch.full((T, k), float("nan"), dtype=torch.float32, device=DEV)
        self.counts = torch.full((E,), -1, **i32)
        self.offsets = torch.full((E + 1,), -1, **i32)
        self.perm = torch.full((R,), -1, **i32)
        self.inv_perm = torch.full((R,), -1, **i32)

    def weights(self, e):
        return self.kept[e]

    def nan_bf16(self, *shape):
        """bf16 buffer poisoned with NaN so that rows a kernel failed to write are caught."""
        return torch.full(shape, float("nan"), dtype=torch.bfloat16, device=DEV)

    def plan(self):
        self.ctx.moe_plan_routing(self.d_logits, self.topk_ids, self.topk_w, self.counts, self.offsets, self.perm,
                                  self.inv_perm)
        torch.cuda.synchronize()

    def check_device_status(self):
        code, detail = self.ctx.moe_last_device_status()
        assert code == 0, f"device status {binding.STATUS_NAMES.get(code, code)} detail {detail:#x}"


def assert_plan_matches(layer: Layer, ref: dict):
    """Routing outputs against the oracle: indices bit-exact, weights within 1e-6."""
    for name in ("topk_ids", "counts", "offsets", "perm", "inv_perm"):
        got = getattr(layer, name).cpu().numpy()
        exp = np.asarray(ref[name]).reshape(got.shape)
        assert got.dtype == np.int32
        assert np.array_equal(got, exp), f"{name} differs from the oracle"
    w = layer.topk_w.cpu().numpy().astype(np.float64)
    assert np.abs(w - ref["topk_w"]).max() <= TOL_W


def stratified_rows(cfg: gen.MoEConfig, plan: dict, seed: int) -> np.ndarray:
    """Rows of the expert-contiguous buffer that between them touch every tile class of the grouped GEMMs:
    the first and the last row of every non-empty expert, and one seeded-random row inside every 128-row block of
    every expert.  A 128-row block is the unit every variant of the kernel is built from: each half of a 256-row
    CTA-pair tile is one block, a block with few rows is a swapped-operand tile, the short last block of a larger
    expert is its own tile; so no tile of the launch is left without a checked row."""
    rng = np.random.default_rng(seed)
    offsets = plan["offsets"]
    rows = []
    for e in range(cfg.E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi == lo:
            continue
        rows += [lo, hi - 1]
        for b0 in range(lo, hi, 128):
            rows.append(int(rng.integers(b0, min(b0 + 128, hi))))
    return np.unique(np.array(rows, dtype=np.int64))


def stratified_tokens(cfg: gen.MoEConfig, plan: dict, n_random: int, seed: int):
    """(tokens, rows): the owners of stratified_rows plus n_random seeded-random tokens, ascending."""
    rows = stratified_rows(cfg, plan, seed)
    rng = np.random.default_rng(seed + 1)
    toks = set((plan["perm"][rows].astype(np.int64) // cfg.k).tolist())
    toks.update(rng.choice(cfg.T, size=min(n_random, cfg.T), replace=False).tolist())
    return np.array(sorted(toks), dtype=np.int64), rows


def assert_rows_close(got: np.ndarray, ref: np.ndarray, what: str, tol: float = TOL_FRO):
    """Relative Frobenius error over all rows together and of every row on its own."""
    assert rel_fro(got, ref) <= tol, f"{what}: relative Frobenius error {rel_fro(got, ref):.2e}"
    num = np.linalg.norm(got - ref, axis=1)
    den = np.maximum(np.linalg.norm(ref, axis=1), 1e-30)
    worst = int(np.argmax(num / den))
    assert (num / den).max() <= tol, f"{what}: row {worst} has relative error {(num / den).max():.2e}"
