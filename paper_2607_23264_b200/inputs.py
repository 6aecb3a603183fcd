"""Seeded synthetic inputs for the single-GPU (EP=1) MoE forward path.

This module only *draws numbers*: token activations, router matrices, router
logits and expert weights, with the shapes and distributions of the five
workloads the library is measured on.  It contains none of the method's
arithmetic (no top-k, no permutation, no expert FFN, no combine) so that the
CPU oracle and the CUDA path can both be fed from it without sharing code.

Conventions
-----------
* bf16 tensors are carried as ``numpy.uint16`` bit patterns (numpy has no
  bfloat16).  Conversion from fp32 is round-to-nearest-even.
* ``N(0, 1/sqrt(fan_in))`` is read as *standard deviation* ``1/sqrt(fan_in)``:
  fan_in = H for the gate, up and router matrices, F for the down matrix.
* Every tensor has its own random stream: ``PCG64DXSM(SeedSequence([seed,
  tensor_id, expert]))``, so any expert's weights can be regenerated on demand
  without materialising the other experts (the DeepSeek-V3-like layer holds
  22.5 GB of bf16 weights).
* Router logits are computed once, on the CPU, in fp64 and rounded to fp32;
  the same fp32 array is then handed to every consumer, so that top-k
  selection is a pure comparison of identical numbers on both sides.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
import os

import numpy as np

_T_X, _T_ROUTER, _T_NOISE, _T_GATE, _T_UP, _T_DOWN = 0, 1, 2, 3, 4, 5


@dataclass(frozen=True)
class MoEConfig:
    """One MoE layer workload: T tokens, hidden H, per-expert ffn F, E experts, top-k."""
    name: str
    T: int
    H: int
    F: int
    E: int
    k: int
    seed: int
    router: str  # "xWr": logits = x.W_r ; "xWr_zipf": + Zipf(1.1) log-bias ; "iid": logits ~ N(0,1)

    @property
    def R(self) -> int:
        """Number of (token, slot) assignments = rows of the expert-contiguous buffers."""
        return self.T * self.k

    @property
    def flops(self) -> int:
        """Algorithmic flops of the three expert projections: 6.R.H.F."""
        return 6 * self.R * self.H * self.F


CONFIGS = {
    # tiny layer, the oracle runs it in well under a second
    "C1": MoEConfig("C1", T=128, H=256, F=512, E=8, k=2, seed=0, router="xWr"),
    # Mixtral-like layer, near-uniform expert loads
    "C2": MoEConfig("C2", T=8192, H=4096, F=14336, E=8, k=2, seed=1, router="xWr"),
    # DeepSeek-V3-like fine-grained layer, skewed loads with empty experts
    "C3": MoEConfig("C3", T=4096, H=7168, F=2048, E=256, k=8, seed=2, router="xWr_zipf"),
    # decode-like small batch, uniform-random routing
    "C4": MoEConfig("C4", T=64, H=7168, F=2048, E=256, k=8, seed=3, router="iid"),
    # profiler-sized cases (small device footprint, still larger than L2):
    # P1 = two Mixtral-like experts at C2's rows per expert (a quarter of C2's grouped-GEMM work)
    "P1": MoEConfig("P1", T=2048, H=4096, F=14336, E=2, k=2, seed=4, router="xWr"),
    # P2 = C2's row movers (dispatch/combine traffic of a 16384-token batch) with token-sized experts
    "P2": MoEConfig("P2", T=16384, H=4096, F=64, E=8, k=2, seed=5, router="xWr"),
    # P3 = a slice of the DeepSeek-V3-like layer: the same expert shape and skewed routing over 32 experts (2.8 GB of
    # weights), which mixes many-row experts, single-block experts and swapped-operand tiles in one launch
    "P3": MoEConfig("P3", T=256, H=7168, F=2048, E=32, k=8, seed=6, router="xWr_zipf"),
}


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round-to-nearest-even.  Inputs are finite."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> fp32, exact."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, tensor_id: int, expert: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64DXSM(np.random.SeedSequence([seed, tensor_id, expert])))


def _normal_bf16(rng: np.random.Generator, shape, std: float) -> np.ndarray:
    a = rng.standard_normal(shape, dtype=np.float32)
    a *= np.float32(std)
    return f32_to_bf16_bits(a)


def make_x(cfg: MoEConfig) -> np.ndarray:
    """Token activations x[T,H] ~ N(0,1), bf16 bits."""
    return _normal_bf16(_rng(cfg.seed, _T_X), (cfg.T, cfg.H), 1.0)


def make_router(cfg: MoEConfig) -> np.ndarray:
    """Router matrix W_r[H,E] ~ N(0, std 1/sqrt(H)), fp32."""
    w = _rng(cfg.seed, _T_ROUTER).standard_normal((cfg.H, cfg.E), dtype=np.float32)
    return w * np.float32(1.0 / np.sqrt(cfg.H))


def zipf_log_bias(E: int, s: float = 1.1) -> np.ndarray:
    """Per-expert logit bias = log of the unnormalised Zipf(s) mass of expert index e (zero-based)."""
    return -s * np.log(np.arange(1, E + 1, dtype=np.float64))


def make_logits(cfg: MoEConfig, x_bits: np.ndarray) -> np.ndarray:
    """Router logits[T,E] fp32.  Produced once here; never recomputed by a consumer."""
    if cfg.router == "iid":
        return _rng(cfg.seed, _T_NOISE).standard_normal((cfg.T, cfg.E), dtype=np.float32)
    x64 = bf16_bits_to_f32(x_bits).astype(np.float64)
    logits = x64 @ make_router(cfg).astype(np.float64)
    if cfg.router == "xWr_zipf":
        logits = logits + zipf_log_bias(cfg.E)[None, :]
    elif cfg.router != "xWr":
        raise ValueError(f"unknown router recipe {cfg.router!r}")
    return logits.astype(np.float32)


def expert_weights(cfg: MoEConfig, e: int):
    """Weights of expert e as bf16 bits: (W_gate[F,H], W_up[F,H], W_down[H,F])."""
    s_in = 1.0 / np.sqrt(cfg.H)
    s_mid = 1.0 / np.sqrt(cfg.F)
    wg = _normal_bf16(_rng(cfg.seed, _T_GATE, e), (cfg.F, cfg.H), s_in)
    wu = _normal_bf16(_rng(cfg.seed, _T_UP, e), (cfg.F, cfg.H), s_in)
    wd = _normal_bf16(_rng(cfg.seed, _T_DOWN, e), (cfg.H, cfg.F), s_mid)
    return wg, wu, wd


def default_threads() -> int:
    return max(1, min(32, os.cpu_count() or 1))


def for_each_expert(cfg: MoEConfig, sink, threads: int | None = None) -> None:
    """Generate every expert's weights (thread pool) and hand them to ``sink(e, wg, wu, wd)``.

    ``sink`` is called from the calling thread, in expert order, so it may copy
    into a preallocated (host or device) tensor without holding all experts.
    """
    threads = threads or default_threads()
    with ThreadPoolExecutor(max_workers=threads) as pool:
        window = 2 * threads
        pending = {}
        nxt = 0
        for e in range(cfg.E):
            while nxt < cfg.E and len(pending) < window:
                pending[nxt] = pool.submit(expert_weights, cfg, nxt)
                nxt += 1
            wg, wu, wd = pending.pop(e).result()
            sink(e, wg, wu, wd)


def stacked_weights(cfg: MoEConfig, threads: int | None = None):
    """All experts stacked on the host: W_gate[E,F,H], W_up[E,F,H], W_down[E,H,F] (bf16 bits)."""
    wg = np.empty((cfg.E, cfg.F, cfg.H), dtype=np.uint16)
    wu = np.empty((cfg.E, cfg.F, cfg.H), dtype=np.uint16)
    wd = np.empty((cfg.E, cfg.H, cfg.F), dtype=np.uint16)

    def sink(e, g, u, d):
        wg[e], wu[e], wd[e] = g, u, d

    for_each_expert(cfg, sink, threads)
    return wg, wu, wd


def random_small_config(rng: np.random.Generator, **fixed) -> MoEConfig:
    """A random small layer for property tests (ragged expert loads, several tiles)."""
    E = int(fixed.get("E", rng.integers(1, 12)))
    k = int(fixed.get("k", rng.integers(1, min(E, 4) + 1)))
    return MoEConfig(
        name="rand",
        T=int(fixed.get("T", rng.integers(1, 400))),
        H=int(fixed.get("H", 64 * rng.integers(1, 5))),
        F=int(fixed.get("F", 64 * rng.integers(1, 6))),
        E=E, k=k,
        seed=int(fixed.get("seed", rng.integers(0, 2**31))),
        router=str(fixed.get("router", "xWr")),
    )


class WeightStream:
    """``weights(e)`` callable that regenerates experts on demand instead of holding them.

    ``order`` is the ascending list of experts the consumer will ask for; the next few are generated
    ahead of time on a thread pool.  Asking for an expert outside ``order`` generates it on the spot.
    """

    def __init__(self, cfg: MoEConfig, order, threads: int | None = None):
        self.cfg = cfg
        self.order = [int(e) for e in order]
        self.pos = {e: i for i, e in enumerate(self.order)}
        self.pool = ThreadPoolExecutor(max_workers=threads or default_threads())
        self.ahead = 2 * (threads or default_threads())
        self.pending = {}
        self.next_submit = 0

    def _fill(self, upto: int):
        while self.next_submit < min(len(self.order), upto):
            e = self.order[self.next_submit]
            self.pending[e] = self.pool.submit(expert_weights, self.cfg, e)
            self.next_submit += 1

    def __call__(self, e: int):
        e = int(e)
        if e not in self.pos:
            return expert_weights(self.cfg, e)
        self._fill(self.pos[e] + 1 + self.ahead)
        fut = self.pending.pop(e, None)
        return fut.result() if fut is not None else expert_weights(self.cfg, e)

    def close(self):
        self.pool.shutdown(wait=False, cancel_futures=True)
