"""Pins of the Algorithm 1 oracle (CPU) and, on the GPU, the kernel's emitted tile order against it."""
import math

import numpy as np
import pytest

from oracle import schedule_oracle as so


def all_orders(G, P, P1, P2, D):
    return [so.algorithm1_order(g, G, P, P1, P2, D) for g in range(G)]


CASES = [(1, 3, 2, 1, 1), (4, 7, 5, 3, 2), (148, 37, 16, 28, 5), (148, 130, 112, 16, 1), (8, 1, 3, 2, 1),
         (5, 9, 4, 4, 0), (3, 6, 2, 5, 100), (7, 11, 3, 9, 3), (2, 5, 1, 1, 2)]


def test_every_tile_exactly_once_and_streams_keep_their_order():
    for (G, P, P1, P2, D) in CASES:
        seen = [[], []]
        for g, seq in enumerate(all_orders(G, P, P1, P2, D)):
            for ph in (0, 1):
                own = [k for q, k in seq if q == ph]
                assert own == list(range(g, P * (P1, P2)[ph], G)), "an instance walks its own stride, in order"
                seen[ph] += own
        assert sorted(seen[0]) == list(range(P * P1)) and sorted(seen[1]) == list(range(P * P2))


def test_lead_is_respected_and_linear2_goes_at_the_first_chance():
    """The two properties that, with the per-stream order above, fix the merge uniquely: a Linear-2 tile of row p
    is never emitted while the instance's pending Linear-1 tile lies before row p + D (dependency lead), and a
    Linear-1 tile is never emitted while the pending Linear-2 tile could already go (no idle Linear-2 work)."""
    for (G, P, P1, P2, D) in CASES:
        for g, seq in enumerate(all_orders(G, P, P1, P2, D)):
            l1 = [k for ph, k in seq if ph == 0]
            l2 = [k for ph, k in seq if ph == 1]
            n1 = n2 = 0                      # tiles of each stream emitted so far
            for ph, k in seq:
                pending_row1 = l1[n1] // P1 if n1 < len(l1) else math.inf
                may_go = n2 < len(l2) and l2[n2] // P2 + D <= pending_row1
                if ph == 1:
                    assert may_go, (G, P, P1, P2, D, g, k)
                    n2 += 1
                else:
                    assert not may_go, (G, P, P1, P2, D, g, k)
                    n1 += 1


def test_hand_worked_small_case():
    # one instance, 3 rows, 2 Linear-1 tiles and 1 Linear-2 tile per row, lead 1:
    # L1 row 0 (k=0,1) -> p1 = 1 -> L2 row 0 -> L1 row 1 (k=2,3) -> L2 row 1 -> L1 row 2 (k=4,5) -> L2 row 2
    assert so.algorithm1_order(0, 1, 3, 2, 1, 1) == [(0, 0), (0, 1), (1, 0), (0, 2), (0, 3), (1, 1), (0, 4), (0, 5), (1, 2)]
    # two instances, 2 rows of 2 + 2 tiles: instance 1 owns the odd tiles.  After its Linear-1 tile 1 (row 0) its
    # next Linear-1 tile is 3 (row 1), so p1 = 1 and Linear-2 tile 1 (row 0) may go: 0 + 1 <= 1; Linear-2 tile 3
    # (row 1) has to wait until the Linear-1 cursor has run off the end.
    assert so.algorithm1_order(1, 2, 2, 2, 2, 1) == [(0, 1), (1, 1), (0, 3), (1, 3)]
    assert so.algorithm1_order(0, 2, 2, 2, 2, 1) == [(0, 0), (1, 0), (0, 2), (1, 2)]


def test_zero_lead_one_instance_alternates_rows_linear2_first():
    # D = 0: a Linear-2 tile may go as soon as the pending Linear-1 tile is in its own row, so row p's Linear-2
    # tiles precede row p's Linear-1 tiles (an order no kernel may run: the data does not exist yet)
    P, P1, P2 = 3, 2, 2
    want = []
    for p in range(P):
        want += [(1, p * P2 + c) for c in range(P2)] + [(0, p * P1 + c) for c in range(P1)]
    assert so.algorithm1_order(0, 1, P, P1, P2, 0) == want


def test_large_lead_is_expert_wave_and_mix_is_preserved():
    G, P, P1, P2 = 4, 10, 6, 3
    for g in range(G):
        seq = so.algorithm1_order(g, G, P, P1, P2, D=P)
        phases = [ph for ph, _ in seq]
        assert phases == sorted(phases), "lead >= rows: all Linear-1 tiles first"
        seq1 = so.algorithm1_order(g, G, P, P1, P2, D=1)
        assert sorted(seq1) == sorted(seq), "interleaving changes the order, not the tile set"
    assert so.lead_knee(128, 148, 2048) == 5 and so.lead_knee(128, 148, 14336) == 1


@pytest.mark.gpu
def test_kernel_emits_algorithm1_order():
    import torch
    from paper_2607_23264_b200 import binding, inputs as gen
    from moe_testlib import DEV, Layer
    for cfg, D in [(gen.MoEConfig("s1", T=700, H=512, F=384, E=6, k=2, seed=41, router="xWr"), 1),
                   (gen.MoEConfig("s2", T=2000, H=256, F=640, E=40, k=4, seed=42, router="xWr_zipf"), 3)]:
        L = Layer(cfg)
        ws = torch.empty(L.ctx.workspace_bytes(), dtype=torch.uint8, device=DEV)
        out = L.nan_bf16(cfg.T, cfg.H)
        L.ctx.moe_fused_forward(L.x, L.d_logits, L.w_gate, L.w_up, L.w_down, out, ws,
                                tuning=binding.make_tuning(1, 0, 1, schedule=1, dep_lead_D=D, debug_flags=1))
        torch.cuda.synchronize()
        L.check_device_status()
        orders = L.ctx.moe_get_ffn_order()
        counts = ws[L.ctx.workspace_layout()["counts"]:][: 4 * cfg.E].view(torch.int32).cpu().numpy()
        P = int(((counts + 127) // 128).sum())
        P1, P2, G = (cfg.F + 127) // 128, (cfg.H + 255) // 256, len(orders)
        for g in range(G):
            assert orders[g] == so.algorithm1_order(g, G, P, P1, P2, D), f"CTA {g}"
