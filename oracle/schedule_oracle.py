"""CPU oracle for the interleaved Linear-1 / Linear-2 tile order (Algorithm 1).  TEST INFRASTRUCTURE ONLY.

The scheduler instance g of G walks two strided cursors.  With P rows (a row is one 128-row block of the
expert-contiguous buffer), P1 Linear-1 tiles per row and P2 Linear-2 tiles per row, tile number k of a GEMM
lies in row k div P_i.  While either cursor has tiles left: if a Linear-2 tile is left and its row p2 satisfies
p2 + D <= p1, where p1 is the row of the instance's next Linear-1 tile (infinite once Linear-1 is exhausted),
the Linear-2 tile is emitted and k2 advances by G; otherwise the Linear-1 tile is emitted and k1 advances by G.

Pins (tests/test_schedule.py): every tile of both GEMMs is emitted exactly once over the G instances; no
instance emits a Linear-2 tile of row p2 before its own Linear-1 cursor has passed row p2 + D - 1; D = 0 with one
instance degenerates to row-by-row alternation starting with Linear-2's wait for Linear-1; a lead of P or more
gives the Expert-Wave order (all Linear-1 first); hand-worked small cases.
"""
from __future__ import annotations

import math


def algorithm1_order(g: int, G: int, P: int, P1: int, P2: int, D: int):
    """Emission order of scheduler instance g: list of (phase, k), phase 0 = Linear-1, 1 = Linear-2."""
    k1 = k2 = g
    out = []
    while k1 < P * P1 or k2 < P * P2:
        p1 = k1 // P1 if k1 < P * P1 else math.inf
        p2 = k2 // P2
        if k2 < P * P2 and p2 + D <= p1:
            out.append((1, k2))
            k2 += G
        else:
            out.append((0, k1))
            k1 += G
    return out


def lead_knee(b_n: int, k_sm: int, h_inter: int) -> int:
    """Anti-starvation knee of the lead: ceil(b_n K_SM / (2 h_inter))."""
    return -((-b_n * k_sm) // (2 * h_inter))
