"""CPU oracle for the interleaved Linear-1 / Linear-2 tile order (Algorithm 1).  TEST INFRASTRUCTURE ONLY.

What the scheduler does, stated as a rule rather than as a loop (Sec. 4.3, "merges the ready Linear-1 and Linear-2
tile streams"; App. A.2 for the symbols).  A row is one 128-row block of the expert-contiguous buffer; a GEMM's
tile number k lies in row k div P_i (P_1 Linear-1 tiles per row, P_2 Linear-2 tiles per row, P rows).  Instance g
of G owns the tiles g, g+G, g+2G, ... of each GEMM and never reorders tiles of the same GEMM.  What the lead D
decides is only where the Linear-2 stream is spliced into the Linear-1 stream: a Linear-2 tile of row p may go as
soon as the instance's *pending* Linear-1 tile lies in row p + D or later (or no Linear-1 tile is pending), and it
goes at the first such moment.  So the j-th Linear-2 tile of the instance is emitted after exactly

    need(j) = number of the instance's Linear-1 tiles that lie in rows < p(j) + D

Linear-1 tiles (rows are non-decreasing along the instance's list, so that count is a prefix length and need is
non-decreasing in j), and before the Linear-1 tile that follows that prefix.  The order is the merge of the two
lists by that splice position.

Pins (tests/test_schedule.py): every tile of both GEMMs is emitted exactly once over the G instances; no instance
emits a Linear-2 tile of row p while its pending Linear-1 tile lies in a row before p + D; nor later than the first
moment that allows it (greediness); a step-by-step simulation written in the test; D = 0 with one instance
degenerates to row-by-row alternation; a lead of P or more gives the Expert-Wave order (all Linear-1 first);
hand-worked small cases.
"""
from __future__ import annotations

from bisect import bisect_left


def algorithm1_order(g: int, G: int, P: int, P1: int, P2: int, D: int):
    """Emission order of scheduler instance g: list of (phase, k), phase 0 = Linear-1, 1 = Linear-2."""
    mine1 = list(range(g, P * P1, G))                  # the instance's Linear-1 tiles, in its own order
    mine2 = list(range(g, P * P2, G))
    rows1 = [k // P1 for k in mine1]                   # non-decreasing
    # splice position of each Linear-2 tile: how many Linear-1 tiles go first
    need = [bisect_left(rows1, k // P2 + D) for k in mine2]
    # merge: Linear-2 tile j sorts before the Linear-1 tile with index need[j], after the one before it
    keyed = [((n, 1, n), (0, k)) for n, k in enumerate(mine1)]
    keyed += [((need[j], 0, j), (1, k)) for j, k in enumerate(mine2)]
    return [tile for _, tile in sorted(keyed)]


def lead_knee(b_n: int, k_sm: int, h_inter: int) -> int:
    """Anti-starvation knee of the lead: ceil(b_n K_SM / (2 h_inter))."""
    return -((-b_n * k_sm) // (2 * h_inter))
