"""CPU oracle for the X-Stage (Burst-Gap) calculator.  TEST INFRASTRUCTURE ONLY.

Plain Python floats (IEEE double), one function per equation, written from the paper's definitions; it shares
nothing with the C implementation in the library.  Pins (tests/test_xstage_model.py,
tests/golden/xstage_paper_numbers.txt): the numbers the paper prints (Q of about 4.25 MiB from the 33 KiB knee;
the FlashAttention-4 audit: 4.6 MiB burst, b_iso of about 4.1 MiB, G* = 6.0 us, M_ub of about 1.0K), the
equivalences the paper states for homogeneous patterns (rho <= 1, delta_b <= 0 and G >= G* coincide; all
rho_n <= 1 keeps q at zero) and a brute-force fluid simulation of the drain.
"""
from __future__ import annotations

import math


def pos(z: float) -> float:
    return z if z > 0.0 else 0.0


def burst_gap(t0: float, rate: float, volume: float, gap: float):
    """Eq. 1: (T_period, T_iss) = (max(T0 + G, V/R), max(T0, V/R - G))."""
    return max(t0 + gap, volume / rate), max(t0, volume / rate - gap)


def recovery_gap(t0: float, rate: float, volume: float) -> float:
    """Eq. 2: G* = [V/R - T0]_+."""
    return pos(volume / rate - t0)


def isolated_occupancy(t0: float, rate: float, volume: float) -> float:
    """Eq. 6, first part: b_iso = [V - R T0]_+."""
    return pos(volume - rate * t0)


def audit(t0: float, rate: float, capacity: float, volumes, gaps, floors=None, q0: float = 0.0):
    """Eqs. 3-6 burst by burst.  Returns dict(rho, delta_b, backlog (q_0..q_N), guard_ok, first_fail)."""
    rho, delta_b, backlog, guard = [], [], [q0], []
    q = q0
    first_fail = len(volumes)
    for n, (v, g) in enumerate(zip(volumes, gaps)):
        f = t0 if floors is None else floors[n]
        period = f + g                               # Eq. 3: P_n
        rho.append(v / (rate * period))              # Eq. 3: rho_n
        delta_b.append(v - rate * period)            # Eq. 4
        fits = q + pos(v - rate * f) <= capacity     # Eq. 6
        guard.append(fits)
        if not fits and first_fail == len(volumes):
            first_fail = n
        q = pos(q + delta_b[-1])                     # Eq. 5
        backlog.append(q)
    return dict(rho=rho, delta_b=delta_b, backlog=backlog, guard_ok=guard, first_fail=first_fail)


def interleaved_gap(t_l2: float, t_l1: float, n1: float, n2: float) -> float:
    """Eq. 7."""
    return t_l2 + n1 / n2 * t_l1


def interleaved_issue_overhead(overhead_wave: float, t_l1: float, n1: float, n2: float) -> float:
    """Eq. 8."""
    return pos(overhead_wave - n1 / n2 * t_l1)


def average_rate_feasible(t0: float, rate: float, volume: float, t_l2: float, t_l1: float, n1: float, n2: float):
    """Eq. 9."""
    return n2 * volume / (n2 * (t0 + t_l2) + n1 * t_l1) <= rate


def lead_knee(b_n: int, k_sm: int, h_inter: int) -> int:
    """App. A.2: ceil(b_n K_SM / (2 h_inter)), in exact integer arithmetic."""
    return -((-b_n * k_sm) // (2 * h_inter))


def mma_stall(t_rs: float, t_cover: float) -> float:
    """App. A.2: [T_RS - T_cover]_+."""
    return pos(t_rs - t_cover)


def fa_recovery_length(b_n: int, g_star: float, sigma: float) -> int:
    """App. C.2: b_n ceil(G*/sigma)."""
    return b_n * math.ceil(g_star / sigma)


def calibrate(periodic, isolated, knee_tolerance: float = 0.10):
    """The three parameters from microbenchmark rows (Sec. 3.3, Sec. 3.5): T0 from the large-gap plateau, R from the
    zero-gap runs, Q from the isolated-burst knee.

    periodic: (volume, gap, t_iss, t_period) tuples of one burst volume; isolated: (volume, t_iss) tuples, ascending.
    Plateau = rows whose gap is among the largest third of the distinct gaps.  The recovered floor of an isolated
    burst is the least-squares line through the smallest third (at least three) of the isolated rows; the knee is the
    row before the first later row that rises more than knee_tolerance above that line; Q = [V_knee - R t_iss]_+.
    Returns (t0, rate or None, capacity or None, knee_volume or None)."""
    import statistics

    import numpy as np
    gaps = sorted({g for _, g, _, _ in periodic})
    top = gaps[len(gaps) - max(1, len(gaps) // 3):]
    t0 = statistics.median(ti for _, g, ti, _ in periodic if g in top)
    zero_gap = [v / tp for v, g, _, tp in periodic if g == 0]
    rate = statistics.median(zero_gap) if zero_gap else None
    if rate is None or len(isolated) < 3:
        return t0, rate, None, None
    n = max(3, len(isolated) // 3)
    vol = np.array([v for v, _ in isolated], dtype=np.float64)
    iss = np.array([t for _, t in isolated], dtype=np.float64)
    if np.ptp(vol[:n]) > 0:
        slope, intercept = np.polyfit(vol[:n], iss[:n], 1)          # library least squares
    else:
        slope, intercept = 0.0, float(iss[:n].mean())
    above = np.flatnonzero(iss[n:] > (1.0 + knee_tolerance) * (intercept + slope * vol[n:]))
    if above.size == 0:
        return t0, rate, None, None
    knee = n + int(above[0]) - 1
    return t0, rate, pos(float(vol[knee]) - rate * float(iss[knee])), float(vol[knee])
