"""ctypes binding of the host-side X-Stage calculator (include/xstage.h): the same names, marshalling only."""
from __future__ import annotations

import ctypes as C

from . import binding


class xstage_params(C.Structure):
    _fields_ = [("t_iss0", C.c_double), ("rate", C.c_double), ("capacity", C.c_double)]


EXPORTS = ("xstage_burst_gap", "xstage_recovery_gap", "xstage_isolated_occupancy", "xstage_audit",
           "xstage_interleaved_gap", "xstage_interleaved_issue_overhead", "xstage_average_rate_feasible",
           "xstage_lead_knee", "xstage_mma_stall", "xstage_fa_recovery_length", "xstage_store_probe")

_ready = False


def _lib():
    global _ready
    lib = binding.load_library()
    if not _ready:
        d, pp, dp = C.c_double, C.POINTER(xstage_params), C.POINTER(C.c_double)
        lib.xstage_burst_gap.argtypes = [pp, d, d, dp, dp]
        lib.xstage_burst_gap.restype = C.c_int
        for name in ("xstage_recovery_gap", "xstage_isolated_occupancy"):
            getattr(lib, name).argtypes = [pp, d]
            getattr(lib, name).restype = d
        lib.xstage_audit.argtypes = [pp, C.c_int64, dp, dp, dp, d, dp, dp, dp, C.POINTER(C.c_int32)]
        lib.xstage_audit.restype = C.c_int64
        for name in ("xstage_interleaved_gap", "xstage_interleaved_issue_overhead"):
            getattr(lib, name).argtypes = [d, d, d, d]
            getattr(lib, name).restype = d
        lib.xstage_average_rate_feasible.argtypes = [pp, d, d, d, d, d]
        lib.xstage_average_rate_feasible.restype = C.c_int
        lib.xstage_lead_knee.argtypes = [C.c_int64] * 3
        lib.xstage_lead_knee.restype = C.c_int64
        lib.xstage_mma_stall.argtypes = [d, d]
        lib.xstage_mma_stall.restype = d
        lib.xstage_fa_recovery_length.argtypes = [C.c_int64, d, d]
        lib.xstage_fa_recovery_length.restype = C.c_int64
        lib.xstage_store_probe.argtypes = [C.c_int32, C.c_int64, C.c_int64, C.c_int32, C.c_void_p, C.c_uint64, dp, dp, dp,
                                           dp, C.c_void_p]
        lib.xstage_store_probe.restype = C.c_int
        _ready = True
    return lib


def _params(t_iss0, rate, capacity=float("inf")):
    return xstage_params(t_iss0, rate, capacity)


def xstage_burst_gap(t_iss0, rate, volume, gap):
    tp, ti = C.c_double(), C.c_double()
    if _lib().xstage_burst_gap(C.byref(_params(t_iss0, rate)), volume, gap, C.byref(tp), C.byref(ti)) != 0:
        raise ValueError("xstage_burst_gap: bad argument")
    return tp.value, ti.value


def xstage_recovery_gap(t_iss0, rate, volume):
    return _lib().xstage_recovery_gap(C.byref(_params(t_iss0, rate)), volume)


def xstage_isolated_occupancy(t_iss0, rate, volume):
    return _lib().xstage_isolated_occupancy(C.byref(_params(t_iss0, rate)), volume)


def xstage_audit(t_iss0, rate, capacity, volumes, gaps, floors=None, q0=0.0):
    n = len(volumes)
    arr = lambda xs: (C.c_double * max(n, 1))(*xs)
    rho, db, bl = (C.c_double * max(n, 1))(), (C.c_double * max(n, 1))(), (C.c_double * (n + 1))()
    guard = (C.c_int32 * max(n, 1))()
    first = _lib().xstage_audit(C.byref(_params(t_iss0, rate, capacity)), n, arr(volumes),
                                arr(floors) if floors is not None else None, arr(gaps), q0, rho, db, bl, guard)
    if first < 0:
        raise ValueError("xstage_audit: bad argument")
    return dict(rho=list(rho)[:n], delta_b=list(db)[:n], backlog=list(bl), guard_ok=[bool(g) for g in guard][:n],
                first_fail=first)


def xstage_interleaved_gap(t_l2, t_l1, n1, n2):
    return _lib().xstage_interleaved_gap(t_l2, t_l1, n1, n2)


def xstage_interleaved_issue_overhead(overhead_wave, t_l1, n1, n2):
    return _lib().xstage_interleaved_issue_overhead(overhead_wave, t_l1, n1, n2)


def xstage_average_rate_feasible(t_iss0, rate, volume, t_l2, t_l1, n1, n2):
    r = _lib().xstage_average_rate_feasible(C.byref(_params(t_iss0, rate)), volume, t_l2, t_l1, n1, n2)
    if r < 0:
        raise ValueError("xstage_average_rate_feasible: bad argument")
    return bool(r)


def xstage_lead_knee(b_n, k_sm, h_inter):
    return _lib().xstage_lead_knee(b_n, k_sm, h_inter)


def xstage_mma_stall(t_rs, t_cover):
    return _lib().xstage_mma_stall(t_rs, t_cover)


def xstage_fa_recovery_length(b_n, recovery_gap, sigma):
    return _lib().xstage_fa_recovery_length(b_n, recovery_gap, sigma)


def xstage_store_probe(producers, bytes_per_burst, gap_clocks, periods, device_buffer, stream=None):
    """Run the local store microbenchmark on a torch CUDA buffer.  Returns dict(issue_mean, issue_max, period_mean
    (lists of `periods` values in SM clocks), clocks_per_us)."""
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    arr = lambda: (C.c_double * periods)()
    im, ix, pm, cpu = arr(), arr(), arr(), C.c_double(0.0)
    rc = _lib().xstage_store_probe(producers, bytes_per_burst, gap_clocks, periods, C.c_void_p(device_buffer.data_ptr()),
                                   device_buffer.numel() * device_buffer.element_size(), im, ix, pm, C.byref(cpu),
                                   C.c_void_p(stream.cuda_stream))
    if rc != 0:
        raise RuntimeError(f"xstage_store_probe failed with code {rc}")
    return dict(issue_mean=list(im), issue_max=list(ix), period_mean=list(pm), clocks_per_us=cpu.value)


def calibrate(periodic, isolated, knee_tolerance=0.10):
    """The paper's calibration (Sec. 3.3, Sec. 3.5) from microbenchmark rows.

    periodic: rows dict(volume, gap, t_iss, t_period) of one burst volume at several gaps, gap 0 included;
    isolated: rows dict(volume, t_iss) from a recovered state, ascending volume.
    T_iss^0 = median issue time over the largest third of the gaps (the plateau); R = V / T_period at zero gap
    (the drain-limited steady state).  Isolated bursts: the recovered issue floor depends on the volume (the
    issue loop itself takes time), so it is a line a + b V fitted to the smallest third of the volumes; the knee
    is the largest volume whose issue time stays within (1 + knee_tolerance) of that line before the first one
    that leaves it; Q = [V_knee - R T_iss(V_knee)]_+ (Eq. 6 from a recovered state).
    Returns dict(t_iss0, rate, capacity, knee_volume, floor_intercept, floor_per_byte); capacity and knee_volume
    are None when no row leaves the floor line."""
    import statistics
    gaps = sorted({r["gap"] for r in periodic})
    plateau = [r["t_iss"] for r in periodic if r["gap"] >= gaps[-max(1, len(gaps) // 3)]]
    t0 = statistics.median(plateau)
    zero = [r for r in periodic if r["gap"] == 0]
    rate = statistics.median(r["volume"] / r["t_period"] for r in zero) if zero else None
    knee, a, b = None, None, None
    if isolated and rate:
        fit = isolated[: max(3, len(isolated) // 3)]
        n = len(fit)
        mx = sum(r["volume"] for r in fit) / n
        my = sum(r["t_iss"] for r in fit) / n
        sxx = sum((r["volume"] - mx) ** 2 for r in fit)
        b = sum((r["volume"] - mx) * (r["t_iss"] - my) for r in fit) / sxx if sxx > 0 else 0.0
        a = my - b * mx
        for i, r in enumerate(isolated):
            if i >= n and r["t_iss"] > (1.0 + knee_tolerance) * (a + b * r["volume"]):
                knee = isolated[i - 1]
                break
    cap = None if knee is None else max(knee["volume"] - rate * knee["t_iss"], 0.0)
    return dict(t_iss0=t0, rate=rate, capacity=cap, knee_volume=None if knee is None else knee["volume"],
                floor_intercept=a, floor_per_byte=b)
