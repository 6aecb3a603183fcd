"""ctypes binding of the host-side X-Stage calculator (include/xstage.h): the same names, marshalling only."""
from __future__ import annotations

import ctypes as C

from . import binding


class xstage_params(C.Structure):
    _fields_ = [("t_iss0", C.c_double), ("rate", C.c_double), ("capacity", C.c_double)]


EXPORTS = ("xstage_burst_gap", "xstage_recovery_gap", "xstage_isolated_occupancy", "xstage_audit",
           "xstage_interleaved_gap", "xstage_interleaved_issue_overhead", "xstage_average_rate_feasible",
           "xstage_lead_knee", "xstage_mma_stall", "xstage_fa_recovery_length", "xstage_store_probe", "xstage_calibrate")

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
        lib.xstage_calibrate.argtypes = [C.c_int64, dp, dp, dp, dp, C.c_int64, dp, dp, d, C.c_void_p]
        lib.xstage_calibrate.restype = C.c_int
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


class xstage_calibration(C.Structure):
    _fields_ = [(n, C.c_double) for n in ("t_iss0", "rate", "capacity", "knee_volume", "floor_intercept",
                                          "floor_per_byte")] + [("has_knee", C.c_int32)]


def xstage_calibrate(periodic, isolated, knee_tolerance=0.10):
    """Calibrate (T_iss^0, R, Q) from microbenchmark rows: marshals the rows into arrays for the C routine.

    periodic: rows dict(volume, gap, t_iss, t_period) of one burst volume at several gaps, gap 0 included;
    isolated: rows dict(volume, t_iss) from a recovered state, ascending volume.
    Returns dict(t_iss0, rate, capacity, knee_volume, floor_intercept, floor_per_byte); rate is None without a
    zero-gap row, capacity and knee_volume are None when no row leaves the floor line."""
    col = lambda rows, key: (C.c_double * len(rows))(*[float(r[key]) for r in rows])
    out = xstage_calibration()
    lib = _lib()
    rc = lib.xstage_calibrate(len(periodic), col(periodic, "volume"), col(periodic, "gap"), col(periodic, "t_iss"),
                              col(periodic, "t_period"), len(isolated), col(isolated, "volume"), col(isolated, "t_iss"),
                              float(knee_tolerance), C.byref(out))
    if rc != 0:
        raise ValueError("xstage_calibrate: bad argument")
    fitted = len(isolated) >= 3 and out.rate > 0
    return dict(t_iss0=out.t_iss0, rate=out.rate if out.rate > 0 else None,
                capacity=out.capacity if out.has_knee else None, knee_volume=out.knee_volume if out.has_knee else None,
                floor_intercept=out.floor_intercept if fitted else None,
                floor_per_byte=out.floor_per_byte if fitted else None)


calibrate = xstage_calibrate
