"""ctypes binding of include/eas_serving.h (argument marshalling only): micro-batcher, router, envelopes, SM table."""
from __future__ import annotations
import ctypes as C
import numpy as np
from .binding import load_library

SERVING_SYMBOLS = [
    "eas_poisson_gap_kappa", "eas_batcher_create", "eas_batcher_destroy", "eas_batcher_gap", "eas_batcher_deadline",
    "eas_batcher_on_arrival", "eas_batcher_on_timer", "eas_router_init", "eas_router_init_from_double", "eas_router_next",
    "eas_envelope_plan", "eas_envelope_order", "eas_sm_table_build", "eas_sm_table_lookup", "eas_has_stage1",
]


class HasCandidate(C.Structure):
    _fields_ = [("n_encode", C.c_int32), ("n_prefill", C.c_int32), ("n_decode", C.c_int32), ("n_local", C.c_int32),
                ("rho_e", C.c_double), ("rho_p", C.c_double), ("rho_d", C.c_double), ("score", C.c_double),
                ("b_max", C.c_int32), ("s_star", C.c_double), ("kept", C.c_int32)]


class Router(C.Structure):
    _fields_ = [("num", C.c_int64), ("den", C.c_int64), ("acc", C.c_int64)]


class SmTable(C.Structure):
    _fields_ = [("n_levels", C.c_int32), ("sm_count", C.c_int32 * 16), ("max_batch", C.c_int32 * 16)]


_declared = False


def lib():
    global _declared
    l = load_library()
    if not _declared:
        l.eas_poisson_gap_kappa.restype = C.c_double
        l.eas_poisson_gap_kappa.argtypes = [C.c_int32, C.c_double]
        l.eas_batcher_create.restype = C.c_void_p
        l.eas_batcher_create.argtypes = [C.c_int32, C.c_double, C.c_double, C.c_double]
        l.eas_batcher_destroy.restype = None
        l.eas_batcher_destroy.argtypes = [C.c_void_p]
        l.eas_batcher_gap.restype = C.c_double
        l.eas_batcher_gap.argtypes = [C.c_void_p]
        l.eas_batcher_deadline.restype = C.c_double
        l.eas_batcher_deadline.argtypes = [C.c_void_p]
        l.eas_batcher_on_arrival.restype = C.c_int32
        l.eas_batcher_on_arrival.argtypes = [C.c_void_p, C.c_double, C.POINTER(C.c_int32), C.POINTER(C.c_double)]
        l.eas_batcher_on_timer.restype = C.c_int32
        l.eas_batcher_on_timer.argtypes = [C.c_void_p, C.c_double, C.POINTER(C.c_int32), C.POINTER(C.c_double)]
        l.eas_router_init.restype = C.c_int32
        l.eas_router_init.argtypes = [C.POINTER(Router), C.c_int64, C.c_int64]
        l.eas_router_init_from_double.restype = C.c_int32
        l.eas_router_init_from_double.argtypes = [C.POINTER(Router), C.c_double, C.c_int64]
        l.eas_router_next.restype = C.c_int32
        l.eas_router_next.argtypes = [C.POINTER(Router)]
        l.eas_envelope_plan.restype = C.c_int32
        l.eas_envelope_plan.argtypes = [C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.c_int32, C.c_int32,
                                        C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        l.eas_envelope_order.restype = C.c_int32
        l.eas_envelope_order.argtypes = [C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.c_int32, C.c_int32,
                                         C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
        l.eas_sm_table_build.restype = C.c_int32
        l.eas_sm_table_build.argtypes = [C.POINTER(C.c_int32), C.c_int32, C.POINTER(C.c_int32), C.c_int32,
                                         C.POINTER(C.c_double), C.POINTER(C.c_double), C.c_double, C.POINTER(SmTable)]
        l.eas_sm_table_lookup.restype = C.c_int32
        l.eas_sm_table_lookup.argtypes = [C.POINTER(SmTable), C.c_int32]
        l.eas_has_stage1.restype = C.c_int32
        l.eas_has_stage1.argtypes = [C.POINTER(HasCandidate), C.c_int32, C.c_double, C.c_double, C.c_double, C.c_double,
                                     C.c_double, C.c_double, C.c_int32]
        _declared = True
    return l


def kappa(B: int, p: float) -> float:
    return lib().eas_poisson_gap_kappa(B, p)


def run_batcher(arrivals, B, lam, p=0.6, max_age=1.0):
    """Feeds a sorted arrival trace through eas_batcher_*; returns [(dispatch_time, size)] including the final flush."""
    l = lib()
    h = l.eas_batcher_create(B, lam, p, max_age)
    if not h:
        raise ValueError("bad batcher arguments")
    sizes, times = (C.c_int32 * 2)(), (C.c_double * 2)()
    out = []
    try:
        for t in arrivals:
            n = l.eas_batcher_on_arrival(h, float(t), sizes, times)
            for k in range(n):
                out.append((times[k], sizes[k]))
        dl = l.eas_batcher_deadline(h)
        if np.isfinite(dl):
            s, tt = C.c_int32(), C.c_double()
            assert l.eas_batcher_on_timer(h, np.nextafter(dl, np.inf), C.byref(s), C.byref(tt)) == 1
            out.append((tt.value, s.value))
    finally:
        l.eas_batcher_destroy(h)
    return out


def route(num: int, den: int, n: int):
    l = lib()
    r = Router()
    if l.eas_router_init(C.byref(r), num, den) != 0:
        raise ValueError("bad ratio")
    return [l.eas_router_next(C.byref(r)) for _ in range(n)]


def router_fraction(s: float, max_den: int = 1000):
    r = Router()
    if lib().eas_router_init_from_double(C.byref(r), s, max_den) != 0:
        raise ValueError("bad ratio")
    return r.num, r.den


def envelope_plan(dest, rows, n_dest):
    d = np.ascontiguousarray(dest, dtype=np.int32)
    r = np.ascontiguousarray(rows, dtype=np.int32)
    offs = np.zeros(len(d), dtype=np.int64)
    tot = np.zeros(n_dest, dtype=np.int64)
    rc = lib().eas_envelope_plan(d.ctypes.data_as(C.POINTER(C.c_int32)), r.ctypes.data_as(C.POINTER(C.c_int32)), len(d), n_dest,
                                 offs.ctypes.data_as(C.POINTER(C.c_int64)), tot.ctypes.data_as(C.POINTER(C.c_int64)))
    if rc != 0:
        raise ValueError("bad envelope arguments")
    return offs.tolist(), tot.tolist()


def envelope_order(dest, rows, n_dest):
    """eas_envelope_order -> (order of the requests that groups them by destination, first output row per envelope)."""
    d = np.ascontiguousarray(dest, dtype=np.int32)
    r = np.ascontiguousarray(rows, dtype=np.int32)
    order = np.zeros(len(d), dtype=np.int32)
    first = np.zeros(n_dest, dtype=np.int64)
    rc = lib().eas_envelope_order(d.ctypes.data_as(C.POINTER(C.c_int32)), r.ctypes.data_as(C.POINTER(C.c_int32)), len(d), n_dest,
                                  order.ctypes.data_as(C.POINTER(C.c_int32)), first.ctypes.data_as(C.POINTER(C.c_int64)))
    if rc != 0:
        raise ValueError("bad envelope arguments")
    return order.tolist(), first.tolist()


def sm_table_build(sm_counts, batches, latency, exclusive, tol=0.2) -> SmTable:
    sc = np.ascontiguousarray(sm_counts, dtype=np.int32)
    bs = np.ascontiguousarray(batches, dtype=np.int32)
    lat = np.ascontiguousarray(latency, dtype=np.float64).reshape(len(sc), len(bs))
    ex = np.ascontiguousarray(exclusive, dtype=np.float64)
    t = SmTable()
    rc = lib().eas_sm_table_build(sc.ctypes.data_as(C.POINTER(C.c_int32)), len(sc), bs.ctypes.data_as(C.POINTER(C.c_int32)),
                                  len(bs), lat.ctypes.data_as(C.POINTER(C.c_double)), ex.ctypes.data_as(C.POINTER(C.c_double)),
                                  tol, C.byref(t))
    if rc != 0:
        raise ValueError("bad table arguments")
    return t


def sm_table_lookup(t: SmTable, batch: int) -> int:
    return lib().eas_sm_table_lookup(C.byref(t), batch)


def has_stage1(cands, rate, c_e, c_p, c_d, alpha, prune=1.2, top_k=3):
    """cands: [(n_E, n_P, n_D, n_L)] -> (rows (rho_E, rho_P, rho_D, score, B_max, s*), kept indices)."""
    arr = (HasCandidate * len(cands))()
    for i, (nE, nP, nD, nL) in enumerate(cands):
        arr[i].n_encode, arr[i].n_prefill, arr[i].n_decode, arr[i].n_local = nE, nP, nD, nL
    n = lib().eas_has_stage1(arr, len(cands), rate, c_e, c_p, c_d, alpha, prune, top_k)
    if n < 0:
        raise ValueError("bad Stage-1 arguments")
    rows = [(a.rho_e, a.rho_p, a.rho_d, a.score, a.b_max, a.s_star) for a in arr]
    return rows, [i for i, a in enumerate(arr) if a.kept]
