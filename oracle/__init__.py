"""Python face of the CPU oracle (test infrastructure; the library never imports this).

Compiles `guide_oracle.c` with gcc on first use and calls it through ctypes.  The naive
per-token cross-check lives in `oracle.naive`.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "guide_oracle.c")
_LIB = os.path.join(_HERE, "libguide_oracle.so")

TIME_MAX, TIME_SUM = 0, 1
POLICY_PREFILL_FIRST, POLICY_SPLIT_FUSE = 0, 1
TP_EXPLICIT, TP_PAPER_LOG2 = 0, 1
ST_WEIGHTS, ST_KV, ST_HEADS, ST_ITER = 1, 2, 4, 8
KEYS = {"latency": 0, "ttft": 1, "ttft_p99": 2, "tpot": 3, "throughput": 4, "cost_per_hr": 5,
        "cost_per_token": 6}
TTFT_STATS = {"mean": 0, "p50": 1, "p99": 2}
F64_FIELDS = ("latency", "ttft", "ttft_p50", "ttft_p99", "tpot", "thr_decode", "cost_per_hr", "cost_per_token")


_LIB_F32 = os.path.join(_HERE, "libguide_oracle_f32.so")


def build(force: bool = False, precision: str = "f64") -> str:
    """gcc -O2, contraction off (GCC fuses multiply-add by default otherwise).  precision "f32" builds
    the same source with the model's arithmetic type set to binary32 (-DREAL=float)."""
    out = _LIB if precision == "f64" else _LIB_F32
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC"]
        if precision != "f64":
            cmd.append("-DREAL=float")
        subprocess.run(cmd + [_SRC, "-o", out, "-lm"], check=True)
    return out


class _Space(C.Structure):
    _fields_ = [("models", C.c_void_p), ("n_m", C.c_uint32),
                ("hw", C.c_void_p), ("hw_mem", C.c_void_p), ("n_h", C.c_uint32),
                ("fw_f", C.c_void_p), ("fw_i", C.c_void_p), ("n_f", C.c_uint32),
                ("batch", C.c_void_p), ("n_b", C.c_uint32),
                ("tp", C.c_void_p), ("n_t", C.c_uint32),
                ("pairs", C.c_void_p), ("n_l", C.c_uint32),
                ("dp", C.c_void_p), ("fw_chunk", C.c_void_p), ("fw_keep", C.c_void_p)]


class _Trace(C.Structure):
    _fields_ = [("arrival", C.c_void_p), ("in_len", C.c_void_p), ("out_len", C.c_void_p), ("n", C.c_uint64)]


class _Out(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in F64_FIELDS] + [
        ("status", C.c_void_p), ("bmax", C.c_void_p), ("n_iters", C.c_void_p), ("n_req_iters", C.c_void_p),
        ("req_ttft", C.c_void_p), ("req_tpot", C.c_void_p), ("n_preempt", C.c_void_p), ("seq_used", C.c_void_p)]


class _Cons(C.Structure):
    _fields_ = [("max_ttft", C.c_double), ("ttft_stat", C.c_int), ("max_latency", C.c_double),
                ("max_cost_per_hr", C.c_double), ("min_throughput", C.c_double)]


class _Metrics(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in F64_FIELDS] + [("status", C.c_void_p)]


_lib = None
_libs = {}


def lib(precision: str = "f64"):
    global _lib
    if precision != "f64":
        if precision not in _libs:
            L = C.CDLL(build(precision=precision))
            L.oracle_simulate.restype = C.c_int
            L.oracle_simulate.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint64,
                                          C.c_int, C.c_int, C.c_uint64, C.c_void_p, C.c_int, C.c_int]
            _libs[precision] = L
        return _libs[precision]
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_simulate.restype = C.c_int
        _lib.oracle_simulate.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint64,
                                         C.c_int, C.c_int, C.c_uint64, C.c_void_p, C.c_int, C.c_int]
        _lib.oracle_threads.restype = C.c_int
        for name in ("oracle_weight_params",):
            getattr(_lib, name).restype = C.c_uint64
            getattr(_lib, name).argtypes = [C.c_void_p]
        for name in ("oracle_weight_bytes_per_gpu", "oracle_kv_bytes_per_token"):
            getattr(_lib, name).restype = C.c_uint64
            getattr(_lib, name).argtypes = [C.c_void_p, C.c_uint64]
        _lib.oracle_usable_bytes.restype = C.c_uint64
        _lib.oracle_usable_bytes.argtypes = [C.c_uint64, C.c_uint64]
        _lib.oracle_phase_time.restype = C.c_double
        _lib.oracle_phase_time.argtypes = [C.c_void_p] * 4 + [C.c_uint64] * 6 + [C.c_int, C.c_int, C.c_void_p]
        _lib.oracle_select_topk.restype = C.c_uint32
        _lib.oracle_select_topk.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p, C.c_int, C.c_uint32,
                                            C.c_void_p, C.c_void_p]
        _lib.oracle_pareto.restype = C.c_uint32
        _lib.oracle_pareto.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p, C.c_int, C.c_int,
                                       C.c_void_p, C.c_uint32]
    return _lib


def threads() -> int:
    return int(lib().oracle_threads())


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _space_struct(space):
    return _Space(_p(space["models"]), len(space["models"]), _p(space["hw"]), _p(space["hw_mem"]), len(space["hw"]),
                  _p(space["fw_f"]), _p(space["fw_i"]), len(space["fw_f"]), _p(space["batch"]), len(space["batch"]),
                  _p(space["tp"]), len(space["tp"]), _p(space["pairs"]), len(space["pairs"]),
                  _p(space["dp"]) if space.get("dp") is not None else None,
                  _p(space["fw_chunk"]) if space.get("fw_chunk") is not None else None,
                  _p(space["fw_keep"]) if space.get("fw_keep") is not None else None)


def simulate(space, trace=None, first=0, count=None, stride=1, time_model=TIME_MAX, tp_model=TP_EXPLICIT,
             max_iters=0, per_request=False, n_threads=0, clamp_seq=False, precision="f64"):
    """Evaluate configs first, first+stride, ...; returns a dict of numpy arrays (one slot per config).
    precision "f32": the closed form with every operation of the model in binary32 (values come back
    widened to float64)."""
    assert precision == "f64" or trace is None, "the reduced-precision variant covers the closed form only"
    n_total = 1
    for k in ("models", "hw", "fw_f", "batch", "tp", "pairs"):
        n_total *= len(space[k])
    if count is None:
        count = (n_total - first + stride - 1) // stride
    assert count == 0 or first + (count - 1) * stride < n_total
    out = {k: np.empty(count, dtype=np.float64) for k in F64_FIELDS}
    out["status"] = np.empty(count, dtype=np.uint8)
    out["bmax"] = np.empty(count, dtype=np.uint32)
    out["n_iters"] = np.empty(count, dtype=np.uint64)
    out["n_req_iters"] = np.empty(count, dtype=np.uint64)
    out["n_preempt"] = np.zeros(count, dtype=np.uint64)
    out["seq_used"] = np.zeros(count, dtype=np.uint32)
    ts = None
    if trace is not None:
        n_req = len(trace["arrival"])
        ts = _Trace(_p(trace["arrival"]), _p(trace["in_len"]), _p(trace["out_len"]), n_req)
        if per_request:
            out["req_ttft"] = np.empty((count, n_req), dtype=np.float64)
            out["req_tpot"] = np.empty((count, n_req), dtype=np.float64)
    o = _Out(*[_p(out[k]) for k in F64_FIELDS], _p(out["status"]), _p(out["bmax"]), _p(out["n_iters"]),
             _p(out["n_req_iters"]),
             _p(out["req_ttft"]) if "req_ttft" in out else None,
             _p(out["req_tpot"]) if "req_tpot" in out else None, _p(out["n_preempt"]), _p(out["seq_used"]))
    sp = _space_struct(space)
    rc = lib(precision).oracle_simulate(C.byref(sp), C.byref(ts) if ts is not None else None, first, count, stride,
                               time_model, tp_model, max_iters, C.byref(o), n_threads, int(bool(clamp_seq)))
    if rc != 0:
        why = {-1: "invalid input", -2: "64-bit overflow", -3: "data parallelism, prompt splitting, cache eviction or sequence clamping with a trace is not modelled"}.get(rc, "?")
        raise ValueError(f"oracle_simulate failed: {rc} ({why})")
    return out


def _cons_struct(cons):
    cons = cons or {}
    inf = float("inf")
    return _Cons(cons.get("max_ttft", inf), TTFT_STATS[cons.get("ttft_stat", "p99")], cons.get("max_latency", inf),
                 cons.get("max_cost_per_hr", inf), cons.get("min_throughput", 0.0))


def _metrics_struct(out):
    return _Metrics(*[_p(out[k]) for k in F64_FIELDS], _p(out["status"]))


def select_topk(out, cons, key, k, first=0):
    n = len(out["status"])
    idx = np.empty(k, dtype=np.uint64)
    val = np.empty(k, dtype=np.float64)
    mt, cs = _metrics_struct(out), _cons_struct(cons)
    found = lib().oracle_select_topk(C.byref(mt), n, first, C.byref(cs), KEYS[key], k, _p(idx), _p(val))
    return idx, val, int(found)


def pareto(out, cons, x, y, cap=4096, first=0):
    n = len(out["status"])
    idx = np.empty(cap, dtype=np.uint64)
    mt, cs = _metrics_struct(out), _cons_struct(cons)
    found = lib().oracle_pareto(C.byref(mt), n, first, C.byref(cs), KEYS[x], KEYS[y], _p(idx), cap)
    return idx[:min(found, cap)].copy(), int(found)


def _m(model):
    return np.ascontiguousarray(model, dtype=np.uint32)


def weight_params(model) -> int:
    m = _m(model)
    return int(lib().oracle_weight_params(_p(m)))


def weight_bytes_per_gpu(model, t) -> int:
    m = _m(model)
    return int(lib().oracle_weight_bytes_per_gpu(_p(m), t))


def kv_bytes_per_token(model, t) -> int:
    m = _m(model)
    return int(lib().oracle_kv_bytes_per_token(_p(m), t))


def usable_bytes(mem, reserve_permille) -> int:
    return int(lib().oracle_usable_bytes(mem, reserve_permille))


def phase_time(model, hw, fw_f, fw_i, t, T, E, A, Cc, R, time_model=TIME_MAX, tp_model=TP_EXPLICIT):
    """(T_phase, detail[16]) with detail = t1..t8 (with multiplicity), t9, t10, t11, S_comm, t13,
    S_fix, S_att, T_phase."""
    m = _m(model)
    h = np.ascontiguousarray(hw, dtype=np.float64)
    ff = np.ascontiguousarray(fw_f, dtype=np.float64)
    fi = np.ascontiguousarray(fw_i, dtype=np.uint32)
    det = np.zeros(16, dtype=np.float64)
    v = lib().oracle_phase_time(_p(m), _p(h), _p(ff), _p(fi), t, T, E, A, Cc, R, time_model, tp_model, _p(det))
    return float(v), det
