"""Thin ctypes binding of libguide.so: same names as include/guide.h, argument marshalling only.

Device memory and streams come from PyTorch (plumbing); every step of the evaluation runs in the
library's CUDA kernels.  There is no CPU fallback: if the shared library is missing this module
raises at import of the first call, and the library's calls fail with GUIDE_ERR_CUDA without a GPU.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libguide.so")

GUIDE_OK, GUIDE_ERR_INVALID, GUIDE_ERR_OVERFLOW, GUIDE_ERR_UNSUPPORTED = 0, -1, -2, -3
GUIDE_ERR_CUDA, GUIDE_ERR_WORKSPACE, GUIDE_ERR_ITER_LIMIT = -4, -5, -6
TIME_MAX, TIME_SUM = 0, 1
GUIDE_POLICY_PREFILL_FIRST, GUIDE_POLICY_SPLIT_FUSE = 0, 1
TP_EXPLICIT, TP_PAPER_LOG2 = 0, 1
ST_WEIGHTS, ST_KV, ST_HEADS, ST_ITER = 1, 2, 4, 8
METRICS = {"latency": 0, "ttft": 1, "ttft_p99": 2, "tpot": 3, "throughput": 4, "cost_per_hr": 5,
           "cost_per_token": 6}
TTFT_STATS = {"mean": 0, "p50": 1, "p99": 2}
TOPK_MAX, PARETO_MAX, TRACE_MAX_BATCH = 1024, 2048, 256
NOALLOC_TOPK_MAX = 64

F64_OUTPUTS = ("latency", "ttft", "ttft_p50", "ttft_p99", "tpot", "thr_decode", "cost_per_hr", "cost_per_token")
ALL_OUTPUTS = F64_OUTPUTS + ("status", "bmax", "n_iters", "n_req_iters")

EXPORTS = ("guide_last_error", "guide_space_create", "guide_space_destroy", "guide_space_size", "guide_space_decode",
           "guide_trace_load", "guide_trace_destroy", "guide_trace_size", "guide_workspace_bytes", "guide_simulate",
           "guide_select_workspace_bytes", "guide_pareto_workspace_bytes", "guide_select_topk", "guide_pareto",
           "guide_simulate_select", "guide_select_topk_noalloc")


class GuideError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"guide error {code}: {msg}")
        self.code = code


class Model(C.Structure):
    _fields_ = [(k, C.c_uint32) for k in ("n_layers", "hidden", "n_heads", "n_kv_heads", "ffn", "vocab", "gated",
                                          "w_bytes", "a_bytes", "kv_bytes")]


class Hw(C.Structure):
    _fields_ = [("peak_flops", C.c_double), ("mem_bw", C.c_double), ("comm_bw", C.c_double), ("comm_lat", C.c_double),
                ("price_per_hr", C.c_double), ("mem_bytes", C.c_uint64)]


class Fw(C.Structure):
    _fields_ = [("e_c", C.c_double * 3), ("e_m", C.c_double * 3), ("e_comm", C.c_double), ("t_ovh", C.c_double),
                ("flash", C.c_uint32), ("kv_block", C.c_uint32), ("reserve_permille", C.c_uint32), ("policy", C.c_uint32),
                ("split_size", C.c_uint32), ("seg_tokens", C.c_uint32), ("kv_keep_permille", C.c_uint32), ("reserved", C.c_uint32)]


class LenPair(C.Structure):
    _fields_ = [("lin", C.c_uint32), ("lout", C.c_uint32)]


class SpaceDesc(C.Structure):
    _fields_ = [("models", C.POINTER(Model)), ("n_models", C.c_uint32), ("hw", C.POINTER(Hw)), ("n_hw", C.c_uint32),
                ("fw", C.POINTER(Fw)), ("n_fw", C.c_uint32), ("batch", C.POINTER(C.c_uint32)), ("n_batch", C.c_uint32),
                ("tp", C.POINTER(C.c_uint32)), ("n_tp", C.c_uint32), ("pairs", C.POINTER(LenPair)), ("n_pairs", C.c_uint32),
                ("dp", C.POINTER(C.c_uint32))]


class Config(C.Structure):
    _fields_ = [(k, C.c_uint32) for k in ("model", "hw", "fw", "batch_pos", "tp_pos", "pair_pos", "batch", "tp", "lin", "lout", "dp")]


class SimOpts(C.Structure):
    _fields_ = [("first", C.c_uint64), ("count", C.c_uint64), ("time_model", C.c_int32), ("tp_model", C.c_int32),
                ("max_iters", C.c_uint64), ("clamp_seq", C.c_int32), ("precision", C.c_int32)]


class Outputs(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ALL_OUTPUTS + ("req_ttft", "req_tpot", "seq_used")]


class Constraints(C.Structure):
    _fields_ = [("max_ttft", C.c_double), ("ttft_stat", C.c_int32), ("reserved", C.c_int32), ("max_latency", C.c_double),
                ("max_cost_per_hr", C.c_double), ("min_throughput", C.c_double)]


class Selection(C.Structure):
    _fields_ = [("topk_cons", C.POINTER(Constraints)), ("key", C.c_int32), ("k", C.c_uint32), ("topk_idx_dev", C.c_void_p),
                ("topk_key_dev", C.c_void_p), ("topk_count_dev", C.c_void_p), ("pareto_cons", C.POINTER(Constraints)),
                ("x_metric", C.c_int32), ("y_metric", C.c_int32), ("front_idx_dev", C.c_void_p), ("front_cap", C.c_uint32),
                ("front_count_dev", C.c_void_p), ("sweep_begin_event", C.c_void_p), ("sweep_end_event", C.c_void_p)]


_lib = None


def lib():
    """The loaded library; raises if it has not been built (no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2412_04788_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.guide_last_error.restype = C.c_char_p
        L.guide_space_create.argtypes = [C.POINTER(SpaceDesc), C.POINTER(C.c_void_p)]
        L.guide_space_destroy.argtypes = [C.c_void_p]
        L.guide_space_destroy.restype = None
        L.guide_space_size.argtypes = [C.c_void_p]
        L.guide_space_size.restype = C.c_uint64
        L.guide_space_decode.argtypes = [C.c_void_p, C.c_uint64, C.POINTER(Config)]
        L.guide_trace_load.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.POINTER(C.c_void_p)]
        L.guide_trace_destroy.argtypes = [C.c_void_p]
        L.guide_trace_destroy.restype = None
        L.guide_trace_size.argtypes = [C.c_void_p]
        L.guide_trace_size.restype = C.c_uint64
        L.guide_workspace_bytes.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(SimOpts)]
        L.guide_workspace_bytes.restype = C.c_size_t
        L.guide_simulate.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(SimOpts), C.POINTER(Outputs), C.c_void_p,
                                     C.c_size_t, C.c_void_p]
        L.guide_select_workspace_bytes.argtypes = [C.c_void_p, C.c_uint32]
        L.guide_select_workspace_bytes.restype = C.c_size_t
        L.guide_pareto_workspace_bytes.argtypes = [C.c_void_p]
        L.guide_pareto_workspace_bytes.restype = C.c_size_t
        L.guide_select_topk.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(Outputs), C.POINTER(SimOpts),
                                        C.POINTER(Constraints), C.c_int, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_size_t, C.c_void_p]
        L.guide_pareto.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(Outputs), C.POINTER(SimOpts), C.POINTER(Constraints),
                                   C.c_int, C.c_int, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.guide_select_topk_noalloc.argtypes = [C.POINTER(Outputs), C.c_uint64, C.c_uint64, C.POINTER(Constraints), C.c_int,
                                                C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.guide_simulate_select.argtypes = [C.c_void_p, C.POINTER(SimOpts), C.POINTER(Outputs), C.POINTER(Selection), C.c_void_p,
                                            C.c_size_t, C.c_void_p, C.c_size_t, C.c_void_p]
        _lib = L
    return _lib


def _check(rc):
    if rc != GUIDE_OK:
        raise GuideError(rc, lib().guide_last_error().decode())


def guide_last_error() -> str:
    return lib().guide_last_error().decode()


class Space:
    """guide_space handle built from the generator's numpy arrays (see inputs.py for the layout)."""

    def __init__(self, space):
        models = (Model * len(space["models"]))(*[Model(*[int(v) for v in row]) for row in space["models"]])
        hws = (Hw * len(space["hw"]))(*[Hw(float(r[0]), float(r[1]), float(r[2]), float(r[3]), float(r[4]), int(m))
                                        for r, m in zip(space["hw"], space["hw_mem"])])
        fws = (Fw * len(space["fw_f"]))()
        for i, (ff, fi) in enumerate(zip(space["fw_f"], space["fw_i"])):
            fws[i].e_c[:] = [float(x) for x in ff[0:3]]
            fws[i].e_m[:] = [float(x) for x in ff[3:6]]
            fws[i].e_comm, fws[i].t_ovh = float(ff[6]), float(ff[7])
            fws[i].flash, fws[i].kv_block, fws[i].reserve_permille, fws[i].policy = (int(x) for x in fi)
            if space.get("fw_chunk") is not None:
                fws[i].split_size, fws[i].seg_tokens = (int(x) for x in space["fw_chunk"][i])
            if space.get("fw_keep") is not None:
                fws[i].kv_keep_permille = int(space["fw_keep"][i])
        batch = (C.c_uint32 * len(space["batch"]))(*[int(v) for v in space["batch"]])
        tp = (C.c_uint32 * len(space["tp"]))(*[int(v) for v in space["tp"]])
        pairs = (LenPair * len(space["pairs"]))(*[LenPair(int(a), int(b)) for a, b in space["pairs"]])
        dp = None                                   # NULL: every data-parallel degree is 1
        if space.get("dp") is not None:
            if len(space["dp"]) != len(space["tp"]):
                raise ValueError("dp and tp describe the same axis: one data-parallel degree per TP degree")
            dp = (C.c_uint32 * len(space["dp"]))(*[int(v) for v in space["dp"]])
        desc = SpaceDesc(models, len(models), hws, len(hws), fws, len(fws), batch, len(batch), tp, len(tp), pairs, len(pairs), dp)
        self.handle = C.c_void_p()
        _check(lib().guide_space_create(C.byref(desc), C.byref(self.handle)))

    @property
    def size(self) -> int:
        return int(lib().guide_space_size(self.handle))

    def decode(self, idx: int) -> dict:
        cfg = Config()
        _check(lib().guide_space_decode(self.handle, idx, C.byref(cfg)))
        return {k: getattr(cfg, k) for k, _ in Config._fields_}

    def close(self):
        if getattr(self, "handle", None) is not None and self.handle:
            lib().guide_space_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Trace:
    def __init__(self, trace):
        a = np.ascontiguousarray(trace["arrival"], dtype=np.float64)
        i = np.ascontiguousarray(trace["in_len"], dtype=np.uint32)
        o = np.ascontiguousarray(trace["out_len"], dtype=np.uint32)
        self.n = len(a)
        self.handle = C.c_void_p()
        _check(lib().guide_trace_load(a.ctypes.data, i.ctypes.data, o.ctypes.data, self.n, C.byref(self.handle)))

    def close(self):
        if getattr(self, "handle", None) is not None and self.handle:
            lib().guide_trace_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


PREC_F64, PREC_F32 = 0, 1


def _opts(first=0, count=0, time_model=TIME_MAX, tp_model=TP_EXPLICIT, max_iters=0, clamp_seq=False, precision=PREC_F64):
    return SimOpts(first, count, time_model, tp_model, max_iters, int(bool(clamp_seq)), precision)


def _cons(cons):
    cons = cons or {}
    inf = float("inf")
    return Constraints(cons.get("max_ttft", inf), TTFT_STATS[cons.get("ttft_stat", "p99")], 0,
                       cons.get("max_latency", inf), cons.get("max_cost_per_hr", inf), cons.get("min_throughput", 0.0))


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def _stream_ptr(stream):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


_TORCH_DTYPES = None


def alloc_outputs(count, n_req=0, fields=ALL_OUTPUTS, per_request=False, device="cuda"):
    """Caller-owned device arrays for guide_outputs, as a dict of torch tensors."""
    import torch
    dt = {"status": torch.uint8, "bmax": torch.int32, "n_iters": torch.int64, "n_req_iters": torch.int64, "seq_used": torch.int32}
    out = {k: torch.empty(count, dtype=dt.get(k, torch.float64), device=device) for k in fields}
    if per_request:
        out["req_ttft"] = torch.empty((count, n_req), dtype=torch.float64, device=device)
        out["req_tpot"] = torch.empty((count, n_req), dtype=torch.float64, device=device)
    return out


def _outputs_struct(out):
    return Outputs(*[_ptr(out.get(k)) for k in ALL_OUTPUTS + ("req_ttft", "req_tpot", "seq_used")])


def guide_workspace_bytes(space: Space, trace: Trace | None) -> int:
    return int(lib().guide_workspace_bytes(space.handle, trace.handle if trace else None, None))


def guide_simulate(space: Space, trace: Trace | None, out: dict, first=0, count=0, time_model=TIME_MAX,
                   tp_model=TP_EXPLICIT, max_iters=0, workspace=None, stream=None, clamp_seq=False, precision=PREC_F64):
    """out: dict of torch CUDA tensors (see alloc_outputs); workspace: torch uint8 CUDA tensor or None."""
    o = _outputs_struct(out)
    opts = _opts(first, count, time_model, tp_model, max_iters, clamp_seq, precision)
    ws_ptr = _ptr(workspace)
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(lib().guide_simulate(space.handle, trace.handle if trace else None, C.byref(opts), C.byref(o), ws_ptr,
                                ws_bytes, _stream_ptr(stream)))


def guide_select_workspace_bytes(space: Space, k: int) -> int:
    return int(lib().guide_select_workspace_bytes(space.handle, k))


def guide_pareto_workspace_bytes(space: Space) -> int:
    return int(lib().guide_pareto_workspace_bytes(space.handle))


def guide_select_topk(space: Space, trace: Trace | None, out: dict | None, cons: dict | None, key: str, k: int,
                      idx_out, key_out, count_out, workspace, first=0, count=0, time_model=TIME_MAX,
                      tp_model=TP_EXPLICIT, stream=None, clamp_seq=False, precision=PREC_F64):
    """idx_out int64[k], key_out float64[k], count_out int32[1], workspace uint8: torch CUDA tensors."""
    o = _outputs_struct(out) if out is not None else None
    opts = _opts(first, count, time_model, tp_model, 0, clamp_seq, precision)
    cs = _cons(cons)
    _check(lib().guide_select_topk(space.handle, trace.handle if trace else None, C.byref(o) if o is not None else None,
                                   C.byref(opts), C.byref(cs), METRICS[key], k, _ptr(idx_out), _ptr(key_out),
                                   _ptr(count_out), _ptr(workspace), workspace.numel() if workspace is not None else 0,
                                   _stream_ptr(stream)))


def guide_pareto(space: Space, trace: Trace | None, out: dict | None, cons: dict | None, x: str, y: str, idx_out,
                 count_out, workspace, first=0, count=0, time_model=TIME_MAX, tp_model=TP_EXPLICIT, stream=None,
                 clamp_seq=False):
    o = _outputs_struct(out) if out is not None else None
    opts = _opts(first, count, time_model, tp_model, 0, clamp_seq)
    cs = _cons(cons)
    _check(lib().guide_pareto(space.handle, trace.handle if trace else None, C.byref(o) if o is not None else None,
                              C.byref(opts), C.byref(cs), METRICS[x], METRICS[y], _ptr(idx_out), idx_out.numel(),
                              _ptr(count_out), _ptr(workspace), workspace.numel() if workspace is not None else 0,
                              _stream_ptr(stream)))


def guide_simulate_select(space: Space, out: dict, topk_cons: dict | None, key: str, k: int, topk_idx, topk_key, topk_count,
                          topk_workspace, pareto_cons: dict | None, x: str, y: str, front_idx, front_count, pareto_workspace,
                          first=0, count=0, time_model=TIME_MAX, tp_model=TP_EXPLICIT, stream=None, sweep_events=None):
    """guide_simulate (closed form) + guide_select_topk + guide_pareto in one call: the metrics go to
    `out`, the two answers to their tensors; on whole spaces the selections cost no pass of their own.
    sweep_events: optional pair of torch.cuda.Event (already recorded once, so that they exist) that the
    library records right before and after the kernels that evaluate and store the metrics."""
    o = _outputs_struct(out)
    opts = _opts(first, count, time_model, tp_model, 0)
    ct, cp = _cons(topk_cons), _cons(pareto_cons)
    sel = Selection(C.pointer(ct), METRICS[key], k, _ptr(topk_idx), _ptr(topk_key), _ptr(topk_count), C.pointer(cp),
                    METRICS[x], METRICS[y], _ptr(front_idx), front_idx.numel(), _ptr(front_count),
                    C.c_void_p(sweep_events[0].cuda_event) if sweep_events else None,
                    C.c_void_p(sweep_events[1].cuda_event) if sweep_events else None)
    _check(lib().guide_simulate_select(space.handle, C.byref(opts), C.byref(o), C.byref(sel), _ptr(topk_workspace),
                                       topk_workspace.numel(), _ptr(pareto_workspace), pareto_workspace.numel(),
                                       _stream_ptr(stream)))


def guide_select_topk_noalloc(out: dict, cons: dict | None, key: str, k: int, idx_out, key_out, count_out,
                              first=0, count=0, stream=None):
    """Top-k over materialised metrics without any workspace: for callers that may not allocate
    device memory.  The partial results go to a fixed array inside the library (k <= 64); calls
    that could overlap on the GPU must be ordered by the caller.  `out` holds the metric arrays
    written by guide_simulate; `count` defaults to the length of out["status"]."""
    o = _outputs_struct(out)
    cs = _cons(cons)
    n = count or out["status"].numel()
    _check(lib().guide_select_topk_noalloc(C.byref(o), first, n, C.byref(cs), METRICS[key], k, _ptr(idx_out),
                                           _ptr(key_out), _ptr(count_out), _stream_ptr(stream)))
