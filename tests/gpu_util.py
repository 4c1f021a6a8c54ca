"""Helpers for the GPU parity tests: run the CUDA path through the binding, compare with the oracle."""
import numpy as np

import oracle
from paper_2412_04788_b200 import guide

REL_TOL = 1e-9          # bar on fp64 metrics; masks, counters and selections must match exactly


def run_simulate(space_np, trace_np=None, per_request=False, **kw):
    import torch
    sp = guide.Space(space_np)
    tr = guide.Trace(trace_np) if trace_np is not None else None
    first = kw.get("first", 0)
    count = kw.get("count", 0) or sp.size - first
    n_req = tr.n if tr else 0
    out = guide.alloc_outputs(count, n_req, per_request=per_request)
    ws = None
    if tr is not None:
        ws = torch.empty(guide.guide_workspace_bytes(sp, tr), dtype=torch.uint8, device="cuda")
    guide.guide_simulate(sp, tr, out, workspace=ws, **kw)
    torch.cuda.synchronize()
    host = {k: v.cpu().numpy() for k, v in out.items()}
    host["bmax"] = host["bmax"].view(np.uint32)
    host["n_iters"] = host["n_iters"].view(np.uint64)
    host["n_req_iters"] = host["n_req_iters"].view(np.uint64)
    return host, out, sp, tr


def assert_parity(got, want, fields=guide.F64_OUTPUTS, exact=("status", "bmax", "n_iters", "n_req_iters"), what=""):
    for k in exact:
        assert np.array_equal(got[k], want[k]), f"{what}{k}: {np.flatnonzero(got[k] != want[k])[:5]}"
    worst = 0.0
    for k in fields:
        g, w = got[k], want[k]
        inf_g, inf_w = np.isinf(g), np.isinf(w)
        assert np.array_equal(inf_g, inf_w), f"{what}{k}: infinities differ"
        assert not np.isnan(g).any(), f"{what}{k}: NaN"
        fin = ~inf_w
        denom = np.maximum(np.abs(w[fin]), 1e-300)
        rel = np.abs(g[fin] - w[fin]) / denom
        rel = np.where(w[fin] == g[fin], 0.0, rel)
        if rel.size:
            worst = max(worst, float(rel.max()))
        assert rel.size == 0 or rel.max() <= REL_TOL, f"{what}{k}: max rel err {rel.max():.3e}"
    return worst


def bit_mismatches(got, want, fields=guide.F64_OUTPUTS):
    """Number of entries whose binary64 pattern differs (the design goal is zero)."""
    return {k: int((got[k].view(np.uint64) != want[k].view(np.uint64)).sum()) for k in fields}


def run_topk(sp, out, cons, key, k, tr=None, **kw):
    import torch
    idx = torch.empty(k, dtype=torch.int64, device="cuda")
    val = torch.empty(k, dtype=torch.float64, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(guide.guide_select_workspace_bytes(sp, k), dtype=torch.uint8, device="cuda")
    guide.guide_select_topk(sp, tr, out, cons, key, k, idx, val, cnt, ws, **kw)
    torch.cuda.synchronize()
    return idx.cpu().numpy().view(np.uint64), val.cpu().numpy(), int(cnt.item())


def run_pareto(sp, out, cons, x, y, cap=guide.PARETO_MAX, tr=None, **kw):
    import torch
    idx = torch.empty(cap, dtype=torch.int64, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(guide.guide_pareto_workspace_bytes(sp), dtype=torch.uint8, device="cuda")
    guide.guide_pareto(sp, tr, out, cons, x, y, idx, cnt, ws, **kw)
    torch.cuda.synchronize()
    n = int(cnt.cpu().numpy().view(np.uint32)[0])
    return idx.cpu().numpy().view(np.uint64)[:min(n, cap)], n


def run_simulate_select(space_np, topk_cons, key, k, pareto_cons, x, y, cap=guide.PARETO_MAX, **kw):
    """guide_simulate_select on a closed-form space: (host metrics, (idx, val, cnt), (front idx, front size), device arrays, space)"""
    import torch
    sp = guide.Space(space_np)
    first = kw.get("first", 0)
    count = kw.get("count", 0) or sp.size - first
    out = guide.alloc_outputs(count, 0)
    idx = torch.empty(k, dtype=torch.int64, device="cuda")
    val = torch.empty(k, dtype=torch.float64, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    fidx = torch.empty(cap, dtype=torch.int64, device="cuda")
    fcnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws_t = torch.empty(guide.guide_select_workspace_bytes(sp, k), dtype=torch.uint8, device="cuda")
    ws_p = torch.empty(guide.guide_pareto_workspace_bytes(sp), dtype=torch.uint8, device="cuda")
    guide.guide_simulate_select(sp, out, topk_cons, key, k, idx, val, cnt, ws_t, pareto_cons, x, y, fidx, fcnt, ws_p, **kw)
    torch.cuda.synchronize()
    host = {name: v.cpu().numpy() for name, v in out.items()}
    host["bmax"] = host["bmax"].view(np.uint32)
    host["n_iters"] = host["n_iters"].view(np.uint64)
    host["n_req_iters"] = host["n_req_iters"].view(np.uint64)
    n = int(fcnt.cpu().numpy().view(np.uint32)[0])
    return (host, (idx.cpu().numpy().view(np.uint64), val.cpu().numpy(), int(cnt.item())),
            (fidx.cpu().numpy().view(np.uint64)[:min(n, cap)], n), out, sp)
