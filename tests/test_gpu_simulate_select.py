"""GPU parity of guide_simulate_select: the closed-form sweep, a top-k and a Pareto selection in
one call (Sec. 3.2 Steps 1-3 with the constraints of Sec. 4.1).  On whole spaces that go through
the line-wise kernels the selections are a by-product of the sweep (sampled bound and killers first,
every config tested while its metrics are stored); everything else runs the three steps in turn.
Either way the metric arrays must equal the oracle's simulation bit for bit, and the two answers
the oracle's selections on those arrays, index for index."""
import numpy as np
import pytest

import oracle
from paper_2412_04788_b200 import guide, inputs as I
from gpu_util import run_simulate_select

pytestmark = pytest.mark.gpu

EXACT = ("status", "bmax", "n_iters", "n_req_iters") + tuple(guide.F64_OUTPUTS)


def check(space_np, want, cons_t, key, k, cons_p, x, y, **kw):
    got, (idx, val, cnt), (fidx, fcnt), _, _ = run_simulate_select(space_np, cons_t, key, k, cons_p, x, y, **kw)
    for f in EXACT:
        assert np.array_equal(got[f].view(np.uint8), want[f].view(np.uint8)), f
    w_idx, w_val, w_cnt = oracle.select_topk(want, cons_t, key, k)
    assert cnt == w_cnt and np.array_equal(idx, w_idx), (key, k, cnt, w_cnt)
    assert np.array_equal(val.view(np.uint64), w_val.view(np.uint64)), (key, k)
    w_f, w_n = oracle.pareto(want, cons_p, x, y, cap=guide.PARETO_MAX)
    assert fcnt == w_n and np.array_equal(fidx, w_f), (x, y, fcnt, w_n)
    return cnt, fcnt


@pytest.mark.parametrize("tm,tpm", [(0, 0), (1, 1)])
def test_an_eighth_of_workload_5_through_the_line_kernels(tm, tpm):
    """2,097,152 configs, length axis of 64: memory kernel + line kernel with both selections riding
    along.  Keys with many ties (cost per hour), negated keys (throughput), k from 1 to 128,
    constraints that differ between the two selections, and constraints nothing meets."""
    w = I.workload(5, scale=0.125)
    want = oracle.simulate(w["space"], time_model=tm, tp_model=tpm)
    ok = want["status"] == 0
    med = float(np.median(want["latency"][ok]))
    tight = {"max_latency": med, "max_cost_per_hr": 60.0, "min_throughput": 50.0, "max_ttft": 5.0, "ttft_stat": "mean"}
    cases = [(w["constraints"], w["topk"]["key"], w["topk"]["k"], w["constraints"], w["pareto"]["x"], w["pareto"]["y"]),
             ({}, "cost_per_hr", 128, tight, "latency", "cost_per_token"),
             (tight, "throughput", 8, {}, "ttft", "throughput"),
             ({}, "latency", 1, {"max_latency": 0.0}, "tpot", "cost_per_hr"),
             ({"max_latency": 0.0}, "cost_per_token", 64, {}, "latency", "cost_per_hr")]
    seen = []
    for cons_t, key, k, cons_p, x, y in cases:
        seen.append(check(w["space"], want, cons_t, key, k, cons_p, x, y, time_model=tm, tp_model=tpm))
    assert seen[0][0] == w["topk"]["k"] and seen[0][1] >= 2          # the benchmark's own selection is not degenerate
    assert seen[3][1] == 0 and seen[4][0] == 0                        # nothing meets a latency bound of zero


def test_spaces_and_ranges_the_line_kernels_do_not_take():
    """Half of workload 2 (a length axis that does not divide into sixteens), a sub-range of it and
    k above the sampled bound's limit: simulate, then the two selections on the arrays, in one call."""
    w = I.workload(2, scale=0.5)
    want = oracle.simulate(w["space"])
    cons = {"max_cost_per_hr": 80.0}
    check(w["space"], want, cons, "cost_per_token", 8, cons, "latency", "cost_per_hr")
    check(w["space"], want, {}, "latency", 200, {}, "ttft", "cost_per_token")
    n = len(want["status"])
    first, count = n // 3 + 5, n // 2
    part = {f: v[first:first + count] for f, v in want.items() if f in EXACT}
    got, (idx, val, cnt), (fidx, fcnt), _, _ = run_simulate_select(w["space"], cons, "tpot", 16, {}, "latency", "cost_per_hr",
                                                                 first=first, count=count)
    for f in EXACT:
        assert np.array_equal(got[f].view(np.uint8), part[f].view(np.uint8)), f
    w_idx, w_val, w_cnt = oracle.select_topk(part, cons, "tpot", 16)
    assert cnt == w_cnt and np.array_equal(idx, w_idx + np.uint64(first))
    w_f, w_n = oracle.pareto(part, {}, "latency", "cost_per_hr", cap=guide.PARETO_MAX)
    assert fcnt == w_n and np.array_equal(fidx, w_f + np.uint64(first))


def test_refused_arguments_queue_nothing():
    import torch
    w = I.workload(2, scale=0.5)
    sp = guide.Space(w["space"])
    out = guide.alloc_outputs(sp.size, 0)
    out["status"].fill_(77)
    idx = torch.empty(8, dtype=torch.int64, device="cuda"); val = torch.empty(8, dtype=torch.float64, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda"); fidx = torch.empty(64, dtype=torch.int64, device="cuda")
    ws_t = torch.empty(guide.guide_select_workspace_bytes(sp, 8), dtype=torch.uint8, device="cuda")
    ws_p = torch.empty(guide.guide_pareto_workspace_bytes(sp), dtype=torch.uint8, device="cuda")
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(guide.GuideError):                              # Pareto workspace too small
        guide.guide_simulate_select(sp, out, {}, "latency", 8, idx, val, cnt, ws_t, {}, "latency", "cost_per_hr", fidx, cnt, small)
    with pytest.raises(guide.GuideError):                              # k out of range
        guide.guide_simulate_select(sp, out, {}, "latency", 0, idx, val, cnt, ws_t, {}, "latency", "cost_per_hr", fidx, cnt, ws_p)
    missing = dict(out); missing["cost_per_hr"] = None
    with pytest.raises(guide.GuideError):                              # a selection's array is not among the outputs
        guide.guide_simulate_select(sp, missing, {}, "latency", 8, idx, val, cnt, ws_t, {}, "latency", "cost_per_hr", fidx, cnt, ws_p)
    torch.cuda.synchronize()
    assert int((out["status"] != 77).sum().item()) == 0
