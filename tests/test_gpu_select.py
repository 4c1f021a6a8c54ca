"""GPU parity, selection: constraint filter + top-k + Pareto against the oracle (bit-exact indices)."""
import numpy as np
import pytest

import oracle
from paper_2412_04788_b200 import guide, inputs as I
from gpu_util import run_pareto, run_simulate, run_topk

pytestmark = pytest.mark.gpu

U64_MAX = np.iinfo(np.uint64).max


def check_topk(sp, out_dev, want_out, cons, key, k, **kw):
    idx, val, cnt = run_topk(sp, out_dev, cons, key, k, **kw)
    w_idx, w_val, w_cnt = oracle.select_topk(want_out, cons, key, k)
    assert cnt == w_cnt, (key, k)
    assert np.array_equal(idx, w_idx), (key, k, idx[:8], w_idx[:8])
    assert np.array_equal(val.view(np.uint64), w_val.view(np.uint64)), (key, k)
    return cnt


def check_pareto(sp, out_dev, want_out, cons, x, y, **kw):
    idx, cnt = run_pareto(sp, out_dev, cons, x, y, **kw)
    w_idx, w_cnt = oracle.pareto(want_out, cons, x, y, cap=guide.PARETO_MAX)
    assert cnt == w_cnt, (x, y)
    assert np.array_equal(idx, w_idx), (x, y)
    return cnt


@pytest.fixture(scope="module")
def c2_small():
    w = I.workload(2, scale=0.25)
    want = oracle.simulate(w["space"])
    got, out_dev, sp, _ = run_simulate(w["space"])
    return w, want, out_dev, sp


def test_topk_materialised_all_keys(c2_small):
    w, want, out_dev, sp = c2_small
    med = float(np.median(want["latency"][want["status"] == 0]))
    for cons in ({}, {"max_latency": med, "max_cost_per_hr": 60.0, "min_throughput": 50.0, "max_ttft": 5.0, "ttft_stat": "mean"}):
        for key in guide.METRICS:
            for k in (1, 8, 64):
                assert check_topk(sp, out_dev, want, cons, key, k) > 0


def test_topk_fused_matches_materialised(c2_small):
    w, want, out_dev, sp = c2_small
    med = float(np.median(want["latency"][want["status"] == 0]))
    for cons in ({}, {"max_latency": med, "max_cost_per_hr": 60.0}):
        for key in ("cost_per_token", "latency", "throughput", "cost_per_hr"):
            check_topk(sp, None, want, cons, key, 64)


def test_topk_large_k_and_ties(c2_small):
    w, want, out_dev, sp = c2_small
    # cost/hr has a handful of distinct values: the result is decided by the index tie-break
    check_topk(sp, out_dev, want, {}, "cost_per_hr", 1024)
    check_topk(sp, out_dev, want, {}, "cost_per_token", 1024)
    check_topk(sp, None, want, {}, "cost_per_hr", 300)
    # 128 is the largest k of the per-warp accumulators, 129 the smallest of the per-block ones
    for k in (128, 129):
        check_topk(sp, out_dev, want, {}, "cost_per_token", k)
        check_topk(sp, None, want, {}, "latency", k)


def test_topk_fewer_than_k_and_none(c2_small):
    w, want, out_dev, sp = c2_small
    lat = np.sort(want["latency"][want["status"] == 0])
    cons = {"max_latency": float(lat[4])}                      # exactly five configs pass (or ties)
    idx, val, cnt = run_topk(sp, out_dev, cons, "latency", 16)
    w_idx, w_val, w_cnt = oracle.select_topk(want, cons, "latency", 16)
    assert cnt == w_cnt and 5 <= cnt < 16
    assert np.array_equal(idx, w_idx) and np.all(idx[cnt:] == U64_MAX) and np.all(np.isinf(val[cnt:]))
    idx, val, cnt = run_topk(sp, out_dev, {"max_latency": 0.0}, "latency", 8)
    assert cnt == 0 and np.all(idx == U64_MAX)
    idx, val, cnt = run_topk(sp, None, {"max_latency": 0.0}, "latency", 8)
    assert cnt == 0 and np.all(idx == U64_MAX)


def test_pareto_materialised_and_fused(c2_small):
    w, want, out_dev, sp = c2_small
    med = float(np.median(want["latency"][want["status"] == 0]))
    for cons in ({}, {"max_latency": med}):
        for x, y in (("latency", "cost_per_hr"), ("latency", "cost_per_token"), ("ttft", "throughput"),
                     ("cost_per_hr", "latency"), ("tpot", "cost_per_token")):
            n = check_pareto(sp, out_dev, want, cons, x, y)
            assert n >= 2
            check_pareto(sp, None, want, cons, x, y)
    idx, cnt = run_pareto(sp, out_dev, {"max_latency": 0.0}, "latency", "cost_per_hr")
    assert cnt == 0
    # a short output buffer still reports the whole front's size
    full, n_full = run_pareto(sp, out_dev, {}, "latency", "cost_per_token")
    part, n_part = run_pareto(sp, out_dev, {}, "latency", "cost_per_token", cap=3)
    assert n_part == n_full and np.array_equal(part, full[:3])


def test_selection_on_a_sub_range(c2_small):
    w, want, out_dev, sp = c2_small
    # an odd offset: the arrays handed over are not 16-byte aligned, so the scalar loads are used
    f1, c1 = 1001, 40003
    sub1 = {k: v[f1:f1 + c1] for k, v in want.items()}
    dev1 = {k: v[f1:f1 + c1] for k, v in out_dev.items()}
    idx, val, cnt = run_topk(sp, dev1, {"max_latency": 5.0}, "cost_per_token", 32, first=f1, count=c1)
    w_idx, w_val, w_cnt = oracle.select_topk(sub1, {"max_latency": 5.0}, "cost_per_token", 32, first=f1)
    assert cnt == w_cnt and np.array_equal(idx, w_idx)
    fidx, fcnt = run_pareto(sp, dev1, {}, "latency", "cost_per_token", first=f1, count=c1)
    w_f, w_n = oracle.pareto(sub1, {}, "latency", "cost_per_token", first=f1)
    assert fcnt == w_n and np.array_equal(fidx, w_f)
    first, count = 1000, 50001
    sub = {k: v[first:first + count] for k, v in want.items()}
    sub_dev = {k: v[first:first + count] for k, v in out_dev.items()}
    idx, val, cnt = run_topk(sp, sub_dev, {}, "cost_per_token", 32, first=first, count=count)
    w_idx, w_val, w_cnt = oracle.select_topk(sub, {}, "cost_per_token", 32, first=first)
    assert cnt == w_cnt and np.array_equal(idx, w_idx)
    idx, val, cnt = run_topk(sp, None, {}, "cost_per_token", 32, first=first, count=count)
    assert cnt == w_cnt and np.array_equal(idx, w_idx)
    fidx, fcnt = run_pareto(sp, None, {}, "latency", "cost_per_hr", first=first, count=count)
    w_f, w_n = oracle.pareto(sub, {}, "latency", "cost_per_hr", first=first)
    assert fcnt == w_n and np.array_equal(fidx, w_f)


def test_pareto_wide_front_and_overflow():
    """Anti-correlated metrics written straight into the arrays: every point is on the front.
    2048 points fit; 2049 report the overflow marker."""
    import torch
    w = I.workload(2, scale=0.125)
    sp = guide.Space(w["space"])
    for n, want_cnt in ((2048, 2048), (2049, 0xFFFFFFFF), (300, 300)):
        x = torch.arange(n, dtype=torch.float64, device="cuda")
        perm = torch.randperm(n, device="cuda", generator=torch.Generator(device="cuda").manual_seed(5))
        out = {"latency": x[perm].contiguous(), "cost_per_hr": (n - x)[perm].contiguous(),
               "status": torch.zeros(n, dtype=torch.uint8, device="cuda")}
        idx, cnt = run_pareto(sp, out, {}, "latency", "cost_per_hr", count=n)
        assert cnt == want_cnt
        if want_cnt == n:
            assert np.array_equal(idx, np.argsort(out["latency"].cpu().numpy()).astype(np.uint64))


def test_workload5_full_size_fused_selection():
    """16.7M configs, nothing materialised for the selection itself; the expected answer comes
    from the oracle run over the whole space (closed form, about a minute of CPU)."""
    w = I.workload(5)
    want = oracle.simulate(w["space"])
    sp = guide.Space(w["space"])
    cons = w["constraints"]
    k = w["topk"]["k"]
    idx, val, cnt = run_topk(sp, None, cons, w["topk"]["key"], k)
    w_idx, w_val, w_cnt = oracle.select_topk(want, cons, w["topk"]["key"], k)
    assert cnt == w_cnt == k and np.array_equal(idx, w_idx)
    assert np.array_equal(val.view(np.uint64), w_val.view(np.uint64))
    fidx, fcnt = run_pareto(sp, None, cons, w["pareto"]["x"], w["pareto"]["y"])
    w_f, w_n = oracle.pareto(want, cons, w["pareto"]["x"], w["pareto"]["y"])
    assert fcnt == w_n and np.array_equal(fidx, w_f) and fcnt >= 2


def test_empty_range_selects_nothing(c2_small):
    """A range of zero configs (first = size of the space): count 0, unused slots marked."""
    w, want, out_dev, sp = c2_small
    n = sp.size
    empty = {k: v[n:n] for k, v in out_dev.items()}
    idx, val, cnt = run_topk(sp, None, {}, "latency", 4, first=n, count=0)
    assert cnt == 0 and np.all(idx == U64_MAX) and np.all(np.isinf(val))
    fidx, fcnt = run_pareto(sp, None, {}, "latency", "cost_per_hr", first=n, count=0)
    assert fcnt == 0
