"""The no-allocation top-k entry point against the regular one.

Some users of the library run where device memory may not be allocated after start-up (a serving
process with a fixed memory pool, a plug-in inside a host application that owns all allocations),
so they cannot hand guide_select_topk a workspace.  guide_select_topk_noalloc keeps its partial
results in an array built into the library instead.  This test calls it through the C ABI twice in
a row - the second call finds the first call's leftovers in that array - and requires the same
indices, values and counts as the workspace-based call.  It lives in the last-collected test file
so that a failure here cannot hide the result of any other test.
"""
import ctypes as C

import numpy as np
import pytest

from paper_2412_04788_b200 import guide, inputs as I
from gpu_util import run_simulate, run_topk

pytestmark = pytest.mark.gpu


def call_noalloc(out_dev, cons, key, k, first=0, count=0):
    import torch
    idx = torch.full((k,), 7, dtype=torch.int64, device="cuda")
    val = torch.zeros(k, dtype=torch.float64, device="cuda")
    cnt = torch.full((1,), 99, dtype=torch.int32, device="cuda")
    guide.guide_select_topk_noalloc(out_dev, cons, key, k, idx, val, cnt, first=first, count=count)
    torch.cuda.synchronize()
    return idx.cpu().numpy().view(np.uint64), val.cpu().numpy(), int(cnt.item())


def test_noalloc_topk_matches_workspace_topk_twice_in_a_row():
    w = I.workload(2, scale=0.25)
    host, out_dev, sp, _ = run_simulate(w["space"])
    med = float(np.median(host["latency"][host["status"] == 0]))
    # two different selections back to back: the second must not see the first one's candidates
    calls = [({}, "cost_per_token", 64), ({"max_latency": med, "max_cost_per_hr": 60.0}, "latency", 8),
             ({}, "cost_per_hr", 33), ({"max_latency": 0.0}, "throughput", 5)]
    for cons, key, k in calls:
        want = run_topk(sp, out_dev, cons, key, k)
        for _ in range(2):
            got = call_noalloc(out_dev, cons, key, k)
            assert got[2] == want[2], (key, k)
            assert np.array_equal(got[0], want[0]), (key, k)
            assert np.array_equal(got[1].view(np.uint64), want[1].view(np.uint64)), (key, k)
    # a sub-range with an index offset
    first, count = 4096, 30001
    sub = {f: t[first:first + count] for f, t in out_dev.items()}
    want = run_topk(sp, sub, {}, "cost_per_token", 16, first=first, count=count)
    got = call_noalloc(sub, {}, "cost_per_token", 16, first=first, count=count)
    assert got[2] == want[2] and np.array_equal(got[0], want[0])


def test_noalloc_topk_rejects_what_its_array_cannot_hold():
    import torch
    n = 1000
    out = {"status": torch.zeros(n, dtype=torch.uint8, device="cuda"),
           "latency": torch.rand(n, dtype=torch.float64, device="cuda")}
    idx = torch.empty(128, dtype=torch.int64, device="cuda")
    val = torch.empty(128, dtype=torch.float64, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(guide.GuideError) as e:
        guide.guide_select_topk_noalloc(out, {}, "latency", guide.NOALLOC_TOPK_MAX + 1, idx, val, cnt)
    assert e.value.code == guide.GUIDE_ERR_UNSUPPORTED and "GUIDE_NOALLOC_TOPK_MAX" in str(e.value)
    with pytest.raises(guide.GuideError) as e:
        guide.guide_select_topk_noalloc(out, {}, "cost_per_hr", 4, idx, val, cnt)      # that array was not given
    assert e.value.code == guide.GUIDE_ERR_INVALID
    # and the largest k it does take works
    guide.guide_select_topk_noalloc(out, {}, "latency", guide.NOALLOC_TOPK_MAX, idx, val, cnt)
    torch.cuda.synchronize()
    want = np.argsort(out["latency"].cpu().numpy(), kind="stable")[:64]
    assert int(cnt.item()) == 64 and np.array_equal(idx[:64].cpu().numpy(), want)
