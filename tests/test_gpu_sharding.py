"""The multi-GPU path on one GPU: workload 2 cut into hardware slices, every slice evaluated and
selected by the library's kernels, the slices' candidates and fronts merged by the same selection
calls (sharding.merge_topk / merge_front with the shards' lists concatenated in place of the
all-gather); the result must be the single-space answer of the oracle."""
import numpy as np
import pytest

import oracle
from paper_2412_04788_b200 import guide, inputs as I, sharding

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world,key,k,x,y", [(2, "cost_per_token", 64, "latency", "cost_per_hr"),
                                             (3, "cost_per_hr", 16, "ttft", "cost_per_token"),
                                             (4, "throughput", 8, "ttft", "throughput")])
def test_slices_merged_by_the_kernels(world, key, k, x, y):
    import torch
    w = I.workload(2, scale=0.5)                      # 8 hardware profiles, 491,520 configs
    g = w["space"]
    cap = guide.PARETO_MAX
    name = {"throughput": "thr_decode"}
    parts = []
    for r in range(world):
        loc, off = sharding.shard_space(g, r, world)
        sp = guide.Space(loc)
        out = guide.alloc_outputs(sp.size)
        guide.guide_simulate(sp, None, out)
        idx = torch.empty(k, dtype=torch.int64, device="cuda")
        val = torch.empty(k, dtype=torch.float64, device="cuda")
        cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
        ws = torch.empty(guide.guide_select_workspace_bytes(sp, k), dtype=torch.uint8, device="cuda")
        guide.guide_select_topk(sp, None, out, w["constraints"], key, k, idx, val, cnt, ws)
        fidx = torch.zeros(cap, dtype=torch.int64, device="cuda")
        fcnt = torch.zeros(1, dtype=torch.int32, device="cuda")
        wsp = torch.empty(guide.guide_pareto_workspace_bytes(sp), dtype=torch.uint8, device="cuda")
        guide.guide_pareto(sp, None, out, w["constraints"], x, y, fidx, fcnt, wsp)
        torch.cuda.synchronize()
        size = int(fcnt.item())
        assert 0 < size <= cap
        used = torch.arange(cap, device="cuda") < size
        sel = torch.where(used, fidx, torch.zeros_like(fidx))
        fx, fy = out[name.get(x, x)][sel], out[name.get(y, y)][sel]
        gfront = torch.where(used, sharding.local_to_global(sel, loc, g, off), torch.full_like(sel, -1))
        parts.append((sharding.local_to_global(idx, loc, g, off), val, gfront, fx, fy))
    spg = guide.Space(g)
    select, front = sharding.kernel_selectors(guide, spg, key, x, y)
    queue = [torch.cat([p[i] for p in parts]) for i in range(5)]
    gather = lambda t: queue.pop(0)
    top, vals, found = sharding.merge_topk(None, None, k, select, gather=gather)
    fr, size = sharding.merge_front(torch.zeros(0, dtype=torch.int64, device="cuda"), None, None, 0, cap, front, gather=gather)
    torch.cuda.synchronize()
    whole = oracle.simulate(g)
    want_idx, want_val, want_found = oracle.select_topk(whole, w["constraints"], key, k)
    want_front, want_size = oracle.pareto(whole, w["constraints"], x, y, cap=cap)
    assert found == want_found and np.array_equal(top.cpu().numpy(), want_idx.view(np.int64))
    assert np.array_equal(vals.cpu().numpy().view(np.uint64), want_val.view(np.uint64))
    assert size == want_size and np.array_equal(fr.cpu().numpy(), want_front.view(np.int64))
