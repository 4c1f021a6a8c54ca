"""GPU parity of the binary32 variant of the closed form: against the oracle built with binary32
arithmetic bit for bit (both sides take every decision in the same precision), against the binary64
oracle within 1e-5 relative; integer outputs identical to the binary64 path."""
import numpy as np
import pytest

import oracle
from paper_2412_04788_b200 import guide, inputs as I
from gpu_util import run_pareto, run_topk

pytestmark = pytest.mark.gpu
FIELDS = guide.ALL_OUTPUTS + ("seq_used",)
F32_TOL = 1e-5


def simulate(space_np, **kw):
    import torch
    sp = guide.Space(space_np)
    out = guide.alloc_outputs(sp.size, fields=FIELDS)
    guide.guide_simulate(sp, None, out, precision=guide.PREC_F32, **kw)
    torch.cuda.synchronize()
    host = {k: v.cpu().numpy() for k, v in out.items()}
    for k, t in (("bmax", np.uint32), ("n_iters", np.uint64), ("n_req_iters", np.uint64), ("seq_used", np.uint32)):
        host[k] = host[k].view(t)
    return host, out, sp


def check(got, want32, want64):
    for k in ("status", "bmax", "n_iters", "n_req_iters", "seq_used"):
        assert np.array_equal(got[k], want32[k]) and np.array_equal(got[k], want64[k]), k
    worst = 0.0
    for k in guide.F64_OUTPUTS:
        assert np.array_equal(got[k].view(np.uint64), want32[k].view(np.uint64)), k          # same precision: same bits
        fin = np.isfinite(want64[k]) & (want64[k] != 0)
        assert np.array_equal(np.isfinite(got[k]), np.isfinite(want64[k])), k
        rel = np.abs(got[k][fin] - want64[k][fin]) / np.abs(want64[k][fin])
        worst = max(worst, float(rel.max()) if rel.size else 0.0)
    assert worst <= F32_TOL, worst
    return worst


def test_hand_worked_toy(golden):
    want = golden["closed_form_b2_Lin4_Lout3"]["t1"]
    sp = I._space(np.array([golden["model"]]), np.array([golden["hw"]]), np.array([10**6]), np.array([[1.0] * 7 + [0.0]]),
                  np.array([[1, 1, 0, 0]]), [2], [1], [(4, 3)])
    got, *_ = simulate(sp)
    assert got["ttft"][0] == want["ttft"] and got["latency"][0] == want["latency"] and got["tpot"][0] == want["tpot"]


@pytest.mark.parametrize("variant", ["plain", "split+dp", "evict+clamp"])
def test_sweep(variant):
    w = I.workload(2, scale=0.5)
    sp = dict(w["space"])
    kw = {}
    if variant == "split+dp":
        sp["fw_chunk"] = np.array([[0, 0], [4, 512], [16, 0]], dtype=np.uint32)
        d, t = I.hybrid_axis(4)
        sp["dp"], sp["tp"] = np.array(d, dtype=np.uint32), np.array(t, dtype=np.uint32)
    if variant == "evict+clamp":
        sp["fw_keep"] = np.array([1000, 500, 250], dtype=np.uint32)
        kw["clamp_seq"] = True
    for tm, tpm in ((0, 0), (1, 1)):
        want32 = oracle.simulate(sp, time_model=tm, tp_model=tpm, precision="f32", **kw)
        want64 = oracle.simulate(sp, time_model=tm, tp_model=tpm, **kw)
        got, *_ = simulate(sp, time_model=tm, tp_model=tpm, **kw)
        worst = check(got, want32, want64)
        assert worst > 1e-9                        # it really is a rounded result
    assert (want64["status"] == 0).sum() > 10000


def test_selection_on_binary32_metrics():
    w = I.workload(2, scale=0.5)
    want = oracle.simulate(w["space"], precision="f32")
    got, out, sp = simulate(w["space"])
    cons = {"max_latency": 30.0}
    for key, k in (("cost_per_token", 64), ("cost_per_hr", 16)):
        w_idx, w_val, w_cnt = oracle.select_topk(want, cons, key, k)
        idx, val, cnt = run_topk(sp, out, cons, key, k)
        assert cnt == w_cnt and np.array_equal(idx, w_idx) and np.array_equal(val.view(np.uint64), w_val.view(np.uint64))
    w_front, w_n = oracle.pareto(want, cons, "latency", "cost_per_hr")
    fr, n = run_pareto(sp, out, cons, "latency", "cost_per_hr")
    assert n == w_n and np.array_equal(fr, w_front)


def test_where_it_is_not_offered(golden):
    import torch
    sp_np = I.workload(1)["space"]
    sp = guide.Space(sp_np)
    tr = guide.Trace({"arrival": np.array([0.0, 1.0]), "in_len": np.zeros(2, np.uint32), "out_len": np.zeros(2, np.uint32)})
    out = guide.alloc_outputs(sp.size, tr.n)
    ws = torch.empty(guide.guide_workspace_bytes(sp, tr), dtype=torch.uint8, device="cuda")
    with pytest.raises(guide.GuideError) as e:
        guide.guide_simulate(sp, tr, out, workspace=ws, precision=guide.PREC_F32)
    assert e.value.code == guide.GUIDE_ERR_UNSUPPORTED
    with pytest.raises(guide.GuideError) as e:
        guide.guide_simulate(sp, None, out, precision=7)
    assert e.value.code == guide.GUIDE_ERR_INVALID
    with pytest.raises(guide.GuideError) as e:                    # the fused selection evaluates in binary64
        run_topk(sp, None, {}, "latency", 4, precision=guide.PREC_F32)
    assert e.value.code == guide.GUIDE_ERR_UNSUPPORTED
