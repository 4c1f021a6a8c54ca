"""GPU parity of the KV-cache eviction share (H2O) and of the sequence-length clamp (Sec. 3.2 Step 1,
Sec. 3.3, Sec. 3.3.2), closed form: hand-worked toy values and sweeps against the oracle, bit for bit."""
import numpy as np
import pytest

import oracle
from paper_2412_04788_b200 import guide, inputs as I
from gpu_util import assert_parity, bit_mismatches, run_pareto, run_topk

pytestmark = pytest.mark.gpu
FIELDS = guide.ALL_OUTPUTS + ("seq_used",)


def simulate(space_np, **kw):
    import torch
    sp = guide.Space(space_np)
    out = guide.alloc_outputs(sp.size, fields=FIELDS)
    guide.guide_simulate(sp, None, out, **kw)
    torch.cuda.synchronize()
    host = {k: v.cpu().numpy() for k, v in out.items()}
    for k, t in (("bmax", np.uint32), ("n_iters", np.uint64), ("n_req_iters", np.uint64), ("seq_used", np.uint32)):
        host[k] = host[k].view(t)
    return host, out, sp


def toy(golden, avail, block, batch, keep, pairs=((4, 3),)):
    weights = 2 * golden["weights"]["params"]
    return I._space(np.array([golden["model"]]), np.array([golden["hw"]]), np.array([weights + avail]), np.array([[1.0] * 7 + [0.0]]),
                    np.array([[1, block, 0, 0]]), list(batch), [1], [list(p) for p in pairs], fw_keep=[keep])


def test_hand_worked_values(golden):
    g = golden["kv_reduction_and_clamp"]
    for row in g["bmax"]["rows"]:
        got, *_ = simulate(toy(golden, g["bmax"]["avail_bytes"], row["block"], [1, row["bmax"], row["bmax"] + 1], row["p"]))
        assert got["bmax"].tolist() == [row["bmax"]] * 3 and got["status"].tolist() == [0, 0, guide.ST_KV], row
    for row in g["decode"]["rows"]:
        got, *_ = simulate(toy(golden, 10**6, 1, [2], row["p"]))
        assert got["latency"][0] == row["latency"] and got["tpot"][0] == row["tpot"] and got["thr_decode"][0] == 4 / row["T_dec"]
        assert got["seq_used"][0] == 7
    for row in g["clamp"]:
        got, *_ = simulate(toy(golden, row["avail"], row["block"], [2], row["p"]), clamp_seq=True)
        assert got["status"][0] == row["status"] and got["seq_used"][0] == row["seq_used"] and got["bmax"][0] == row["bmax"], row
        if row["status"] == 0:
            ref, *_ = simulate(toy(golden, 10**6, row["block"], [2], row["p"], pairs=[(row["lin_used"], 3)]))
            for k in guide.F64_OUTPUTS:
                assert got[k][0] == ref[k][0], (row, k)


def sweep(keep, chunk=None, dp=False):
    w = I.workload(2, scale=0.5)
    sp = dict(w["space"])
    sp["fw_keep"] = np.array(keep, dtype=np.uint32)
    if chunk is not None:
        sp["fw_chunk"] = np.array(chunk, dtype=np.uint32)
    if dp:
        d, t = I.hybrid_axis(4)
        sp["dp"], sp["tp"] = np.array(d, dtype=np.uint32), np.array(t, dtype=np.uint32)
    return sp


@pytest.mark.parametrize("clamp", [False, True])
@pytest.mark.parametrize("keep,chunk,dp", [([1000, 500, 250], None, False), ([0, 999, 1], [[0, 0], [4, 512], [16, 0]], True)])
def test_sweeps_against_the_oracle(keep, chunk, dp, clamp):
    sp = sweep(keep, chunk, dp)
    for tm, tpm in ((0, 0), (1, 1)):
        want = oracle.simulate(sp, time_model=tm, tp_model=tpm, clamp_seq=clamp)
        got, *_ = simulate(sp, time_model=tm, tp_model=tpm, clamp_seq=clamp)
        assert_parity(got, want, exact=("status", "bmax", "n_iters", "n_req_iters", "seq_used"))
        assert sum(bit_mismatches(got, want).values()) == 0
    assert (want["status"] == 0).sum() > 10000
    if clamp:
        n_l = len(sp["pairs"])
        S = (sp["pairs"][:, 0] + sp["pairs"][:, 1])[np.arange(len(want["status"])) % n_l]
        assert ((want["status"] == 0) & (want["seq_used"] < S)).sum() > 1000      # the sweep has cut configs


def test_selection_with_the_options():
    """Materialised and fused selection see the same metrics: the fused calls evaluate with clamp_seq and
    with the frameworks' eviction shares."""
    sp_np = sweep([1000, 500, 250])
    want = oracle.simulate(sp_np, clamp_seq=True)
    got, out, sp = simulate(sp_np, clamp_seq=True)
    cons = {"max_latency": 30.0}
    for key, k in (("cost_per_token", 64), ("latency", 8)):
        w_idx, w_val, w_cnt = oracle.select_topk(want, cons, key, k)
        for fused in (False, True):
            idx, val, cnt = run_topk(sp, None if fused else out, cons, key, k, clamp_seq=True)
            assert cnt == w_cnt and np.array_equal(idx, w_idx) and np.array_equal(val.view(np.uint64), w_val.view(np.uint64)), (key, fused)
    w_front, w_n = oracle.pareto(want, cons, "latency", "cost_per_hr")
    for fused in (False, True):
        fr, n = run_pareto(sp, None if fused else out, cons, "latency", "cost_per_hr", clamp_seq=True)
        assert n == w_n and np.array_equal(fr, w_front), fused


def test_refused_with_a_trace(golden):
    import torch
    tr = guide.Trace({"arrival": np.array([0.0, 1.0]), "in_len": np.zeros(2, np.uint32), "out_len": np.zeros(2, np.uint32)})
    for space_np, kw in ((toy(golden, 10**6, 1, [2], 500), {}), (toy(golden, 10**6, 1, [2], 1000), {"clamp_seq": True})):
        sp = guide.Space(space_np)
        out = guide.alloc_outputs(sp.size, tr.n)
        ws = torch.empty(guide.guide_workspace_bytes(sp, tr), dtype=torch.uint8, device="cuda")
        with pytest.raises(guide.GuideError) as e:
            guide.guide_simulate(sp, tr, out, workspace=ws, **kw)
        assert e.value.code == guide.GUIDE_ERR_UNSUPPORTED
    with pytest.raises(guide.GuideError) as e:
        guide.Space(toy(golden, 10**6, 1, [2], 1001))
    assert e.value.code == guide.GUIDE_ERR_INVALID
