"""GPU parity of the hybrid parallelism axis (Sec. 3.5.2, Sec. 3.5.3): entry i of the parallelism
axis is the pair (dp[i], tp[i]); a replica serves ceil(batch / dp) requests (Sec. 3.2 Step 1).
Every kernel that reads the batch axis is covered: the split pair on whole spaces, the tiled and
the one-thread-per-config kernels on small spaces and sub-ranges, both selection forms."""
import numpy as np
import pytest

import oracle
from paper_2412_04788_b200 import guide, inputs as I
from gpu_util import assert_parity, bit_mismatches, run_pareto, run_simulate, run_topk

pytestmark = pytest.mark.gpu


def test_toy_replicas_match_hand_worked_values(golden):
    sp = I._space(np.array([golden["model"]]), np.array([golden["hw"]]), np.array([10**6]),
                  np.array([[1.0] * 7 + [0.0]]), np.array([[1, 1, 0, 0]]), [4, 3], [1, 1], [(4, 3)], dp=[2, 1])
    got, _, space, _ = run_simulate(sp)
    want = golden["closed_form_b2_Lin4_Lout3"]["t1"]
    for c, b in ((0, 4), (2, 3)):                      # two replicas of at most two requests each
        assert got["ttft"][c] == want["ttft"] and got["latency"][c] == want["latency"] and got["tpot"][c] == want["tpot"]
        assert got["thr_decode"][c] == (want["thr_decode_num"] * b / 2) / want["thr_decode_den"]
        assert got["cost_per_hr"][c] == 2.0 and got["n_req_iters"][c] == 3 * b
    assert [space.decode(i)["dp"] for i in range(4)] == [2, 1, 2, 1]
    assert [space.decode(i)["batch"] for i in range(4)] == [4, 4, 3, 3]


@pytest.mark.parametrize("time_model,tp_model", [(0, 0), (1, 1)])
def test_hybrid_sweep_whole_space(time_model, tp_model):
    """2,211,840 configs, 15 (dp, tp) pairs under a budget of 8 GPUs, batch sizes that do not
    divide by the replica counts: all outputs, bit for bit."""
    w = I.hybrid_workload(8)
    want = oracle.simulate(w["space"], time_model=time_model, tp_model=tp_model)
    got, *_ = run_simulate(w["space"], time_model=time_model, tp_model=tp_model)
    assert_parity(got, want, what="hybrid-8 ")
    assert sum(bit_mismatches(got, want).values()) == 0
    ok = want["status"] == 0
    assert ok.any() and (want["status"] & guide.ST_KV).any()
    # the replicas matter: some config fits only because its batch is shared out
    n_tl = 15 * 64
    dp = np.asarray(w["space"]["dp"])[(np.arange(len(ok)) % n_tl) // 64]
    base = I._space(*(w["space"][k] for k in ("models", "hw", "hw_mem", "fw_f", "fw_i", "batch", "tp", "pairs")))
    alone = oracle.simulate(base, time_model=time_model, tp_model=tp_model)
    assert ((alone["status"] & guide.ST_KV) != 0)[ok & (dp > 1)].any()


def test_hybrid_small_spaces_and_sub_ranges():
    """Below the size the split kernels take, and ragged sub-ranges of a larger space."""
    w = I.hybrid_workload(4, n_hw=2, n_fw=1)
    want = oracle.simulate(w["space"])
    got, *_ = run_simulate(w["space"])
    assert_parity(got, want, what="hybrid-4 ")
    assert sum(bit_mismatches(got, want).values()) == 0
    w = I.hybrid_workload(8, n_hw=3, n_fw=2)
    want = oracle.simulate(w["space"])
    n = len(want["status"])
    for first, count in ((0, 0), (5, 1), (n - 4097, 4097), (99999, 250001)):
        got, *_ = run_simulate(w["space"], first=first, count=count)
        c = count or n - first
        sub = {k: v[first:first + c] for k, v in want.items()}
        assert_parity(got, sub, what=f"[{first},{count}) ")
        assert sum(bit_mismatches(got, sub).values()) == 0


def test_hybrid_selection_materialised_and_fused():
    w = I.hybrid_workload(8)
    want = oracle.simulate(w["space"])
    got, out, sp, _ = run_simulate(w["space"])
    med = float(np.median(want["latency"][want["status"] == 0]))
    for cons in ({}, {"max_latency": med, "max_cost_per_hr": 40.0}):
        for key, k in (("cost_per_token", 64), ("latency", 8), ("throughput", 16), ("cost_per_hr", 8)):
            w_idx, w_val, w_cnt = oracle.select_topk(want, cons, key, k)
            for mat in (out, None):
                idx, val, cnt = run_topk(sp, mat, cons, key, k)
                assert cnt == w_cnt and np.array_equal(idx, w_idx), (key, k, mat is None)
                assert np.array_equal(val.view(np.uint64), w_val.view(np.uint64)), (key, k, mat is None)
        for x, y in (("latency", "cost_per_hr"), ("tpot", "cost_per_token"), ("ttft", "throughput")):
            w_f, w_n = oracle.pareto(want, cons, x, y, cap=guide.PARETO_MAX)
            for mat in (out, None):
                fidx, fcnt = run_pareto(sp, mat, cons, x, y)
                assert fcnt == w_n and np.array_equal(fidx, w_f), (x, y, mat is None)
    # small space: the accumulator kernels, fused
    w = I.hybrid_workload(4, n_hw=2, n_fw=1)
    want = oracle.simulate(w["space"])
    sp = guide.Space(w["space"])
    idx, val, cnt = run_topk(sp, None, {}, "cost_per_token", 64)
    w_idx, w_val, w_cnt = oracle.select_topk(want, {}, "cost_per_token", 64)
    assert cnt == w_cnt and np.array_equal(idx, w_idx) and np.array_equal(val.view(np.uint64), w_val.view(np.uint64))
    fidx, fcnt = run_pareto(sp, None, {}, "latency", "cost_per_hr")
    w_f, w_n = oracle.pareto(want, {}, "latency", "cost_per_hr", cap=guide.PARETO_MAX)
    assert fcnt == w_n and np.array_equal(fidx, w_f)


def test_trace_with_replicas_is_refused():
    w = I.workload(1)
    space = dict(w["space"])
    space["dp"] = np.array([1, 2, 1], dtype=np.uint32)
    with pytest.raises(guide.GuideError, match="data-parallel") as e:
        run_simulate(space, w["trace"])
    assert e.value.code == guide.GUIDE_ERR_UNSUPPORTED
    space["dp"] = np.array([1, 1, 1], dtype=np.uint32)           # an axis of ones is no replica split
    got, *_ = run_simulate(space, w["trace"])
    want = oracle.simulate(w["space"], w["trace"])
    assert_parity(got, want, what="C1 trace, dp = 1 ")
