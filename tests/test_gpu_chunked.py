"""GPU parity of prompt processing in pieces (Sec. 3.3.1 sub-batches of split_size requests,
Sec. 3.3.2 prompt segments): framework profiles that set split_size / seg_tokens."""
import numpy as np
import pytest

import oracle
from paper_2412_04788_b200 import guide, inputs as I
from gpu_util import assert_parity, bit_mismatches, run_pareto, run_simulate, run_topk

pytestmark = pytest.mark.gpu


def toy(golden, batch, chunk, pairs=((4, 3),), dp=None):
    return I._space(np.array([golden["model"]]), np.array([golden["hw"]]), np.array([10**6]),
                    np.array([[1.0] * 7 + [0.0]]), np.array([[1, 1, 0, 0]]), list(batch), [1], [list(p) for p in pairs],
                    dp=dp, fw_chunk=[list(chunk)])


def test_toy_sub_batches_match_hand_worked_values(golden):
    want = golden["closed_form_b2_Lin4_Lout3"]["t1"]
    got, *_ = run_simulate(toy(golden, [2, 4, 5, 1], (2, 0)))
    assert got["ttft"][0] == want["ttft"] and got["latency"][0] == want["latency"]
    assert got["ttft"][1] == 2.0 * want["ttft"] and got["ttft"][2] == 2.0 * want["ttft"] + got["ttft"][3]
    assert got["n_iters"].tolist() == [3, 4, 5, 3] and got["n_req_iters"].tolist() == [6, 12, 15, 3]
    seg, *_ = run_simulate(toy(golden, [2], (0, 2)))
    assert seg["ttft"][0] > want["ttft"] and seg["n_iters"][0] == 4 and seg["n_req_iters"][0] == 8
    assert seg["ttft"][0] == oracle.simulate(toy(golden, [2], (0, 2)))["ttft"][0]


@pytest.mark.parametrize("time_model,tp_model", [(0, 0), (1, 0), (0, 1)])
def test_chunked_sweep(time_model, tp_model):
    """491,520 configs, one framework in three unsplit: all outputs, bit for bit."""
    w = I.chunked_workload()
    want = oracle.simulate(w["space"], time_model=time_model, tp_model=tp_model)
    got, *_ = run_simulate(w["space"], time_model=time_model, tp_model=tp_model)
    assert_parity(got, want, what="C2-chunked ")
    assert sum(bit_mismatches(got, want).values()) == 0
    # nothing but the prompt time changes; sub-batches alone (profile 2) can only cost time: every
    # pass reads the weights again.  (Segments can also save time: their tokens attend the prompt
    # up to their own segment, the unsplit pass is charged the full rectangle.)
    plain = oracle.simulate(I.workload(2, scale=0.5)["space"], time_model=time_model, tp_model=tp_model)
    ok = want["status"] == 0
    assert np.array_equal(want["status"], plain["status"]) and np.array_equal(want["bmax"], plain["bmax"])
    sp = w["space"]
    per_f = len(sp["batch"]) * len(sp["tp"]) * len(sp["pairs"])
    f = (np.arange(len(ok)) // per_f) % 3
    assert np.array_equal(want["ttft"][f == 0], plain["ttft"][f == 0])
    sub = ok & (f == 2)
    assert (want["ttft"][sub] >= plain["ttft"][sub] * (1 - 1e-12)).all() and (want["ttft"][sub] > plain["ttft"][sub]).any()
    assert (want["ttft"][ok & (f == 1)] != plain["ttft"][ok & (f == 1)]).any()
    assert np.array_equal(want["tpot"], plain["tpot"])


def test_chunked_sub_ranges_and_replicas():
    w = I.chunked_workload(scale=0.125, n_gpus=4)
    want = oracle.simulate(w["space"])
    n = len(want["status"])
    for first, count in ((0, 0), (3, 1), (n - 5000, 5000), (77777, 100001)):
        got, *_ = run_simulate(w["space"], first=first, count=count)
        c = count or n - first
        sub = {k: v[first:first + c] for k, v in want.items()}
        assert_parity(got, sub, what=f"[{first},{count}) ")
        assert sum(bit_mismatches(got, sub).values()) == 0


def test_profiles_that_split_nothing_take_the_fast_kernels():
    w = I.workload(2, scale=0.5)
    sp = dict(w["space"])
    sp["fw_chunk"] = np.zeros((3, 2), dtype=np.uint32)
    a, *_ = run_simulate(sp)
    b, *_ = run_simulate(w["space"])
    for k in a:
        assert np.array_equal(a[k].view(np.uint8), b[k].view(np.uint8)), k
    sp["fw_chunk"] = np.array([[1 << 20, 1 << 20]] * 3, dtype=np.uint32)     # larger than every batch and prompt
    c, *_ = run_simulate(sp)
    for k in a:
        assert np.array_equal(a[k].view(np.uint8), c[k].view(np.uint8)), k


def test_chunked_selection():
    w = I.chunked_workload()
    want = oracle.simulate(w["space"])
    got, out, sp, _ = run_simulate(w["space"])
    med = float(np.median(want["ttft"][want["status"] == 0]))
    for cons in ({}, {"max_ttft": med, "ttft_stat": "mean"}):
        for key, k in (("cost_per_token", 64), ("ttft", 8), ("latency", 8)):
            w_idx, w_val, w_cnt = oracle.select_topk(want, cons, key, k)
            for mat in (out, None):
                idx, val, cnt = run_topk(sp, mat, cons, key, k)
                assert cnt == w_cnt and np.array_equal(idx, w_idx), (key, k, mat is None)
                assert np.array_equal(val.view(np.uint64), w_val.view(np.uint64)), (key, k, mat is None)
        for x, y in (("latency", "cost_per_hr"), ("ttft", "throughput")):
            w_f, w_n = oracle.pareto(want, cons, x, y, cap=guide.PARETO_MAX)
            for mat in (out, None):
                fidx, fcnt = run_pareto(sp, mat, cons, x, y)
                assert fcnt == w_n and np.array_equal(fidx, w_f), (x, y, mat is None)


def test_trace_with_split_profiles_is_refused():
    w = I.workload(1)
    space = dict(w["space"])
    space["fw_chunk"] = np.array([[0, 256]], dtype=np.uint32)
    with pytest.raises(guide.GuideError, match="prompt-first") as e:
        run_simulate(space, w["trace"])
    assert e.value.code == guide.GUIDE_ERR_UNSUPPORTED
