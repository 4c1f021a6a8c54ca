"""GPU parity of the streaming selection path (sample -> bound / killers -> one filter pass ->
exact finish) that materialised metrics of 2^18 configs or more go through.

The metric arrays are written by the test (seeded), not by the simulation, so that the cases the
bound and the killers must survive can be built directly: ties on the key, fewer passing configs
than k, nothing passing, sorted inputs, good configs hidden from the sample, wide fronts, duplicate
points, ragged lengths.  Expected answers come from the oracle's selection on the same arrays;
indices and counts must match exactly.
"""
import numpy as np
import pytest

import oracle
from paper_2412_04788_b200 import guide, inputs as I
from gpu_util import run_pareto, run_simulate, run_simulate_select, run_topk

pytestmark = pytest.mark.gpu

U64_MAX = np.iinfo(np.uint64).max
N_MIN = 1 << 18                      # smallest range the streaming path takes


def synth(n, seed, pass_frac=0.3):
    rng = np.random.default_rng(seed)
    out = {k: rng.random(n) for k in guide.F64_OUTPUTS}
    out["latency"] = out["latency"] * 10.0
    out["thr_decode"] = out["thr_decode"] * 1000.0
    out["cost_per_hr"] = np.floor(out["cost_per_hr"] * 64.0) + 1.0          # few distinct values
    out["status"] = np.where(rng.random(n) < pass_frac, 0, 2).astype(np.uint8)
    return out


def to_dev(out):
    import torch
    return {k: torch.from_numpy(np.ascontiguousarray(v)).cuda() for k, v in out.items()}


@pytest.fixture(scope="module")
def sp():
    space = guide.Space(I.workload(5, scale=0.125)["space"])       # 2,097,152 configs: room for every range below
    assert space.size >= 6 * N_MIN + 1
    return space


def check_topk(sp, host, dev, cons, key, k):
    n = len(host["status"])
    idx, val, cnt = run_topk(sp, dev, cons, key, k, count=n)
    w_idx, w_val, w_cnt = oracle.select_topk(host, cons, key, k)
    assert cnt == w_cnt, (key, k, cnt, w_cnt)
    assert np.array_equal(idx, w_idx), (key, k, idx[:4], w_idx[:4])
    assert np.array_equal(val.view(np.uint64), w_val.view(np.uint64)), (key, k)
    return cnt


def check_pareto(sp, host, dev, cons, x, y):
    n = len(host["status"])
    idx, cnt = run_pareto(sp, dev, cons, x, y, count=n)
    w_idx, w_cnt = oracle.pareto(host, cons, x, y, cap=guide.PARETO_MAX)
    assert cnt == w_cnt, (x, y, cnt, w_cnt)
    assert np.array_equal(idx, w_idx), (x, y)
    return cnt


def test_topk_random_keys_bounds_and_ragged_lengths(sp):
    for n, seed in ((N_MIN, 1), (N_MIN + 1, 2), (3 * N_MIN + 1023, 3), (5 * N_MIN + 65, 4)):
        host = synth(n, seed)
        dev = to_dev(host)
        for cons in ({}, {"max_latency": 4.0, "max_cost_per_hr": 40.0, "min_throughput": 100.0, "max_ttft": 0.9,
                          "ttft_stat": "p50"}):
            for key in ("cost_per_token", "throughput", "cost_per_hr", "latency"):
                for k in (1, 64, 128):
                    assert check_topk(sp, host, dev, cons, key, k) == k


def test_topk_ties_on_the_key(sp):
    """Every key equal: the key alone excludes nothing, the index half of the (key, index) bound
    does; the answer is the k lowest passing indices."""
    n = 2 * N_MIN + 77
    host = synth(n, 5)
    host["cost_per_token"][:] = 0.25
    dev = to_dev(host)
    check_topk(sp, host, dev, {}, "cost_per_token", 64)
    # a few distinct values, with many configs on each
    check_topk(sp, host, dev, {}, "cost_per_hr", 128)
    check_topk(sp, host, dev, {"max_latency": 5.0}, "cost_per_hr", 8)


def test_topk_fewer_passing_than_k_and_none(sp):
    n = N_MIN + 4096
    host = synth(n, 6)
    host["status"][:] = 2
    keep = np.array([5, 70000, 70001, n - 1, n - 3000])
    host["status"][keep] = 0
    dev = to_dev(host)
    idx, val, cnt = run_topk(sp, dev, {}, "latency", 16, count=n)
    w_idx, w_val, w_cnt = oracle.select_topk(host, {}, "latency", 16)
    assert cnt == w_cnt == 5 and np.array_equal(idx, w_idx)
    assert np.all(idx[cnt:] == U64_MAX) and np.all(np.isinf(val[cnt:]))
    host["status"][:] = 1
    dev = to_dev(host)
    idx, val, cnt = run_topk(sp, dev, {}, "latency", 8, count=n)
    assert cnt == 0 and np.all(idx == U64_MAX) and np.all(np.isinf(val))
    fidx, fcnt = run_pareto(sp, dev, {}, "latency", "cost_per_hr", count=n)
    assert fcnt == 0


def test_topk_sorted_inputs_and_winners_in_one_corner(sp):
    n = 4 * N_MIN
    host = synth(n, 7, pass_frac=1.0)
    for order in (np.arange(n, dtype=np.float64), np.arange(n, 0, -1, dtype=np.float64)):
        host["cost_per_token"] = order
        dev = to_dev(host)
        check_topk(sp, host, dev, {}, "cost_per_token", 64)
    # all good keys inside one stretch of 2000 configs, most of which no sample row touches
    host = synth(n, 8)
    host["cost_per_token"] += 10.0
    host["cost_per_token"][600000:602000] -= 10.0
    dev = to_dev(host)
    check_topk(sp, host, dev, {}, "cost_per_token", 128)


def test_topk_bound_in_two_kernels():
    """The top-k bound is one cooperative kernel where the device launches cooperatively, two
    kernels otherwise; GUIDE_NO_COOPERATIVE forces the second form.  The library reads the variable
    once per process, so the check runs in a child process: same cases, same oracle."""
    import os
    import subprocess
    import sys
    code = (
        "import sys; sys.path.insert(0, 'tests')\n"
        "import test_gpu_select_stream as t\n"
        "from paper_2412_04788_b200 import guide, inputs as I\n"
        "sp = guide.Space(I.workload(5, scale=0.125)['space'])\n"
        "for n, seed in ((t.N_MIN + 1, 21), (5 * t.N_MIN + 65, 22)):\n"
        "    host = t.synth(n, seed); dev = t.to_dev(host)\n"
        "    for key, k in (('cost_per_token', 64), ('cost_per_hr', 128), ('throughput', 1)):\n"
        "        assert t.check_topk(sp, host, dev, {'max_latency': 6.0}, key, k) == k\n"
        "print('two-kernel bound ok')\n")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, "-c", code], cwd=root, env=dict(os.environ, GUIDE_NO_COOPERATIVE="1"),
                         capture_output=True, text=True, timeout=600)
    assert res.returncode == 0 and "two-kernel bound ok" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]


def test_fused_streaming_selection_half_of_workload_2():
    """Nothing materialised, 491,520 configs: the sample rows are evaluated into the workspace, the
    bound / killers come from them and the model walk is the filter pass.  All keys, with and
    without constraints, both time models."""
    w = I.workload(2, scale=0.5)
    sp2 = guide.Space(w["space"])
    assert sp2.size >= N_MIN
    for tm, tpm in ((0, 0), (1, 1)):
        want = oracle.simulate(w["space"], time_model=tm, tp_model=tpm)
        med = float(np.median(want["latency"][want["status"] == 0]))
        for cons in ({}, {"max_latency": med, "max_cost_per_hr": 60.0, "min_throughput": 50.0, "max_ttft": 5.0, "ttft_stat": "mean"}):
            for key in guide.METRICS:
                for k in ((1, 64, 128) if key == "cost_per_token" else (8,)):
                    idx, val, cnt = run_topk(sp2, None, cons, key, k, time_model=tm, tp_model=tpm)
                    w_idx, w_val, w_cnt = oracle.select_topk(want, cons, key, k)
                    assert cnt == w_cnt and np.array_equal(idx, w_idx), (tm, key, k)
                    assert np.array_equal(val.view(np.uint64), w_val.view(np.uint64)), (tm, key, k)
            for x, y in (("latency", "cost_per_hr"), ("latency", "cost_per_token"), ("ttft", "throughput"), ("tpot", "cost_per_hr")):
                fidx, fcnt = run_pareto(sp2, None, cons, x, y, time_model=tm, tp_model=tpm)
                w_f, w_n = oracle.pareto(want, cons, x, y, cap=guide.PARETO_MAX)
                assert fcnt == w_n and np.array_equal(fidx, w_f), (tm, x, y)
    # nothing passes
    idx, val, cnt = run_topk(sp2, None, {"max_latency": 0.0}, "latency", 8)
    assert cnt == 0 and np.all(idx == U64_MAX)
    fidx, fcnt = run_pareto(sp2, None, {"max_latency": 0.0}, "latency", "cost_per_hr")
    assert fcnt == 0


def test_pareto_random_pairs(sp):
    for n, seed in ((N_MIN, 11), (2 * N_MIN + 513, 12), (6 * N_MIN + 1, 13)):
        host = synth(n, seed)
        dev = to_dev(host)
        for cons in ({}, {"max_latency": 3.0, "min_throughput": 200.0}):
            for x, y in (("latency", "cost_per_hr"), ("latency", "cost_per_token"), ("ttft", "throughput"),
                         ("cost_per_hr", "latency")):
                assert check_pareto(sp, host, dev, cons, x, y) >= 1


def test_pareto_duplicates_keep_the_lowest_index(sp):
    n = 2 * N_MIN
    host = synth(n, 14)
    host["latency"] = np.floor(host["latency"] * 3.0)            # 30 distinct x, 64 distinct y: heavy duplication
    dev = to_dev(host)
    check_pareto(sp, host, dev, {}, "latency", "cost_per_hr")
    host["latency"][:] = 1.0                                     # one x: the front is one point, the first with the smallest y
    dev = to_dev(host)
    assert check_pareto(sp, host, dev, {}, "latency", "cost_per_hr") == 1


def test_pareto_wide_fronts(sp):
    """Anti-correlated metrics on part of the range: 1500 front points go through the streaming
    path's own finish, 2048 are the most a front may have, 2049 and 6000 report the overflow marker
    (6000 also overflows the survivor list, so the general kernel redoes the call)."""
    n = 2 * N_MIN + 9
    rng = np.random.default_rng(15)
    for width, want in ((1500, 1500), (2048, 2048), (2049, 0xFFFFFFFF), (6000, 0xFFFFFFFF)):
        host = synth(n, 16)
        host["latency"] += 10.0 * width
        host["cost_per_hr"] += 10.0 * width
        where = rng.choice(n, size=width, replace=False)
        t = np.arange(width, dtype=np.float64)
        host["latency"][where] = t
        host["cost_per_hr"][where] = width - t
        host["status"][where] = 0
        dev = to_dev(host)
        idx, cnt = run_pareto(sp, dev, {}, "latency", "cost_per_hr", count=n)
        assert cnt == want, (width, cnt)
        if want == width:
            assert np.array_equal(idx, where.astype(np.uint64))


def test_workload5_full_size_materialised_selection():
    """The benchmark's own configuration: 16.7M configs simulated into arrays, then top-64 and the
    Pareto front read from them; the oracle evaluates the whole space (about a minute of CPU)."""
    w = I.workload(5)
    want = oracle.simulate(w["space"])
    got, out_dev, sp5, _ = run_simulate(w["space"])
    for f in ("status", "bmax", "n_iters", "n_req_iters") + tuple(guide.F64_OUTPUTS):     # the whole sweep, bit for bit
        assert np.array_equal(got[f].view(np.uint8), want[f].view(np.uint8)), f
    cons, k, key = w["constraints"], w["topk"]["k"], w["topk"]["key"]
    idx, val, cnt = run_topk(sp5, out_dev, cons, key, k)
    w_idx, w_val, w_cnt = oracle.select_topk(want, cons, key, k)
    assert cnt == w_cnt == k and np.array_equal(idx, w_idx)
    assert np.array_equal(val.view(np.uint64), w_val.view(np.uint64))
    fidx, fcnt = run_pareto(sp5, out_dev, cons, w["pareto"]["x"], w["pareto"]["y"])
    w_f, w_n = oracle.pareto(want, cons, w["pareto"]["x"], w["pareto"]["y"])
    assert fcnt == w_n and np.array_equal(fidx, w_f) and fcnt >= 2
    for key2, k2 in (("latency", 128), ("throughput", 8)):
        idx, val, cnt = run_topk(sp5, out_dev, {}, key2, k2)
        w_idx, w_val, w_cnt = oracle.select_topk(want, {}, key2, k2)
        assert cnt == w_cnt and np.array_equal(idx, w_idx)
    # the same step as one call: the sweep with both selections riding along
    del out_dev, got
    got, (idx, val, cnt), (fidx, fcnt), _, _ = run_simulate_select(w["space"], cons, key, k, cons, w["pareto"]["x"], w["pareto"]["y"])
    for f in ("status", "bmax", "n_iters", "n_req_iters") + tuple(guide.F64_OUTPUTS):
        assert np.array_equal(got[f].view(np.uint8), want[f].view(np.uint8)), f
    w_idx, w_val, w_cnt = oracle.select_topk(want, cons, key, k)
    assert cnt == w_cnt == k and np.array_equal(idx, w_idx) and np.array_equal(val.view(np.uint64), w_val.view(np.uint64))
    assert fcnt == w_n and np.array_equal(fidx, w_f)
