"""GPU parity, trace-driven continuous batching: warp-per-config kernel against the oracle."""
import numpy as np
import pytest

import oracle
from paper_2412_04788_b200 import guide, inputs as I
from gpu_util import assert_parity, bit_mismatches, run_simulate, run_topk

pytestmark = pytest.mark.gpu

SMALL = [4, 256, 8, 4, 512, 1000, 1, 2, 2, 2]


def toy_space(golden, mem, kv_block, batch):
    return I._space(np.array([golden["model"]]), np.array([golden["hw"]]), np.array([mem]), np.array([[1.0] * 7 + [0.0]]),
                    np.array([[1, kv_block, 0, 0]]), list(batch), [1], [(4, 3)])


def test_hand_worked_timelines(golden):
    for tl in golden["timelines"]:
        sp = toy_space(golden, tl["mem"], tl["kv_block"], [tl["max_batch"]])
        n = len(tl["arrival"])
        tr = {"arrival": np.array(tl["arrival"]), "in_len": np.zeros(n, np.uint32), "out_len": np.zeros(n, np.uint32)}
        got, *_ = run_simulate(sp, tr, per_request=True)
        assert got["status"][0] == 0
        for k in ("latency", "ttft", "ttft_p50", "ttft_p99", "tpot"):
            assert got[k][0] == tl[k], (tl["name"], k)
        assert got["req_ttft"][0].tolist() == tl["req_ttft"] and got["req_tpot"][0].tolist() == tl["req_tpot"]
        assert got["thr_decode"][0] == tl["dec_tok"] / tl["dec_time"]
        assert got["n_iters"][0] == tl["n_iters"] and got["n_req_iters"][0] == tl["n_req_iters"]


def test_workload1_full(golden):
    """504 configs x the 256-request trace, lengths taken from each config; every output incl. the
    per-request ones; then the top-8 by cost per token under the 500 ms p99-TTFT objective."""
    w = I.workload(1)
    want = oracle.simulate(w["space"], w["trace"], per_request=True)
    got, out_dev, sp, tr = run_simulate(w["space"], w["trace"], per_request=True)
    assert_parity(got, want, fields=guide.F64_OUTPUTS + ("req_ttft", "req_tpot"))
    assert sum(bit_mismatches(got, want, guide.F64_OUTPUTS + ("req_ttft", "req_tpot")).values()) == 0
    assert (want["status"] == 0).sum() > 100
    for key in ("cost_per_token", "cost_per_hr"):
        idx, val, cnt = run_topk(sp, out_dev, w["constraints"], key, 8, tr=tr)
        w_idx, w_val, w_cnt = oracle.select_topk(want, w["constraints"], key, 8)
        assert cnt == w_cnt and np.array_equal(idx, w_idx)
        assert np.array_equal(val.view(np.uint64), w_val.view(np.uint64))


def test_costs_are_price_times_gpus(golden):
    """Hand-worked hourly costs (price x t x dp in closed form, price x t on a trace) reach the GPU."""
    c = golden["costs"]
    model = list(golden["model"])
    model[2], model[3] = c["heads"], c["heads"]
    hw = list(golden["hw"])
    hw[4] = c["price_per_gpu_hr"]
    mk = lambda batch, tp, dp=None: I._space(np.array([model]), np.array([hw]), np.array([10**6]), np.array([[1.0] * 7 + [0.0]]),
                                             np.array([[1, 1, 0, 0]]), batch, tp, [(4, 3)], dp=dp)
    rows = c["closed_form"]
    got, *_ = run_simulate(mk([6], [r["t"] for r in rows], [r["dp"] for r in rows]))
    assert got["status"].tolist() == [0] * len(rows)
    assert got["cost_per_hr"].tolist() == [r["cost_per_hr"] for r in rows]
    assert got["cost_per_token"].tolist() == [(r["cost_per_hr"] / 3600.0) / thr for r, thr in zip(rows, got["thr_decode"])]
    rows = c["trace"]
    tr = {"arrival": np.array([0.0, 1.0, 1.5]), "in_len": np.zeros(3, np.uint32), "out_len": np.zeros(3, np.uint32)}
    got, *_ = run_simulate(mk([2], [r["t"] for r in rows]), tr)
    assert got["status"].tolist() == [0] * len(rows)
    assert got["cost_per_hr"].tolist() == [r["cost_per_hr"] for r in rows]
    assert got["cost_per_token"].tolist() == [(r["cost_per_hr"] / 3600.0) / thr for r, thr in zip(rows, got["thr_decode"])]


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_memory_pressure_small(seed):
    """Tiny model and memories, 4-token blocks: preemption and recompute happen in most configs."""
    n = 96
    tr = {"arrival": I.poisson_arrivals(seed, n, 3000.0), "in_len": I.randint(seed, 81, n, 1, 60).astype(np.uint32),
          "out_len": I.randint(seed, 82, n, 1, 40).astype(np.uint32)}
    hw, _ = I.seeded_hw(seed, 6, mem_gb=[1] * 6)
    w_bytes, kv_tok = oracle.weight_bytes_per_gpu(SMALL, 1), oracle.kv_bytes_per_token(SMALL, 1)
    mem = np.array([w_bytes + nb * 4 * kv_tok + 7 for nb in (20, 25, 26, 40, 90, 5000)], dtype=np.uint64)
    fw_f, fw_i = I.seeded_fw(seed, 2, kv_block=4, reserve_permille=0)
    sp = I._space(np.array([SMALL]), hw, mem, fw_f, fw_i, [1, 2, 5, 17, 64, 256], [1, 2, 4], [(1, 1)])
    want = oracle.simulate(sp, tr, per_request=True)
    got, *_ = run_simulate(sp, tr, per_request=True)
    assert_parity(got, want, fields=guide.F64_OUTPUTS + ("req_ttft", "req_tpot"))
    assert sum(bit_mismatches(got, want, guide.F64_OUTPUTS + ("req_ttft", "req_tpot")).values()) == 0
    assert want["n_preempt"].sum() > 0
    assert (want["status"] == guide.ST_KV).any() and (want["status"] == 0).any()


@pytest.mark.parametrize("policy", ["prefill_first", "split_fuse"])
def test_block_sizes_and_long_runs(policy):
    """Runs of several hundred decode iterations (the warp kernels take them 32 at a time) cut short
    by arrivals, completions and block shortages at every offset; block sizes that are not powers of
    two, one-token blocks, the largest the histogram covers and one beyond it; idle gaps between
    bursts of arrivals."""
    n = 72
    gaps = I.randint(5, 90, n, 0, 4)
    arrival = np.cumsum(np.where(gaps == 0, 0.02, 1e-5 * gaps))          # bursts, then a long pause
    tr = {"arrival": arrival, "in_len": I.randint(5, 91, n, 1, 90).astype(np.uint32),
          "out_len": I.randint(5, 92, n, 1, 400).astype(np.uint32)}
    blocks = [1, 3, 12, 64, 100]
    hw, _ = I.seeded_hw(5, 4, mem_gb=[1] * 4)
    w_bytes, kv_tok = oracle.weight_bytes_per_gpu(SMALL, 1), oracle.kv_bytes_per_token(SMALL, 1)
    mem = np.array([w_bytes + tokens * kv_tok + 3 for tokens in (600, 1500, 4000, 10**6)], dtype=np.uint64)
    fw_f, fw_i = I.seeded_fw(5, len(blocks), kv_block=4, reserve_permille=0)
    fw_i[:, 1] = blocks
    kw = {}
    if policy == "split_fuse":
        fw_i[:, 3] = guide.GUIDE_POLICY_SPLIT_FUSE
        kw["fw_chunk"] = [[0, 48]] * len(blocks)
    sp = I._space(np.array([SMALL]), hw, mem, fw_f, fw_i, [1, 2, 7, 40, 256], [1], [(1, 1)], **kw)
    want = oracle.simulate(sp, tr, per_request=True)
    got, *_ = run_simulate(sp, tr, per_request=True)
    fields = guide.F64_OUTPUTS + ("req_ttft", "req_tpot")
    assert_parity(got, want, fields=fields)
    assert sum(bit_mismatches(got, want, fields).values()) == 0
    ok = want["status"] == 0
    assert ok.sum() >= 40 and want["n_preempt"][ok].sum() > 0
    assert (want["n_iters"][ok] > 3000).any()                          # long schedules are in the sample


@pytest.mark.parametrize("k", [3, 4])
def test_workloads_3_and_4_reduced(k):
    """Workloads 3 and 4 with a shortened trace and one hardware profile in eight: same axes,
    laws and seeds, sized so the oracle takes seconds."""
    w = I.workload(k, scale=1 / 32 if k == 3 else 1 / 64, trace_scale=1 / 8 if k == 3 else 1 / 4)
    want = oracle.simulate(w["space"], w["trace"], per_request=(k == 3))
    got, *_ = run_simulate(w["space"], w["trace"], per_request=(k == 3))
    fields = guide.F64_OUTPUTS + (("req_ttft", "req_tpot") if k == 3 else ())
    assert_parity(got, want, fields=fields)
    assert sum(bit_mismatches(got, want, fields).values()) == 0
    assert (want["status"] == 0).sum() > 50


def test_lane_kernel_on_small_spaces():
    """The one-lane-per-config kernel is launched only for spaces with tens of thousands of configs of
    small max batch; GUIDE_LANE_MIN_CONFIGS=1 sends every such config of a small space to it.  The
    library reads the variable once per process, so the cases run in a child process: memory pressure
    with 4-token blocks, block sizes and long runs, the reduced workloads 3 and 4."""
    import os
    import subprocess
    import sys
    code = (
        "import sys; sys.path.insert(0, 'tests')\n"
        "import test_gpu_trace as t\n"
        "t.test_memory_pressure_small(2)\n"
        "t.test_block_sizes_and_long_runs('prefill_first')\n"
        "t.test_workloads_3_and_4_reduced(3)\n"
        "t.test_workloads_3_and_4_reduced(4)\n"
        "print('lane kernel ok')\n")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, "-c", code], cwd=root, env=dict(os.environ, GUIDE_LANE_MIN_CONFIGS="1"),
                         capture_output=True, text=True, timeout=900)
    assert res.returncode == 0 and "lane kernel ok" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]


def test_iteration_cap_and_models(golden):
    sp = toy_space(golden, 10**6, 1, [1])
    tr = {"arrival": np.array([0.0, 1.0]), "in_len": np.zeros(2, np.uint32), "out_len": np.zeros(2, np.uint32)}
    got, *_ = run_simulate(sp, tr, max_iters=5)
    assert got["status"][0] == guide.ST_ITER and np.isinf(got["latency"][0])
    got, *_ = run_simulate(sp, tr, max_iters=6)
    assert got["status"][0] == 0
    w = I.workload(1, scale=1.0, trace_scale=0.25)
    for tm, tpm in ((1, 0), (0, 1)):
        want = oracle.simulate(w["space"], w["trace"], time_model=tm, tp_model=tpm)
        got, *_ = run_simulate(w["space"], w["trace"], time_model=tm, tp_model=tpm)
        assert_parity(got, want)
        assert sum(bit_mismatches(got, want).values()) == 0


@pytest.mark.parametrize("policy", ["prefill_first", "split_fuse"])
def test_iteration_cap_inside_long_runs(policy):
    """The iteration cap can fall anywhere in a run that the warp kernels take 32 iterations at a time:
    caps around the batch boundaries, one below the schedule's length and exactly its length."""
    n = 6
    tr = {"arrival": np.zeros(n), "in_len": np.full(n, 5, np.uint32), "out_len": np.array([40, 70, 33, 65, 97, 129], np.uint32)}
    hw, _ = I.seeded_hw(3, 1, mem_gb=[1])
    fw_f, fw_i = I.seeded_fw(3, 1, kv_block=4, reserve_permille=0)
    kw = {}
    if policy == "split_fuse":
        fw_i[:, 3] = guide.GUIDE_POLICY_SPLIT_FUSE
        kw["fw_chunk"] = [[0, 16]]
    sp = I._space(np.array([SMALL]), hw, np.array([10**9], dtype=np.uint64), fw_f, fw_i, [1, 2, 8], [1], [(1, 1)], **kw)
    full = oracle.simulate(sp, tr)
    assert (full["status"] == 0).all()
    caps = sorted({1, 2, 31, 32, 33, 34, 63, 64, 65, 66, 96, 97, 128, 129, 130}
                  | {int(v) + d for v in full["n_iters"] for d in (-1, 0, 1)})
    for cap in caps:
        want = oracle.simulate(sp, tr, max_iters=cap)
        got, *_ = run_simulate(sp, tr, max_iters=cap)
        assert np.array_equal(got["status"], want["status"]), cap
        assert np.array_equal(got["n_iters"], want["n_iters"]), cap
        assert sum(bit_mismatches(got, want).values()) == 0, cap


def test_run_to_run_identical():
    """The same launch twice gives the same bits (no dependence on scheduling order)."""
    w = I.workload(4, scale=1 / 64, trace_scale=1 / 4)
    a, *_ = run_simulate(w["space"], w["trace"])
    b, *_ = run_simulate(w["space"], w["trace"])
    for k in guide.F64_OUTPUTS:
        assert np.array_equal(a[k].view(np.uint64), b[k].view(np.uint64))


@pytest.mark.parametrize("k,stride", [(3, 5), (4, 3)])
def test_full_size_trace_workloads_sampled(k, stride):
    """Workloads 3 and 4 at full size in the launch shape the benchmark times (whole space, so the
    heaviest-first work order is on); every `stride`-th config is recomputed by the oracle and must
    match bit for bit, per-request values included for workload 3.  The strides are odd primes, so
    the sample visits every position of every axis.  GUIDE_TRACE_PARITY_STRIDE overrides the stride (1 = every config of both workloads: about three
    minutes on a 16-core host)."""
    import os
    import torch
    stride = int(os.environ.get("GUIDE_TRACE_PARITY_STRIDE", stride))      # 1 = every config (minutes of oracle time)
    w = I.workload(k)
    sp, tr = guide.Space(w["space"]), guide.Trace(w["trace"])
    n = sp.size
    out = guide.alloc_outputs(n, tr.n, per_request=(k == 3))
    ws = torch.empty(guide.guide_workspace_bytes(sp, tr), dtype=torch.uint8, device="cuda")
    guide.guide_simulate(sp, tr, out, workspace=ws)
    torch.cuda.synchronize()
    count = (n + stride - 1) // stride
    want = oracle.simulate(w["space"], w["trace"], first=0, count=count, stride=stride, per_request=(k == 3))
    for f in guide.F64_OUTPUTS:
        got = out[f][::stride].cpu().numpy()
        assert np.array_equal(got.view(np.uint64), want[f].view(np.uint64)), f
    assert np.array_equal(out["status"][::stride].cpu().numpy(), want["status"])
    assert np.array_equal(out["bmax"][::stride].cpu().numpy().view(np.uint32), want["bmax"])
    assert np.array_equal(out["n_iters"][::stride].cpu().numpy().view(np.uint64), want["n_iters"])
    assert np.array_equal(out["n_req_iters"][::stride].cpu().numpy().view(np.uint64), want["n_req_iters"])
    if k == 3:
        assert np.array_equal(out["req_ttft"][::stride].cpu().numpy().view(np.uint64), want["req_ttft"].view(np.uint64))
        assert np.array_equal(out["req_tpot"][::stride].cpu().numpy().view(np.uint64), want["req_tpot"].view(np.uint64))
    # properties over the whole result
    ok = out["status"] == 0
    assert 0 < int(ok.sum()) <= n
    assert bool((out["ttft_p50"][ok] <= out["ttft_p99"][ok]).all())
    assert bool(torch.isfinite(out["latency"][ok]).all()) and bool(torch.isinf(out["latency"][~ok]).all())
    if k == 4:
        assert want["n_preempt"].sum() > 0          # the sampled configs include evictions


def test_block_sizes_outside_the_histogram_path():
    """KV blocks of 100 and 65 tokens (above the 64-entry phase histogram: needs are counted by a
    slot scan and iterations are not bursted), next to 1, 3, 64: all against the oracle."""
    n = 80
    tr = {"arrival": I.poisson_arrivals(9, n, 2500.0), "in_len": I.randint(9, 81, n, 1, 300).astype(np.uint32),
          "out_len": I.randint(9, 82, n, 1, 150).astype(np.uint32)}
    hw, _ = I.seeded_hw(9, 3, mem_gb=[1] * 3)
    w_bytes, kv_tok = oracle.weight_bytes_per_gpu(SMALL, 1), oracle.kv_bytes_per_token(SMALL, 1)
    mem = np.array([w_bytes + tok * kv_tok for tok in (1000, 3000, 200000)], dtype=np.uint64)
    fw_f, fw_i = I.seeded_fw(9, 5, reserve_permille=0)
    fw_i[:, 1] = [100, 65, 1, 3, 64]
    sp = I._space(np.array([SMALL]), hw, mem, fw_f, fw_i, [1, 4, 33, 256], [1, 2], [(1, 1)])
    want = oracle.simulate(sp, tr, per_request=True)
    got, *_ = run_simulate(sp, tr, per_request=True)
    fields = guide.F64_OUTPUTS + ("req_ttft", "req_tpot")
    assert_parity(got, want, fields=fields)
    assert sum(bit_mismatches(got, want, fields).values()) == 0
    assert want["n_preempt"].sum() > 0 and (want["status"] == 0).sum() >= 40


def test_counts_beyond_2_to_53_use_the_integer_path():
    """64 KiB KV elements and 16k-token prompts: with a few hundred residents the per-iteration KV
    read count exceeds 2^53, so it cannot be carried as an exact double; the kernel must fall back
    to the integer form (the small-batch configs of the same space stay on the fast path) and
    still agree with the oracle bit for bit."""
    fat = [1, 2**15, 2**5, 2**5, 16, 64, 1, 2, 2, 2**16]
    n = 300
    tr = {"arrival": np.zeros(n), "in_len": (2**14 - np.arange(n)).astype(np.uint32),
          "out_len": (2 + np.arange(n) % 3).astype(np.uint32)}
    hw, _ = I.seeded_hw(4, 2, mem_gb=[1, 1])
    mem = np.array([2**61, 2**62], dtype=np.uint64)
    fw_f, fw_i = I.seeded_fw(4, 2)
    fw_i[1, 0] = 0                      # one profile without FlashAttention: score-matrix terms too
    sp = I._space(np.array([fat]), hw, mem, fw_f, fw_i, [2, 256], [1, 4], [(1, 1)])
    assert 256 * (2**14 + 5) * 2**15 * 2**16 >= 2**53          # the premise, for max batch 256
    want = oracle.simulate(sp, tr, per_request=True)
    assert (want["status"] == 0).all()
    got, *_ = run_simulate(sp, tr, per_request=True)
    fields = guide.F64_OUTPUTS + ("req_ttft", "req_tpot")
    assert_parity(got, want, fields=fields)
    assert sum(bit_mismatches(got, want, fields).values()) == 0


def test_single_request_and_single_config():
    tr = {"arrival": np.array([0.25]), "in_len": np.array([17], np.uint32), "out_len": np.array([1], np.uint32)}
    hw, mem = I.seeded_hw(2, 1, mem_gb=[8])
    fw_f, fw_i = I.seeded_fw(2, 1)
    sp = I._space(np.array([SMALL]), hw, mem, fw_f, fw_i, [1], [1], [(1, 1)])
    want = oracle.simulate(sp, tr, per_request=True)
    got, *_ = run_simulate(sp, tr, per_request=True)
    assert_parity(got, want, fields=guide.F64_OUTPUTS + ("req_ttft", "req_tpot"))
    assert got["n_iters"][0] == 1 and got["thr_decode"][0] == 0.0 and np.isinf(got["cost_per_token"][0])
