"""GPU parity of the split-and-fuse scheduling policy of the trace simulation (token budget per
iteration, prompts chunked in arrival order and fused with decoding; Sec. 2.3.2 / Sec. 3.1)."""
import numpy as np
import pytest

import oracle
from paper_2412_04788_b200 import guide, inputs as I
from gpu_util import assert_parity, bit_mismatches, run_simulate

pytestmark = pytest.mark.gpu

SMALL = [2, 64, 4, 2, 128, 100, 1, 2, 2, 2]


def fuse_space(space, budgets):
    """the space with every framework on the split-and-fuse policy (budgets: tokens per iteration)"""
    sp = dict(space)
    fw_i = np.array(space["fw_i"], dtype=np.uint32).copy()
    fw_i[:, 3] = guide.GUIDE_POLICY_SPLIT_FUSE
    sp["fw_i"] = fw_i
    sp["fw_chunk"] = np.array([[0, bgt] for bgt in budgets], dtype=np.uint32)
    return sp


def check(space, trace, what, per_request=True):
    want = oracle.simulate(space, trace, per_request=per_request)
    got, *_ = run_simulate(space, trace, per_request=per_request)
    fields = guide.F64_OUTPUTS + (("req_ttft", "req_tpot") if per_request else ())
    assert_parity(got, want, fields=fields, what=what)
    assert sum(bit_mismatches(got, want, fields=fields).values()) == 0
    return want


def test_hand_worked_timeline():
    tr = {"arrival": np.array([0.0, 0.0]), "in_len": np.array([6, 3], np.uint32), "out_len": np.array([3, 2], np.uint32)}
    hw, _ = I.seeded_hw(7, 1, mem_gb=[1])
    fw_f, fw_i = I.seeded_fw(7, 1, kv_block=4, reserve_permille=0)
    fw_i[0, 3] = guide.GUIDE_POLICY_SPLIT_FUSE
    sp = I._space(np.array([SMALL]), hw, np.array([10**9]), fw_f, fw_i, [4], [1], [(1, 1)], fw_chunk=[[0, 4]])
    want = check(sp, tr, "timeline ")
    assert want["n_iters"][0] == 4 and want["n_req_iters"][0] == 7


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_traces_under_memory_pressure(seed):
    """Tiny memories force evictions in both phases of a request; budgets from one token to more
    than everything waiting; all block counts x batch limits x budgets as one space."""
    n = 40
    tr = {"arrival": I.poisson_arrivals(seed, n, 2000.0),
          "in_len": I.randint(seed, 81, n, 1, 60).astype(np.uint32),
          "out_len": I.randint(seed, 82, n, 1, 30).astype(np.uint32)}
    w_bytes = oracle.weight_bytes_per_gpu(SMALL, 1)
    kv_tok = oracle.kv_bytes_per_token(SMALL, 1)
    mems = [w_bytes + nb * 4 * kv_tok + 5 for nb in (23, 31, 60, 1000)]
    hw, _ = I.seeded_hw(seed, 4, mem_gb=[1] * 4)
    fw_f, fw_i = I.seeded_fw(seed, 5, kv_block=4, reserve_permille=0)
    fw_i[:, 3] = guide.GUIDE_POLICY_SPLIT_FUSE
    fw_i[4, 1] = 1                                                         # unpaged
    sp = I._space(np.array([SMALL]), hw, np.array(mems), fw_f, fw_i, [1, 3, 8, 32], [1, 2], [(1, 1)],
                  fw_chunk=[[0, 1], [0, 5], [0, 16], [0, 64], [0, 7]])
    want = oracle.simulate(sp, tr, per_request=True)
    got, *_ = run_simulate(sp, tr, per_request=True)
    fields = guide.F64_OUTPUTS + ("req_ttft", "req_tpot")
    assert_parity(got, want, fields=fields)
    assert sum(bit_mismatches(got, want, fields=fields).values()) == 0
    assert (want["n_preempt"] > 0).any() and (want["status"] == 0).all()


def test_mixed_policies_workload_1():
    """Workload 1 with a second framework on split-and-fuse next to the prompt-first one: the two
    schedulers side by side in one launch, requests taking the config's lengths."""
    w = I.workload(1)
    sp = dict(w["space"])
    sp["fw_f"] = np.concatenate([sp["fw_f"], sp["fw_f"]])
    fw_i = np.concatenate([sp["fw_i"], sp["fw_i"]]).astype(np.uint32)
    fw_i[1, 3] = guide.GUIDE_POLICY_SPLIT_FUSE
    sp["fw_i"] = fw_i
    sp["fw_chunk"] = np.array([[0, 0], [0, 512]], dtype=np.uint32)
    want = check(sp, w["trace"], "C1 mixed ")
    plain = oracle.simulate(w["space"], w["trace"])
    st = want["status"].reshape(4, 2, -1)
    assert np.array_equal(want["latency"].reshape(4, 2, -1)[:, 0], plain["latency"].reshape(4, 1, -1)[:, 0])
    ok = (st[:, 0] == 0) & (st[:, 1] == 0)
    assert (want["ttft_p99"].reshape(4, 2, -1)[:, 1][ok] != want["ttft_p99"].reshape(4, 2, -1)[:, 0][ok]).any()


def test_lognormal_trace_workload_3_small():
    w = I.workload(3, scale=1 / 32, trace_scale=1 / 8)                    # 1 hw x 4 fw ... x 512 requests
    sp = fuse_space(w["space"], [256, 512, 2048, 8192])
    check(sp, w["trace"], "C3 small ", per_request=False)


def test_iteration_limit_and_bad_profiles():
    tr = {"arrival": np.array([0.0, 1.0]), "in_len": np.zeros(2, np.uint32), "out_len": np.zeros(2, np.uint32)}
    hw, _ = I.seeded_hw(7, 1, mem_gb=[1])
    fw_f, fw_i = I.seeded_fw(7, 1, kv_block=4, reserve_permille=0)
    fw_i[0, 3] = guide.GUIDE_POLICY_SPLIT_FUSE
    sp = I._space(np.array([SMALL]), hw, np.array([10**9]), fw_f, fw_i, [1], [1], [(4, 3)], fw_chunk=[[0, 2]])
    want = oracle.simulate(sp, tr)
    assert want["n_iters"][0] == 2 * (2 + 2)                              # two chunks and two decode steps per request
    for cap in (7, 8):
        w_cap = oracle.simulate(sp, tr, max_iters=cap)
        got, *_ = run_simulate(sp, tr, max_iters=cap)
        assert got["status"][0] == w_cap["status"][0] == (guide.ST_ITER if cap == 7 else 0)
    for chunk in ([[0, 0]], [[2, 4]]):                                    # no budget; a sub-batch size
        with pytest.raises(guide.GuideError) as e:
            run_simulate(I._space(np.array([SMALL]), hw, np.array([10**9]), fw_f, fw_i, [1], [1], [(4, 3)], fw_chunk=chunk), tr)
        assert e.value.code == guide.GUIDE_ERR_INVALID


def test_benchmark_case_sampled():
    """The case bench.py times: workload 3 on half of its hardware axis (32,768 configs x 4096
    requests), every framework on the split-and-fuse policy with token budgets 256 .. 8192, in one
    launch; every 29th config is recomputed by the oracle and must match bit for bit, per-request
    values included.  GUIDE_TRACE_PARITY_STRIDE overrides the stride."""
    import os
    import torch
    stride = int(os.environ.get("GUIDE_TRACE_PARITY_STRIDE", 29))
    w = I.workload(3, scale=0.5, trace_scale=1.0)
    space = fuse_space(w["space"], [256, 512, 2048, 8192])
    sp, tr = guide.Space(space), guide.Trace(w["trace"])
    n = sp.size
    out = guide.alloc_outputs(n, tr.n, per_request=True)
    ws = torch.empty(guide.guide_workspace_bytes(sp, tr), dtype=torch.uint8, device="cuda")
    guide.guide_simulate(sp, tr, out, workspace=ws)
    torch.cuda.synchronize()
    count = (n + stride - 1) // stride
    want = oracle.simulate(space, w["trace"], first=0, count=count, stride=stride, per_request=True)
    for f in guide.F64_OUTPUTS + ("req_ttft", "req_tpot"):
        got = out[f][::stride].cpu().numpy()
        assert np.array_equal(got.view(np.uint64), want[f].view(np.uint64)), f
    assert np.array_equal(out["status"][::stride].cpu().numpy(), want["status"])
    assert np.array_equal(out["n_iters"][::stride].cpu().numpy().view(np.uint64), want["n_iters"])
    assert np.array_equal(out["n_req_iters"][::stride].cpu().numpy().view(np.uint64), want["n_req_iters"])
    assert int((out["status"] == 0).sum()) > n // 2
