"""GPU parity, closed form: the CUDA kernels against the oracle, element by element."""
import numpy as np
import pytest

import oracle
from paper_2412_04788_b200 import guide, inputs as I
from gpu_util import assert_parity, bit_mismatches, run_simulate

pytestmark = pytest.mark.gpu


def test_toy_matches_hand_worked_values(golden):
    sp = I._space(np.array([golden["model"]]), np.array([golden["hw"]]), np.array([10**6]),
                  np.array([[1.0] * 7 + [0.0]]), np.array([[1, 1, 0, 0]]), [2], [1, 2], [(4, 3)])
    got, *_ = run_simulate(sp)
    want = golden["closed_form_b2_Lin4_Lout3"]["t1"]
    assert got["status"].tolist() == [0, guide.ST_HEADS]
    assert got["ttft"][0] == want["ttft"] and got["latency"][0] == want["latency"] and got["tpot"][0] == want["tpot"]


@pytest.mark.parametrize("k", [1, 2, 5])
def test_workload_closed_form_small(k):
    """Workloads 1, 2 and 5 with a shrunken hardware axis: whole space, all outputs."""
    w = I.workload(k, scale=0.25 if k != 5 else 1 / 16)
    want = oracle.simulate(w["space"])
    got, *_ = run_simulate(w["space"])
    assert_parity(got, want, what=f"C{k} ")
    assert sum(bit_mismatches(got, want).values()) == 0
    assert (want["status"] == 0).any() and (want["status"] != 0).any()


def test_flat_and_tiled_kernels_agree_on_ranges():
    """A sub-range goes through the one-thread-per-config kernel, the whole space through the
    tiled one; ragged first/count values straddle tiles."""
    w = I.workload(2, scale=0.125)
    want = oracle.simulate(w["space"])
    n = len(want["status"])
    for first, count in ((0, 0), (0, 1), (7, 1000), (n - 333, 333), (12345, 7777), (1, n - 1)):
        got, *_ = run_simulate(w["space"], first=first, count=count)
        c = count or n - first
        sub = {k: v[first:first + c] for k, v in want.items()}
        assert_parity(got, sub, what=f"[{first},{count}) ")
        assert sum(bit_mismatches(got, sub).values()) == 0


@pytest.mark.parametrize("time_model,tp_model", [(1, 0), (0, 1), (1, 1)])
def test_time_and_tp_models(time_model, tp_model):
    w = I.workload(2, scale=0.125)
    want = oracle.simulate(w["space"], time_model=time_model, tp_model=tp_model)
    got, *_ = run_simulate(w["space"], time_model=time_model, tp_model=tp_model)
    assert_parity(got, want)
    assert sum(bit_mismatches(got, want).values()) == 0


def test_ragged_tile_shapes():
    """(TP, length) planes that do not fill a warp or a block, unpaged and odd block sizes."""
    hw, mem = I.seeded_hw(3, 3, mem_gb=[24, 80, 192])
    fw_f, fw_i = I.seeded_fw(3, 2, kv_block=1)
    fw_i[1, 1] = 24
    for tp, lins, louts in (([1], [100], [1]), ([1, 2, 8], [1, 77, 3000], [1, 2, 300, 333, 1000]),
                            ([1, 2, 4, 8, 16], list(range(10, 400, 13)), [5, 6, 7, 500])):
        sp = I._space(I.models_from_shapes(I.SHAPES_8[1:4]), hw, mem, fw_f, fw_i, [1, 3, 200], tp, I.pairs_grid(lins, louts))
        want = oracle.simulate(sp)
        got, *_ = run_simulate(sp)
        assert_parity(got, want)
        assert sum(bit_mismatches(got, want).values()) == 0


def test_null_outputs_are_skipped():
    import torch
    w = I.workload(1)
    sp = guide.Space(w["space"])
    out = {"latency": torch.empty(sp.size, dtype=torch.float64, device="cuda"),
           "status": torch.empty(sp.size, dtype=torch.uint8, device="cuda")}
    guide.guide_simulate(sp, None, out)
    torch.cuda.synchronize()
    want = oracle.simulate(w["space"])
    assert np.array_equal(out["status"].cpu().numpy(), want["status"])
    assert np.array_equal(out["latency"].cpu().numpy(), want["latency"])


def test_split_kernels_mixed_block_sizes_and_ragged_plane():
    """A whole space of 216,000 configs goes through the memory kernel + model kernel pair: three KV
    block sizes (unpaged, 16, 24) so the sorted pair walk has three segments, a (TP, length) plane
    of 60 positions that fills neither a 64-wide group nor a 256-wide tile, small memories so that
    most foursomes are mixed."""
    hw, mem = I.seeded_hw(11, 40, mem_choices=[16, 24, 48, 80])
    fw_f, fw_i = I.seeded_fw(12, 3, kv_block=16)
    fw_i[0, 1] = 1
    fw_i[2, 1] = 24
    sp = I._space(I.models_from_shapes(I.SHAPES_8[0:6]), hw, mem, fw_f, fw_i, [1, 3, 17, 64, 200], [1, 2, 4, 8, 16],
                  I.pairs_grid([64, 700, 3000], [1, 2, 130, 4000]))
    want = oracle.simulate(sp)
    assert len(want["status"]) == 216000
    for tm, tpm in ((0, 0), (1, 1)):
        want = oracle.simulate(sp, time_model=tm, tp_model=tpm)
        got, *_ = run_simulate(sp, time_model=tm, tp_model=tpm)
        assert_parity(got, want)
        assert sum(bit_mismatches(got, want).values()) == 0
    assert (want["status"] == 0).any() and (want["status"] != 0).any()


def test_line_kernels_mixed_block_sizes_and_output_subsets():
    """4,915,200 configs, enough lines per resident warp for the pair of kernels that shares out
    128-byte lines: three KV block sizes (three segments in the sorted pair walk, four chunks of
    pairs), a TP degree that does not divide every model's heads, memories small enough that most
    lines are mixed; then calls with only some output arrays."""
    import torch
    hw, mem = I.seeded_hw(21, 80, mem_choices=[16, 24, 48, 80, 192])
    fw_f, fw_i = I.seeded_fw(22, 3, kv_block=16)
    fw_i[0, 1] = 1
    fw_i[2, 1] = 24
    sp_np = I._space(I.models_from_shapes(I.SHAPES_8), hw, mem, fw_f, fw_i,
                     [1, 2, 3, 5, 8, 13, 17, 32, 50, 64, 100, 128, 200, 256, 400, 512], [1, 2, 4, 8, 16],
                     I.pairs_grid([64, 700, 3000, 8000], [1, 2, 64, 130, 500, 1000, 2000, 4000]))
    assert len(sp_np["pairs"]) % 16 == 0
    for tm, tpm in ((0, 0), (1, 1)):
        want = oracle.simulate(sp_np, time_model=tm, tp_model=tpm)
        assert len(want["status"]) == 4915200
        got, *_ = run_simulate(sp_np, time_model=tm, tp_model=tpm)
        assert_parity(got, want)
        assert sum(bit_mismatches(got, want).values()) == 0
    ok = want["status"] == 0
    assert 0.05 < ok.mean() < 0.95 and (want["status"] & guide.ST_HEADS).any()
    lines = ok.reshape(-1, 16)
    assert (lines.any(axis=1) & ~lines.all(axis=1)).mean() > 0.05          # mixed lines: constants next to metrics
    want = oracle.simulate(sp_np)
    sp = guide.Space(sp_np)
    n = sp.size
    for fields in (("latency",), ("status", "bmax"), ("thr_decode", "cost_per_token", "n_iters"),
                   ("ttft_p50", "ttft_p99", "status", "n_req_iters"), ("cost_per_hr", "tpot")):
        out = guide.alloc_outputs(n, fields=fields)
        for t in out.values():
            t.fill_(7)
        guide.guide_simulate(sp, None, out)
        torch.cuda.synchronize()
        for f in fields:
            g = out[f].cpu().numpy()
            x = want["ttft"] if f in ("ttft_p50", "ttft_p99") else want[f]
            assert np.array_equal(g.view(np.uint8), x.view(np.uint8)), (fields, f)
    # arrays that do not start on a 128-byte boundary go through the kernels that share out sectors
    base = torch.empty(n + 4, dtype=torch.float64, device="cuda")
    out = {"latency": base[4:], "status": torch.empty(n, dtype=torch.uint8, device="cuda")}
    guide.guide_simulate(sp, None, out)
    torch.cuda.synchronize()
    assert np.array_equal(out["latency"].cpu().numpy().view(np.uint64), want["latency"].view(np.uint64))


def test_split_kernels_output_subsets():
    """Whole-space calls with only some output arrays: each kernel of the pair must skip the rest."""
    import torch
    w = I.workload(2, scale=0.125)
    want = oracle.simulate(w["space"])
    sp = guide.Space(w["space"])
    n = sp.size
    assert n >= 65536
    for fields in (("latency",), ("status", "bmax"), ("thr_decode", "cost_per_token", "n_iters"), ("ttft_p99", "status", "n_req_iters")):
        out = guide.alloc_outputs(n, fields=fields)
        for t in out.values():
            t.fill_(7)
        guide.guide_simulate(sp, None, out)
        torch.cuda.synchronize()
        for f in fields:
            g = out[f].cpu().numpy()
            x = want["ttft"] if f == "ttft_p99" else want[f]
            assert np.array_equal(g.view(np.uint8), x.view(np.uint8)), (fields, f)


def test_full_size_grid_983040():
    """Workload 2 at full size in the launch shape the benchmark times; compared in full."""
    w = I.workload(2)
    want = oracle.simulate(w["space"])
    got, *_ = run_simulate(w["space"])
    assert len(got["status"]) == 983040
    assert_parity(got, want)
    assert sum(bit_mismatches(got, want).values()) == 0


def test_full_size_sweep_sampled():
    """Workload 5 (16.7M configs) in the benchmark's launch shape: every 4099th config against
    the oracle, plus whole-array properties (TTFT <= latency, infeasible <=> non-finite)."""
    import torch
    w = I.workload(5)
    sp = guide.Space(w["space"])
    n = sp.size
    out = guide.alloc_outputs(n, fields=("latency", "ttft", "thr_decode", "cost_per_token", "status", "bmax"))
    guide.guide_simulate(sp, None, out)
    torch.cuda.synchronize()
    stride = 4099
    count = (n + stride - 1) // stride
    want = oracle.simulate(w["space"], first=0, count=count, stride=stride)
    for k in ("latency", "ttft", "thr_decode", "cost_per_token"):
        assert np.array_equal(out[k][::stride].cpu().numpy().view(np.uint64), want[k].view(np.uint64)), k
    assert np.array_equal(out["status"][::stride].cpu().numpy(), want["status"])
    assert np.array_equal(out["bmax"][::stride].cpu().numpy().view(np.uint32), want["bmax"])
    ok = out["status"] == 0
    assert bool((out["ttft"][ok] <= out["latency"][ok]).all())
    assert bool(torch.isinf(out["latency"][~ok]).all()) and bool(torch.isfinite(out["latency"][ok]).all())
    assert 0 < int(ok.sum()) < n
