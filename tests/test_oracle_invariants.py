"""Invariants of the model and brute-force cross-checks of the oracle on tiny inputs."""
import numpy as np
import pytest

import oracle
from oracle import naive
from paper_2412_04788_b200 import inputs as I

LL = [32, 4096, 32, 32, 11008, 32000, 1, 2, 2, 2]
SMALL = [4, 256, 8, 4, 512, 1000, 1, 2, 2, 2]


def grid_space(seed=3, model=LL, mem_gb=(24, 80), batch=(1, 2, 4, 8, 16), tp=(1, 2, 4), lins=(64, 128, 512, 2048),
               louts=(1, 2, 64, 256), n_fw=2, kv_block=16):
    hw, mem = I.seeded_hw(seed, len(mem_gb), mem_gb=list(mem_gb))
    fw_f, fw_i = I.seeded_fw(seed, n_fw, kv_block=kv_block)
    return I._space(np.array([model]), hw, mem, fw_f, fw_i, list(batch), list(tp), I.pairs_grid(lins, louts))


def test_monotone_in_batch_and_lengths():
    """Latency and TTFT never decrease with batch size, prompt length or output length
    (round-to-nearest is monotone, so this holds bit for bit on feasible neighbours)."""
    sp = grid_space()
    out = oracle.simulate(sp)
    shape = (2, 2, 5, 3, 4, 4)          # hw, fw, batch, tp, Lin, Lout
    lat = np.where(out["status"] == 0, out["latency"], np.nan).reshape(shape)
    ttft = np.where(out["status"] == 0, out["ttft"], np.nan).reshape(shape)
    for arr in (lat, ttft):
        for axis in (2, 4, 5):
            d = np.diff(arr, axis=axis)
            assert np.all((d >= 0) | np.isnan(d))
    ok = out["status"] == 0
    assert ok.sum() > 400
    assert np.all(out["ttft"][ok] <= out["latency"][ok])
    assert np.all(out["ttft"][ok] > 0)


def test_feasibility_is_exactly_weights_plus_kv_within_capacity():
    sp = grid_space(mem_gb=(16, 24, 48), batch=(1, 8, 64, 512), tp=(1, 2, 3 + 1, 64))
    out = oracle.simulate(sp)
    n = I.space_size(sp)
    for idx in range(n):
        m, h, f, b, t, l = I.decode_index(sp, idx)
        tp, batch = int(sp["tp"][t]), int(sp["batch"][b])
        lin, lout = (int(x) for x in sp["pairs"][l])
        usable = oracle.usable_bytes(int(sp["hw_mem"][h]), int(sp["fw_i"][f][2]))
        w = oracle.weight_bytes_per_gpu(LL, tp)
        kv = oracle.kv_bytes_per_token(LL, tp)
        blk = int(sp["fw_i"][f][1])
        s_blk = -(-(lin + lout) // blk) * blk
        fits = usable > w and w + batch * s_blk * kv <= usable and 32 % tp == 0
        assert (out["status"][idx] == 0) == fits, idx


def test_max_le_sum_le_twice_max():
    sp = grid_space(mem_gb=(80,), tp=(1, 2))
    a = oracle.simulate(sp, time_model=oracle.TIME_MAX)
    b = oracle.simulate(sp, time_model=oracle.TIME_SUM)
    ok = a["status"] == 0
    assert np.array_equal(a["status"], b["status"])
    assert np.all(a["latency"][ok] <= b["latency"][ok])
    assert np.all(b["latency"][ok] <= 2 * a["latency"][ok])


def test_tp_communication_term_is_additive():
    """With a free interconnect TP only divides work; latency(t=2) is then at most latency(t=1).
    A slow interconnect makes small prompts slower under TP (the TTFT rise of Sec. 2.4.3)."""
    hw = np.array([[4e14, 2e12, 1e18, 0.0, 3.0], [4e14, 2e12, 2e9, 2e-5, 3.0]])
    fw_f, fw_i = I.seeded_fw(9, 1)
    sp = I._space(np.array([LL]), hw, np.array([80 * I.GB] * 2), fw_f, fw_i, [1], [1, 2], [(128, 64)])
    out = oracle.simulate(sp)
    ttft = out["ttft"].reshape(2, 2)
    assert ttft[0, 1] < ttft[0, 0]
    assert ttft[1, 1] > ttft[1, 0]


def _iter_time(model, sp, h, f, t):
    hw, ff, fi = sp["hw"][h], sp["fw_f"][f], sp["fw_i"][f]
    return lambda T, E, A, Cc: oracle.phase_time(model, hw, ff, fi, t, T, E, A, Cc, 1)[0]


@pytest.mark.parametrize("seed", [1, 2, 3, 4])
def test_trace_sim_against_naive_scheduler(seed):
    """Random tiny traces under memory pressure: the oracle's index-pointer queue and counters
    against an explicit scheduler with request objects, a waiting list and a block free list."""
    n = 24
    arrival = I.poisson_arrivals(seed, n, 2000.0)
    in_len = I.randint(seed, 81, n, 1, 40).astype(np.uint32)
    out_len = I.randint(seed, 82, n, 1, 24).astype(np.uint32)
    tr = {"arrival": arrival, "in_len": in_len, "out_len": out_len}
    hw, _ = I.seeded_hw(seed, 1, mem_gb=[1])
    fw_f, fw_i = I.seeded_fw(seed, 1, kv_block=4, reserve_permille=0)
    w_bytes = oracle.weight_bytes_per_gpu(SMALL, 1)
    kv_tok = oracle.kv_bytes_per_token(SMALL, 1)
    total_preempt = 0
    for n_blocks in (16, 23, 40, 400):
        mem = w_bytes + n_blocks * 4 * kv_tok + 5       # 5 spare bytes: floor must drop them
        for b in (1, 3, 8):
            sp = I._space(np.array([SMALL]), hw, np.array([mem]), fw_f, fw_i, [b], [1], [(1, 1)])
            got = oracle.simulate(sp, tr, per_request=True)
            assert got["status"][0] == 0
            ref = naive.trace_sim(arrival.tolist(), in_len.tolist(), out_len.tolist(), b, n_blocks, 4,
                                  _iter_time(SMALL, sp, 0, 0, 1))
            assert got["latency"][0] == ref["makespan"]
            ttft = np.array(ref["first"]) - arrival
            assert np.array_equal(got["req_ttft"][0], ttft)
            tpot = [(fi - fr) / (o - 1) if o > 1 else 0.0 for fi, fr, o in zip(ref["finish"], ref["first"], out_len)]
            assert np.array_equal(got["req_tpot"][0], np.array(tpot))
            assert got["n_iters"][0] == ref["n_iters"] and got["n_req_iters"][0] == ref["n_req_iters"]
            assert got["n_preempt"][0] == ref["n_preempt"]
            assert got["thr_decode"][0] == (ref["dec_tok"] / ref["dec_time"] if ref["dec_time"] else 0.0)
            assert ref["max_running"] <= b
            s = 0.0
            for v in ttft:
                s = s + v
            assert got["ttft"][0] == s / n
            srt = np.sort(ttft)
            assert got["ttft_p50"][0] == srt[(50 * n + 99) // 100 - 1]
            assert got["ttft_p99"][0] == srt[(99 * n + 99) // 100 - 1]
            total_preempt += ref["n_preempt"]
            if n_blocks == 400:
                assert ref["n_preempt"] == 0          # room for every request at once
    assert total_preempt > 0                           # the pressure cases really preempt


def test_trace_sim_request_too_large_is_infeasible():
    tr = {"arrival": np.array([0.0, 0.1]), "in_len": np.array([8, 100], np.uint32), "out_len": np.array([4, 30], np.uint32)}
    hw, _ = I.seeded_hw(1, 1, mem_gb=[1])
    fw_f, fw_i = I.seeded_fw(1, 1, kv_block=4, reserve_permille=0)
    w_bytes = oracle.weight_bytes_per_gpu(SMALL, 1)
    kv_tok = oracle.kv_bytes_per_token(SMALL, 1)
    for n_blocks, want in ((32, oracle.ST_KV), (33, 0)):       # request 1 needs ceil(130/4) = 33 blocks
        sp = I._space(np.array([SMALL]), hw, np.array([w_bytes + n_blocks * 4 * kv_tok]), fw_f, fw_i, [2], [1], [(1, 1)])
        out = oracle.simulate(sp, tr, per_request=True)
        assert out["status"][0] == want
        assert out["bmax"][0] == n_blocks // 33
        if want:
            assert np.all(np.isinf(out["req_ttft"]))


def test_percentile_ranks_on_1024():
    """Nearest rank: 1024 requests -> p50 is sorted[511], p99 is sorted[1013]."""
    n = 1024
    tr = I.make_trace(77, n, 500.0, lengths=True, in_clip=64, out_clip=8)
    hw, mem = I.seeded_hw(77, 1, mem_gb=[1])
    fw_f, fw_i = I.seeded_fw(77, 1)
    sp = I._space(np.array([SMALL]), hw, mem, fw_f, fw_i, [16], [1], [(1, 1)])
    out = oracle.simulate(sp, tr, per_request=True)
    srt = np.sort(out["req_ttft"][0])
    assert out["ttft_p50"][0] == srt[511] and out["ttft_p99"][0] == srt[1013]


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_selection_against_brute_force(seed):
    sp = grid_space(seed=seed, mem_gb=(24, 48, 80), lins=(128, 512, 2048), louts=(1, 64, 256))
    out = oracle.simulate(sp)
    n = len(out["status"])
    assert n <= 2000
    med = float(np.median(out["latency"][out["status"] == 0]))
    cons = {"max_latency": med, "max_cost_per_hr": 100.0}
    passing = (out["status"] == 0) & (out["latency"] <= med) & (out["cost_per_hr"] <= 100.0)
    for key, arr in (("cost_per_token", out["cost_per_token"]), ("latency", out["latency"]),
                     ("cost_per_hr", out["cost_per_hr"]), ("throughput", 0.0 - out["thr_decode"])):
        idx, val, found = oracle.select_topk(out, cons, key, 16)
        want = naive.topk_bruteforce(arr.tolist(), passing.tolist(), 16)
        assert found == len(want) and idx[:found].tolist() == want, key
        src = out["thr_decode"] if key == "throughput" else arr
        assert np.array_equal(val[:found], src[want])
    for x, y in (("latency", "cost_per_hr"), ("latency", "cost_per_token"), ("ttft", "throughput")):
        xs = out[x] if x != "throughput" else 0.0 - out["thr_decode"]
        ys = out[y] if y != "throughput" else 0.0 - out["thr_decode"]
        front, found = oracle.pareto(out, cons, x, y)
        want = naive.pareto_bruteforce(xs.tolist(), ys.tolist(), passing.tolist())
        assert found == len(want) and front.tolist() == want, (x, y)
        assert found >= 2


def test_topk_fewer_than_k_and_ties():
    sp = grid_space(mem_gb=(24,), batch=(1, 2), tp=(1, 2), lins=(64,), louts=(2, 4), n_fw=1)
    out = oracle.simulate(sp)
    ok = int((out["status"] == 0).sum())
    idx, val, found = oracle.select_topk(out, {}, "cost_per_hr", 64)
    assert found == ok < 64
    assert np.all(idx[found:] == np.iinfo(np.uint64).max) and np.all(np.isinf(val[found:]))
    # cost/hr only depends on (hardware, TP): ties everywhere, broken by the lowest index
    v = val[:found]
    assert np.all(np.diff(v) >= 0)
    for a, b in zip(range(found - 1), range(1, found)):
        if v[a] == v[b]:
            assert idx[a] < idx[b]
    idx0, _, found0 = oracle.select_topk(out, {"max_latency": 0.0}, "latency", 4)
    assert found0 == 0 and np.all(idx0 == np.iinfo(np.uint64).max)


def test_strided_and_ranged_evaluation_agree():
    sp = grid_space()
    full = oracle.simulate(sp)
    part = oracle.simulate(sp, first=5, count=40, stride=7)
    for k in oracle.F64_FIELDS + ("status", "bmax"):
        assert np.array_equal(part[k], full[k][5:5 + 40 * 7:7])


@pytest.mark.parametrize("seed", [1, 2, 3, 4])
def test_split_fuse_against_naive_scheduler(seed):
    """The split-and-fuse policy (token budget per iteration, prompts chunked in arrival order,
    decodes fused in) against an explicit scheduler with request objects and per-token loops."""
    n = 24
    arrival = I.poisson_arrivals(seed, n, 2000.0)
    in_len = I.randint(seed, 81, n, 1, 40).astype(np.uint32)
    out_len = I.randint(seed, 82, n, 1, 24).astype(np.uint32)
    tr = {"arrival": arrival, "in_len": in_len, "out_len": out_len}
    hw, _ = I.seeded_hw(seed, 1, mem_gb=[1])
    fw_f, fw_i = I.seeded_fw(seed, 1, kv_block=4, reserve_permille=0)
    fw_i[0, 3] = oracle.POLICY_SPLIT_FUSE
    w_bytes = oracle.weight_bytes_per_gpu(SMALL, 1)
    kv_tok = oracle.kv_bytes_per_token(SMALL, 1)
    total_preempt = chunked = fused = 0
    for n_blocks in (16, 23, 40, 400):
        mem = w_bytes + n_blocks * 4 * kv_tok + 5
        for b, budget in ((1, 7), (3, 16), (8, 5), (8, 64), (4, 1)):
            sp = I._space(np.array([SMALL]), hw, np.array([mem]), fw_f, fw_i, [b], [1], [(1, 1)], fw_chunk=[[0, budget]])
            got = oracle.simulate(sp, tr, per_request=True)
            assert got["status"][0] == 0
            ref = naive.trace_sim_fuse(arrival.tolist(), in_len.tolist(), out_len.tolist(), b, n_blocks, 4, budget,
                                       _iter_time(SMALL, sp, 0, 0, 1))
            assert got["latency"][0] == ref["makespan"]
            ttft = np.array(ref["first"]) - arrival
            assert np.array_equal(got["req_ttft"][0], ttft)
            tpot = [(fi - fr) / (o - 1) if o > 1 else 0.0 for fi, fr, o in zip(ref["finish"], ref["first"], out_len)]
            assert np.array_equal(got["req_tpot"][0], np.array(tpot))
            assert got["n_iters"][0] == ref["n_iters"] and got["n_req_iters"][0] == ref["n_req_iters"]
            assert got["n_preempt"][0] == ref["n_preempt"]
            assert got["thr_decode"][0] == (ref["dec_tok"] / ref["dec_time"] if ref["dec_time"] else 0.0)
            total_preempt += ref["n_preempt"]
            # what the policy is for: prompts longer than the budget take several iterations, and
            # iterations mix decoding requests with prompt chunks
            per_req = {}
            for _, dec, chunks in ref["log"]:
                for i, _seen, _q in chunks:
                    per_req[i] = per_req.get(i, 0) + 1
                fused += bool(dec and chunks)
                assert len(dec) + sum(q for *_, q in chunks) <= max(budget, len(dec))
            chunked += sum(1 for i, c in per_req.items() if c > 1)
            # every prompt token (and every token recomputed after an eviction) is processed once per residency
            if ref["n_preempt"] == 0:
                assert sum(q for _, _, chunks in ref["log"] for *_, q in chunks) == int(in_len.sum())
    assert total_preempt > 0 and chunked > 0 and fused > 0


def test_split_fuse_timeline_worked_by_hand():
    """Two requests, budget 4, block size 4, ample memory.  Request 0: prompt 6, 3 tokens out, at t = 0;
    request 1: prompt 3, 2 tokens out, also at t = 0.
      iteration 1: chunk (0: 4 of 6)                         T=4 E=0 A=4*4=16      C=4
      iteration 2: chunk (0: last 2, attends 6) + (1: 2 of 3) T=4 E=1 A=2*6+2*2=16  C=6+2=8
      iteration 3: decode 0 (ctx 7) + chunk (1: last 1, attends 3)  T=2 E=2 A=7+3=10 C=10
      iteration 4: decode 0 (ctx 8), decode 1 (ctx 4)         T=2 E=2 A=12 C=12   -> both finish"""
    tr = {"arrival": np.array([0.0, 0.0]), "in_len": np.array([6, 3], np.uint32), "out_len": np.array([3, 2], np.uint32)}
    hw, _ = I.seeded_hw(7, 1, mem_gb=[1])
    fw_f, fw_i = I.seeded_fw(7, 1, kv_block=4, reserve_permille=0)
    fw_i[0, 3] = oracle.POLICY_SPLIT_FUSE
    sp = I._space(np.array([SMALL]), hw, np.array([10**9]), fw_f, fw_i, [4], [1], [(1, 1)], fw_chunk=[[0, 4]])
    got = oracle.simulate(sp, tr, per_request=True)
    it = _iter_time(SMALL, sp, 0, 0, 1)
    t1 = it(4, 0, 16, 4)
    t2 = t1 + it(4, 1, 16, 8)
    t3 = t2 + it(2, 2, 10, 10)
    t4 = t3 + it(2, 2, 12, 12)
    assert got["latency"][0] == t4
    assert got["req_ttft"][0].tolist() == [t2, t3]
    assert got["req_tpot"][0].tolist() == [(t4 - t2) / 2, (t4 - t3) / 1]
    assert got["n_iters"][0] == 4 and got["n_req_iters"][0] == 1 + 2 + 2 + 2
    assert got["thr_decode"][0] == 3 / ((t3 - t2) + (t4 - t3))
    # a budget that covers everything waiting is prompt-first scheduling when nothing decodes yet
    both = oracle.simulate(I._space(np.array([SMALL]), hw, np.array([10**9]), fw_f, fw_i, [4], [1], [(1, 1)],
                                    fw_chunk=[[0, 9]]), tr, per_request=True)
    fw_p = fw_i.copy()
    fw_p[0, 3] = 0
    first = oracle.simulate(I._space(np.array([SMALL]), hw, np.array([10**9]), fw_f, fw_p, [4], [1], [(1, 1)]), tr,
                            per_request=True)
    assert both["req_ttft"][0].tolist() == first["req_ttft"][0].tolist()       # one pass over 6 + 3 tokens either way
    # the policy needs its budget and is a trace policy only
    with pytest.raises(ValueError):
        oracle.simulate(I._space(np.array([SMALL]), hw, np.array([10**9]), fw_f, fw_i, [4], [1], [(1, 1)]), tr)
    with pytest.raises(ValueError):
        oracle.simulate(I._space(np.array([SMALL]), hw, np.array([10**9]), fw_f, fw_i, [4], [1], [(1, 1)],
                                 fw_chunk=[[2, 4]]), tr)
