"""Pins the oracle to things other than itself: hand-worked values (tests/golden), closed forms,
special cases and the paper's own equations."""
import math

import numpy as np
import pytest

import oracle
from oracle import naive
from paper_2412_04788_b200 import inputs as I


def toy_space(golden, mem, kv_block, batch, pairs=((4, 3),), tp=(1,), e=None, t_ovh=0.0, flash=1, reserve=0,
              layers=None, dp=None, chunk=None, keep=None):
    model = list(golden["model"])
    if layers:
        model[0] = layers
    fw_f = list(e) if e is not None else [1.0] * 7
    return I._space(np.array([model]), np.array([golden["hw"]]), np.array([mem]),
                    np.array([fw_f + [t_ovh]]), np.array([[flash, kv_block, reserve, 0]]),
                    list(batch), list(tp), [list(p) for p in pairs], dp=None if dp is None else list(dp),
                    fw_chunk=None if chunk is None else [list(chunk)], fw_keep=None if keep is None else [keep])


def test_weight_count_and_kv_bytes(golden):
    assert oracle.weight_params(golden["model"]) == golden["weights"]["params"]
    assert oracle.kv_bytes_per_token(golden["model"], 1) == golden["weights"]["kv_bytes_per_token_t1"]
    ll = golden["llama7b_shape"]
    assert oracle.weight_params(ll["model"]) == ll["params"]
    assert oracle.kv_bytes_per_token(ll["model"], 1) == ll["kv_bytes_per_token_t1"]
    # tensor parallelism splits weights (rounded up) and KV evenly
    assert oracle.weight_bytes_per_gpu(ll["model"], 4) == math.ceil(ll["params"] * 2 / 4)
    assert oracle.kv_bytes_per_token(ll["model"], 4) == ll["kv_bytes_per_token_t1"] // 4


def test_bmax_table(golden):
    """Sec. 3.3.1: B_max = floor(C_available / kv bytes per request)."""
    ll = golden["llama7b_shape"]
    model = np.array([ll["model"]])
    for s_key, row in ll["bmax_reserve0_block1"].items():
        S = int(s_key.split("=")[1])
        for gb, want in row.items():
            sp = I._space(model, np.array([[1e14, 1e12, 1e11, 1e-6, 2.0]]), np.array([int(gb) * 10**9]),
                          np.array([[0.5] * 7 + [0.0]]), np.array([[1, 1, 0, 0]]), [1, want, want + 1], [1],
                          [(S - 128, 128)])
            out = oracle.simulate(sp)
            assert out["bmax"].tolist() == [want] * 3
            assert out["status"].tolist() == [0, 0, oracle.ST_KV]
            assert np.isinf(out["latency"][2]) and out["thr_decode"][2] == 0.0


def test_kv_block_rounding_and_reserve(golden):
    """Fixed-granularity allocation rounds a request up to whole blocks (Sec. 2.4.1); the reserve
    is an integer permille of device memory."""
    ll = golden["llama7b_shape"]
    model = np.array([ll["model"]])
    mem = 24 * 10**9
    usable = mem - (mem // 1000) * 100
    assert oracle.usable_bytes(mem, 100) == usable
    sp = I._space(model, np.array([[1e14, 1e12, 1e11, 1e-6, 2.0]]), np.array([mem]),
                  np.array([[0.5] * 7 + [0.0]]), np.array([[1, 16, 100, 0]]), [1], [1], [(100, 29)])
    out = oracle.simulate(sp)
    s_blk = 144  # ceil(129/16)*16
    assert out["bmax"][0] == (usable - ll["params"] * 2) // (s_blk * ll["kv_bytes_per_token_t1"])


def test_phase_times_worked_by_hand(golden):
    for ph in golden["phases"]:
        model = list(golden["model"])
        if "layers" in ph:
            model[0] = ph["layers"]
        fw_f = ph["e_c"] + ph["e_m"] + [ph["e_comm"], ph["t_ovh"]]
        tm = oracle.TIME_SUM if ph["time_model"] == "sum" else oracle.TIME_MAX
        v, d = oracle.phase_time(model, golden["hw"], fw_f, [ph["flash"], 1, 0, 0], ph["t"],
                                 ph["T"], ph["E"], ph["A"], ph["C"], ph["R"], time_model=tm)
        assert v == ph["T_phase"], ph["name"]
        assert d[15] == ph["T_phase"]
        if "tasks_1_to_8" in ph:
            assert d[:8].tolist() == ph["tasks_1_to_8"], ph["name"]
        if "attn_9_to_11" in ph:
            assert d[8:11].tolist() == ph["attn_9_to_11"], ph["name"]
        for key, slot in (("S_comm", 11), ("head", 12), ("S_fix", 13), ("S_att", 14)):
            if key in ph:
                assert d[slot] == ph[key], (ph["name"], key)


def test_closed_form_toy(golden):
    want = golden["closed_form_b2_Lin4_Lout3"]
    sp = toy_space(golden, 10**6, 1, [2], tp=(1, 2))
    out = oracle.simulate(sp)
    # the toy has a single KV head, so two-way tensor parallelism is flagged (its stage times
    # are still pinned through the phase test above)
    assert out["status"].tolist() == [0, oracle.ST_HEADS]
    assert out["ttft"][0] == want["t1"]["ttft"] and out["latency"][0] == want["t1"]["latency"]
    assert out["tpot"][0] == want["t1"]["tpot"]
    assert out["thr_decode"][0] == want["t1"]["thr_decode_num"] / want["t1"]["thr_decode_den"]
    ff, fi = [1.0] * 7 + [0.0], [1, 1, 0, 0]
    pre2 = oracle.phase_time(golden["model"], golden["hw"], ff, fi, 2, 8, 2, 32, 8, 1)[0]
    dec2 = oracle.phase_time(golden["model"], golden["hw"], ff, fi, 2, 4, 4, 22, 22, 2)[0]
    assert pre2 == want["t2"]["ttft"] and pre2 + dec2 == want["t2"]["latency"]
    assert out["ttft_p50"][0] == out["ttft"][0] == out["ttft_p99"][0]          # TTFT is the prefill time
    assert out["cost_per_hr"][0] == 1.0 and np.isinf(out["cost_per_hr"][1])
    assert out["cost_per_token"][0] == (1.0 / 3600.0) / out["thr_decode"][0]
    assert out["n_iters"].tolist() == [3, 0] and out["n_req_iters"].tolist() == [6, 0]


def test_data_parallel_replicas(golden):
    """Sec. 3.2 Step 1 (the batch a replica sees is the whole batch over the DP degree) and the
    hybrid rule of Sec. 3.5.2 - 3.5.3: dp replicas of the hand-worked batch-2 case."""
    want = golden["closed_form_b2_Lin4_Lout3"]["t1"]
    sp = toy_space(golden, 10**6, 1, [4, 3], tp=(1, 1), dp=(2, 1))
    out = oracle.simulate(sp)
    assert out["status"].tolist() == [0, 0, 0, 0]
    num, den = want["thr_decode_num"], want["thr_decode_den"]        # 2 requests x 2 steps over the decode time
    for c, b in ((0, 4), (2, 3)):                                     # dp = 2: each replica runs at most 2 requests
        assert out["ttft"][c] == want["ttft"] and out["latency"][c] == want["latency"] and out["tpot"][c] == want["tpot"]
        assert out["thr_decode"][c] == (num * b / 2) / den            # every replica's tokens count
        assert out["cost_per_hr"][c] == 2.0                           # price 1.0 x 1 GPU x 2 replicas
        assert out["cost_per_token"][c] == (2.0 / 3600.0) / out["thr_decode"][c]
        assert out["n_iters"][c] == 3 and out["n_req_iters"][c] == 3 * b
    # dp = 1 next to it: four (three) requests on one replica take longer than two
    assert out["latency"][1] > out["latency"][3] > want["latency"] and out["cost_per_hr"][1] == 1.0
    # an explicit axis of ones is the same as none
    ones = oracle.simulate(toy_space(golden, 10**6, 1, [4, 3], tp=(1, 1), dp=(1, 1)))
    none = oracle.simulate(toy_space(golden, 10**6, 1, [4, 3], tp=(1, 1)))
    for k in ones:
        assert np.array_equal(ones[k], none[k]), k
    # memory is per replica: room for exactly two requests of 4 + 3 tokens
    mem = oracle.weight_bytes_per_gpu(golden["model"], 1) + 2 * 7 * oracle.kv_bytes_per_token(golden["model"], 1)
    out = oracle.simulate(toy_space(golden, mem, 1, [4, 5], tp=(1, 1), dp=(1, 2)))
    assert out["bmax"].tolist() == [2, 2, 2, 2]
    assert out["status"].tolist() == [oracle.ST_KV, 0, oracle.ST_KV, oracle.ST_KV]     # ceil(5 / 2) = 3 > 2
    # general degrees against the single-replica run of the share: times bit for bit
    hw, mem = I.seeded_hw(9, 2, mem_gb=[80, 192])
    fw_f, fw_i = I.seeded_fw(9, 2)
    models = I.models_from_shapes(I.SHAPES_8[:3])
    pairs = [(128, 64), (500, 1), (33, 17)]
    batch, degrees = [1, 7, 24, 100], [1, 2, 3, 5, 8]
    shares = sorted({-(-b // d) for b in batch for d in degrees})
    for t in (1, 2):
        hyb = oracle.simulate(I._space(models, hw, mem, fw_f, fw_i, batch, [t] * len(degrees), pairs, dp=degrees))
        one = oracle.simulate(I._space(models, hw, mem, fw_f, fw_i, shares, [t], pairs))
        H = {k: v.reshape(3, 2, 2, len(batch), len(degrees), 3) for k, v in hyb.items()}
        O = {k: v.reshape(3, 2, 2, len(shares), 1, 3) for k, v in one.items()}
        for bi, b in enumerate(batch):
            for di, d in enumerate(degrees):
                si = shares.index(-(-b // d))
                for k in ("status", "bmax", "latency", "ttft", "tpot", "n_iters"):
                    assert np.array_equal(H[k][:, :, :, bi, di], O[k][:, :, :, si, 0]), (k, b, d)
                ok = H["status"][:, :, :, bi, di] == 0
                n = np.array([p[1] - 1 for p in pairs])
                t_dec = (O["latency"] - O["ttft"])[:, :, :, si, 0]
                thr = H["thr_decode"][:, :, :, bi, di]
                dec = ok & (n > 0)                                    # a single output token has no decode stage
                with np.errstate(invalid="ignore"):
                    assert np.allclose(thr[dec], ((b * n) / t_dec)[dec], rtol=1e-12, atol=0)
                assert np.all(thr[ok & (n == 0)] == 0.0)
                assert np.array_equal(H["cost_per_hr"][:, :, :, bi, di][ok], (O["cost_per_hr"][:, :, :, si, 0] * d)[ok]) \
                    or np.allclose(H["cost_per_hr"][:, :, :, bi, di][ok], (O["cost_per_hr"][:, :, :, si, 0] * d)[ok], rtol=1e-15)
                assert np.array_equal(H["n_req_iters"][:, :, :, bi, di][ok], np.broadcast_to(b * (1 + n), ok.shape)[ok])
    # no replica split of a trace, no zero degree
    tr = {"arrival": np.array([0.0, 1.0]), "in_len": np.zeros(2, np.uint32), "out_len": np.zeros(2, np.uint32)}
    with pytest.raises(ValueError, match="data parallelism"):
        oracle.simulate(toy_space(golden, 10**6, 1, [2], dp=(2,)), tr)
    with pytest.raises(ValueError):
        oracle.simulate(toy_space(golden, 10**6, 1, [2], dp=(0,)))


def test_prompt_sub_batches_and_segments(golden):
    """Sec. 3.3.1 (sub-batches of split_size requests plus a remainder) and Sec. 3.3.2 (prompts cut
    into ceil(Lin / segment) segments): hand-worked batch-2 case, explicit token walks."""
    want = golden["closed_form_b2_Lin4_Lout3"]["t1"]
    hw, ff, fi = golden["hw"], [1.0] * 7 + [0.0], [1, 1, 0, 0]
    one = oracle.simulate(toy_space(golden, 10**6, 1, [1, 2, 4, 5]))
    # sub-batches of two: 2 = one pass, 4 = two equal passes, 5 = two passes and a single request
    out = oracle.simulate(toy_space(golden, 10**6, 1, [1, 2, 4, 5], chunk=(2, 0)))
    assert out["ttft"][1] == want["ttft"] and out["latency"][1] == want["latency"]
    assert out["ttft"][2] == 2.0 * want["ttft"] and out["ttft"][3] == 2.0 * want["ttft"] + one["ttft"][0]
    assert out["ttft"][0] == one["ttft"][0]
    assert out["n_iters"].tolist() == [1 + 2, 1 + 2, 2 + 2, 3 + 2]
    assert out["n_req_iters"].tolist() == [3, 6, 12, 15]
    # the decode stage is that of the whole batch
    assert np.array_equal(out["latency"] - out["ttft"] > 0, [True] * 4)
    for c in range(4):
        assert out["tpot"][c] == one["tpot"][c] and out["thr_decode"][c] == one["thr_decode"][c]
    # segments of two tokens of the 4-token prompt, two requests: (T, E, A, C) by hand
    out = oracle.simulate(toy_space(golden, 10**6, 1, [2], chunk=(0, 2)))
    p1, d1 = oracle.phase_time(golden["model"], hw, ff, fi, 1, 4, 0, 8, 4, 1)     # 2 x 2 tokens attend 2; no token out
    p2, d2 = oracle.phase_time(golden["model"], hw, ff, fi, 1, 4, 2, 16, 8, 1)    # 2 x 2 tokens attend 4; 2 tokens out
    assert out["ttft"][0] == (0.0 + p1) + p2
    assert d1[12] == 0.0 and d2[12] > 0.0                                         # no LM head without an emitted token
    assert p1 == golden["model"][0] * ((d1[13] + d1[14]) + d1[11])                # layers x per-layer time, nothing else
    assert out["n_iters"][0] == 2 + 2 and out["n_req_iters"][0] == 2 * (2 + 2)
    assert out["ttft"][0] > want["ttft"]                                          # the weights are read twice
    # sizes that split nothing change nothing, bit for bit
    base = oracle.simulate(toy_space(golden, 10**6, 1, [1, 2, 3], pairs=[(4, 3), (7, 1)]))
    for chunk in ((0, 0), (3, 7), (100, 100), (0, 8)):
        same = oracle.simulate(toy_space(golden, 10**6, 1, [1, 2, 3], pairs=[(4, 3), (7, 1)], chunk=chunk))
        for k in base:
            assert np.array_equal(base[k], same[k]), (chunk, k)
    # general sizes against explicit walks over sub-batches, segments, sequences and tokens
    hw2 = [3.0e3, 5.0e2, 1.0e2, 1e-3, 2.0]
    ff2, fi2 = [0.5, 0.25, 0.75, 0.5, 0.5, 0.25, 0.5, 1e-2], [0, 1, 0, 0]
    for b, lin, lout, split, seg in [(5, 7, 3, 2, 3), (7, 16, 2, 3, 16), (4, 9, 1, 4, 2), (6, 5, 4, 1, 1), (3, 33, 2, 5, 8)]:
        for tm in (oracle.TIME_MAX, oracle.TIME_SUM):
            sp = I._space(np.array([golden["model"]]), np.array([hw2]), np.array([10**9]), np.array([ff2]),
                          np.array([fi2]), [b], [1], [(lin, lout)], fw_chunk=[[split, seg]])
            out = oracle.simulate(sp, time_model=tm)
            subs = naive.sub_batches(b, split)
            per_size = {}
            for sb in set(subs):
                t = 0.0
                for T, E, A, Cc in naive.segment_passes(sb, lin, seg):
                    t = t + oracle.phase_time(golden["model"], hw2, ff2, fi2, 1, T, E, A, Cc, 1, time_model=tm)[0]
                per_size[sb] = t
            t_pre = subs.count(split) * per_size[split] if split in per_size else 0.0
            if b % split:
                t_pre = t_pre + per_size[b % split]
            assert out["ttft"][0] == t_pre, (b, lin, split, seg)
            n_seg = len(naive.segment_passes(1, lin, seg))
            assert out["n_iters"][0] == len(subs) * n_seg + (lout - 1)
            assert out["n_req_iters"][0] == b * (n_seg + lout - 1)
            # all prompt tokens are processed exactly once
            assert sum(T for sb in subs for T, *_ in naive.segment_passes(sb, lin, seg)) == b * lin
    # a replica's share is what gets split (Sec. 3.2 Step 1)
    out = oracle.simulate(toy_space(golden, 10**6, 1, [8, 7], tp=(1,), dp=(2,), chunk=(2, 0)))
    assert out["ttft"].tolist() == [2.0 * want["ttft"]] * 2 and out["n_iters"].tolist() == [4, 4]
    # traces keep the prompt-first policy: splitting is refused there
    tr = {"arrival": np.array([0.0, 1.0]), "in_len": np.zeros(2, np.uint32), "out_len": np.zeros(2, np.uint32)}
    with pytest.raises(ValueError, match="splitting"):
        oracle.simulate(toy_space(golden, 10**6, 1, [2], chunk=(0, 2)), tr)


def test_closed_form_aggregates_match_token_loops(golden):
    """The aggregated stage sums against an explicit walk over sequences, steps and tokens."""
    hw, ff, fi = golden["hw"], [1.0] * 7 + [0.0], [1, 1, 0, 0]
    for b, lin, lout in [(1, 1, 1), (2, 4, 3), (3, 7, 5), (5, 16, 9), (1, 33, 2)]:
        sp = toy_space(golden, 10**9, 1, [b], pairs=[(lin, lout)])
        out = oracle.simulate(sp)
        T, E, A, Cc = naive.prefill_aggregates(b, lin)
        t_pre, _ = oracle.phase_time(golden["model"], hw, ff, fi, 1, T, E, A, Cc, 1)
        assert out["ttft"][0] == t_pre
        T, E, A, Cc, R = naive.decode_aggregates(b, lin, lout)
        t_dec = oracle.phase_time(golden["model"], hw, ff, fi, 1, T, E, A, Cc, R)[0] if R else 0.0
        assert out["latency"][0] == t_pre + t_dec
        if R:
            assert out["tpot"][0] == t_dec / R and out["thr_decode"][0] == (b * R) / t_dec
        else:
            assert out["tpot"][0] == 0.0 and out["thr_decode"][0] == 0.0 and np.isinf(out["cost_per_token"][0])


def _cost_space(golden, batch, tp, dp=None, pairs=((4, 3),)):
    """The toy decoder with 8 heads (every degree up to 8 divides them) at the price of the cost pins."""
    c = golden["costs"]
    model = list(golden["model"])
    model[2], model[3] = c["heads"], c["heads"]
    hw = list(golden["hw"])
    hw[4] = c["price_per_gpu_hr"]
    return model, hw, I._space(np.array([model]), np.array([hw]), np.array([10**6]), np.array([[1.0] * 7 + [0.0]]),
                               np.array([[1, 1, 0, 0]]), list(batch), list(tp), [list(p) for p in pairs],
                               dp=None if dp is None else list(dp))


def test_closed_form_cost_is_price_times_all_gpus(golden):
    """Sec. 4.1 (selection under a budget) with Sec. 3.5.2: a deployment pays for t GPUs per replica
    and dp replicas, so cost per hour = price x t x dp; cost per token = (cost per hour / 3600) /
    decode throughput.  Values worked by hand in tests/golden (price 3 $/h per GPU)."""
    rows = golden["costs"]["closed_form"]
    model, hw, sp = _cost_space(golden, [6], [r["t"] for r in rows], dp=[r["dp"] for r in rows])
    out = oracle.simulate(sp)
    assert out["status"].tolist() == [0] * len(rows)
    assert out["cost_per_hr"].tolist() == [r["cost_per_hr"] for r in rows]
    ff, fi = [1.0] * 7 + [0.0], [1, 1, 0, 0]
    for i, r in enumerate(rows):
        b = -(-6 // r["dp"])                                       # the replica's share of the batch of 6
        ctx = b * (2 * 4 + 3)                                      # two decode steps attending 5 and 6 tokens
        t_dec = oracle.phase_time(model, hw, ff, fi, r["t"], 2 * b, 2 * b, ctx, ctx, 2)[0]
        assert out["thr_decode"][i] == (6 * 2) / t_dec             # all replicas' tokens over one replica's time
        assert out["cost_per_token"][i] == (r["cost_per_hr"] / 3600.0) / out["thr_decode"][i]
    # twice the GPUs at the same throughput would cost twice as much per token: the factor is not folded away
    assert out["cost_per_hr"][2] == 4.0 * out["cost_per_hr"][0]


def test_trace_cost_is_price_times_tp_degree(golden):
    """The trace simulation models one replica of t GPUs: cost per hour = price x t (Sec. 4.1), cost
    per token = (cost per hour / 3600) / decode throughput, the throughput being decode tokens over
    the time of the decode iterations (Sec. 5.1), which the hand-worked timelines pin."""
    rows = golden["costs"]["trace"]
    model, hw, sp = _cost_space(golden, [2], [r["t"] for r in rows])
    tr = {"arrival": np.array([0.0, 1.0, 1.5]), "in_len": np.zeros(3, np.uint32), "out_len": np.zeros(3, np.uint32)}
    out = oracle.simulate(sp, tr)
    assert out["status"].tolist() == [0] * len(rows)
    assert out["cost_per_hr"].tolist() == [r["cost_per_hr"] for r in rows]
    for i, r in enumerate(rows):
        assert out["thr_decode"][i] > 0.0
        assert out["cost_per_token"][i] == (r["cost_per_hr"] / 3600.0) / out["thr_decode"][i]
    # the same trace on the unsharded toy at price 1: the first timeline's decode tokens and time
    tl = golden["timelines"][0]
    sp1 = toy_space(golden, tl["mem"], tl["kv_block"], [tl["max_batch"]])
    n = len(tl["arrival"])
    tr1 = {"arrival": np.array(tl["arrival"]), "in_len": np.zeros(n, np.uint32), "out_len": np.zeros(n, np.uint32)}
    out1 = oracle.simulate(sp1, tr1)
    assert out1["cost_per_hr"][0] == 1.0
    assert out1["cost_per_token"][0] == (1.0 / 3600.0) / (tl["dec_tok"] / tl["dec_time"])


def test_cache_eviction_keeps_a_share_of_the_kv(golden):
    """H2O (Sec. 3.2 Step 1, Sec. 3.3): a request's cache holds ceil(p c / 1000) of its c tokens - in the
    memory check (per request, then whole blocks) and in the decode stage's attention work and KV
    read (on the stage total).  The prompt pass is not touched.  Values worked by hand."""
    g = golden["kv_reduction_and_clamp"]
    weights = 2 * golden["weights"]["params"]
    for row in g["bmax"]["rows"]:
        out = oracle.simulate(toy_space(golden, weights + g["bmax"]["avail_bytes"], row["block"], [1, row["bmax"], row["bmax"] + 1],
                                        keep=row["p"]))
        assert out["bmax"].tolist() == [row["bmax"]] * 3, row
        assert out["status"].tolist() == [0, 0, oracle.ST_KV], row
    base = golden["closed_form_b2_Lin4_Lout3"]["t1"]
    for row in g["decode"]["rows"]:
        out = oracle.simulate(toy_space(golden, 10**6, 1, [2], keep=row["p"]))
        assert out["ttft"][0] == base["ttft"]                                  # the prompt is attended in full
        assert out["latency"][0] == row["latency"] and out["latency"][0] - out["ttft"][0] == row["T_dec"]
        assert out["tpot"][0] == row["tpot"] and out["thr_decode"][0] == 4 / row["T_dec"]
        kept = next(k["kept"] for k in g["kept"] if k["p"] == row["p"] and k["c"] == 22)
        _, d = oracle.phase_time(golden["model"], golden["hw"], [1.0] * 7 + [0.0], [1, 1, 0, 0], 1, 4, 4, kept, kept, 2)
        assert d[14] == row["S_att"]
    # 0 and 1000 both mean that nothing is evicted; more than everything is refused
    full = oracle.simulate(toy_space(golden, 10**6, 1, [1, 2, 3]))
    for p in (0, 1000):
        same = oracle.simulate(toy_space(golden, 10**6, 1, [1, 2, 3], keep=p))
        for k in full:
            assert np.array_equal(full[k], same[k]), (p, k)
    with pytest.raises(ValueError):
        oracle.simulate(toy_space(golden, 10**6, 1, [2], keep=1001))
    # a smaller share never costs time or room (rounding is monotone)
    hw, mem = I.seeded_hw(31, 3, mem_gb=[24, 48, 80])
    fw_f, fw_i = I.seeded_fw(31, 1)
    sp = lambda p: I._space(I.models_from_shapes(I.SHAPES_8[:4]), hw, mem, fw_f, fw_i, [1, 8, 64], [1, 2], I.pairs_grid([64, 1000], [1, 33, 512]),
                            fw_keep=[p])
    prev = oracle.simulate(sp(1000))
    for p in (900, 501, 500, 37, 1):
        cur = oracle.simulate(sp(p))
        both = (prev["status"] == 0) & (cur["status"] == 0)
        assert np.all(cur["bmax"] >= prev["bmax"]) and np.all(cur["status"][prev["status"] == 0] == 0)
        assert np.all(cur["latency"][both] <= prev["latency"][both]) and np.array_equal(cur["ttft"][both], prev["ttft"][both])
        prev = cur
    # the trace simulation does not model it
    tr = {"arrival": np.array([0.0, 1.0]), "in_len": np.zeros(2, np.uint32), "out_len": np.zeros(2, np.uint32)}
    with pytest.raises(ValueError, match="cache eviction"):
        oracle.simulate(toy_space(golden, 10**6, 1, [2], keep=500), tr)


def test_sequence_cut_to_what_fits(golden):
    """Sec. 3.3.2: S_max = floor(C_available / (KV bytes per token x B)); a longer sequence is cut to it
    (whole blocks; the prompt is cut, the output tokens stay), and the length used is reported."""
    g = golden["kv_reduction_and_clamp"]
    weights = 2 * golden["weights"]["params"]
    for row in g["clamp"]:
        sp = toy_space(golden, weights + row["avail"], row["block"], [2], keep=row["p"])
        out = oracle.simulate(sp, clamp_seq=True)
        assert out["status"][0] == row["status"] and out["seq_used"][0] == row["seq_used"] and out["bmax"][0] == row["bmax"], row
        if row["status"] == 0:
            # the same numbers as the shorter prompt evaluated where memory is ample
            ref = oracle.simulate(toy_space(golden, 10**6, row["block"], [2], pairs=[(row["lin_used"], 3)], keep=row["p"]))
            for k in oracle.F64_FIELDS + ("n_iters", "n_req_iters"):
                assert out[k][0] == ref[k][0], (row, k)
        else:
            assert np.isinf(out["latency"][0])
        # without the option the long sequence is judged as it is
        plain = oracle.simulate(sp)
        assert plain["seq_used"][0] == (7 if plain["status"][0] == 0 else 0)
        assert (plain["status"][0] == 0) == (row["seq_used"] == 7)
    # a sweep: cut configs are exactly those that did not fit by their KV need alone and have room for
    # one prompt token; nothing else changes; a cut config fills its memory to within one block per request
    hw, mem = I.seeded_hw(32, 4, mem_gb=[16, 24, 48, 80])
    fw_f, fw_i = I.seeded_fw(32, 2)
    sp = I._space(I.models_from_shapes(I.SHAPES_8[:5]), hw, mem, fw_f, fw_i, [1, 16, 256], [1, 4], I.pairs_grid([128, 4096, 8192], [64, 2048]),
                  fw_keep=[1000, 400])
    a, c = oracle.simulate(sp), oracle.simulate(sp, clamp_seq=True)
    cut = (c["status"] == 0) & (a["status"] != 0)
    assert cut.sum() > 20 and np.all(a["status"][cut] == oracle.ST_KV)
    same = ~cut
    for k in a:
        assert np.array_equal(a[k][same], c[k][same]), k
    n_l = len(sp["pairs"])
    S = (sp["pairs"][:, 0] + sp["pairs"][:, 1])[np.arange(len(cut)) % n_l]
    lout = sp["pairs"][:, 1][np.arange(len(cut)) % n_l]
    assert np.all(c["seq_used"][cut] < S[cut]) and np.all(c["seq_used"][cut] > lout[cut])
    tr = {"arrival": np.array([0.0, 1.0]), "in_len": np.zeros(2, np.uint32), "out_len": np.zeros(2, np.uint32)}
    with pytest.raises(ValueError, match="clamping"):
        oracle.simulate(toy_space(golden, 10**6, 1, [2]), tr, clamp_seq=True)


def test_binary32_variant(golden):
    """The reduced-precision variant of the closed form (every operation of the model in binary32): the
    hand-worked toy values are dyadic with few bits, so they must come out bit for bit here too; on a
    sweep it stays within 1e-5 of the binary64 result (about sixty rounded operations of 6e-8 each on
    sums of positive terms); integer outputs do not depend on the precision."""
    want = golden["closed_form_b2_Lin4_Lout3"]["t1"]
    out = oracle.simulate(toy_space(golden, 10**6, 1, [2], tp=(1, 2)), precision="f32")
    assert out["ttft"][0] == want["ttft"] and out["latency"][0] == want["latency"] and out["tpot"][0] == want["tpot"]
    assert out["thr_decode"][0] == float(np.float32(want["thr_decode_num"]) / np.float32(want["thr_decode_den"]))
    for row in golden["kv_reduction_and_clamp"]["decode"]["rows"]:
        o = oracle.simulate(toy_space(golden, 10**6, 1, [2], keep=row["p"]), precision="f32")
        assert o["latency"][0] == row["latency"] and o["tpot"][0] == row["tpot"]
    w = I.workload(2, scale=0.25)
    a = oracle.simulate(w["space"])
    b = oracle.simulate(w["space"], precision="f32")
    for k in ("status", "bmax", "n_iters", "n_req_iters", "seq_used"):
        assert np.array_equal(a[k], b[k]), k
    ok = a["status"] == 0
    worst = 0.0
    for k in oracle.F64_FIELDS:
        assert np.array_equal(np.isinf(a[k]), np.isinf(b[k])), k
        fin = ok & np.isfinite(a[k]) & (a[k] != 0)
        assert np.array_equal(b[k][fin], b[k][fin].astype(np.float32).astype(np.float64)), k     # binary32 values
        rel = np.abs(b[k][fin] - a[k][fin]) / np.abs(a[k][fin])
        worst = max(worst, float(rel.max()))
    assert 1e-9 < worst <= 1e-5, worst          # really rounded, and within the bar
    with pytest.raises(AssertionError):
        tr = {"arrival": np.array([0.0]), "in_len": np.zeros(1, np.uint32), "out_len": np.zeros(1, np.uint32)}
        oracle.simulate(toy_space(golden, 10**6, 1, [2]), tr, precision="f32")


def test_paper_log2_rule(golden):
    """Sec. 3.2: multi-GPU throughput = N T_single / (1 + log2 P_TP)."""
    model = list(golden["model"])
    model[2], model[3] = 8, 8          # 8 heads so that every degree divides
    sp = I._space(np.array([model]), np.array([golden["hw"]]), np.array([10**6]), np.array([[1.0] * 7 + [0.0]]),
                  np.array([[1, 1, 0, 0]]), [2], [1, 2, 4, 8], [(4, 3)])
    out = oracle.simulate(sp, tp_model=oracle.TP_PAPER_LOG2)
    assert out["status"].tolist() == [0] * 4
    thr, lat = out["thr_decode"], out["latency"]
    for i, t in enumerate((2, 4, 8), start=1):
        assert lat[i] == lat[0] * golden["paper_log2_rule"]["time_factor"][str(t)]
        assert thr[i] == pytest.approx(thr[0] * golden["paper_log2_rule"]["throughput_ratio_vs_t1"][str(t)], rel=1e-15)


def test_iteration_times(golden):
    hw, ff, fi = golden["hw"], [1.0] * 7 + [0.0], [1, 1, 0, 0]
    it = golden["iteration_times_t1"]
    pt = lambda T, E, A, Cc: oracle.phase_time(golden["model"], hw, ff, fi, 1, T, E, A, Cc, 1)[0]
    assert pt(4, 1, 16, 4) == it["prefill T=4 E=1 A=16"]
    assert pt(5, 1, 25, 5) == it["prefill T=5 E=1 A=25 (recompute of prompt 4 + 1 generated)"]
    assert pt(8, 2, 32, 8) == it["prefill T=8 E=2 A=32"]
    assert pt(1, 1, 5, 5) == it["decode n=1 ctx=5"]
    assert pt(1, 1, 6, 6) == it["decode n=1 ctx=6"]
    assert pt(2, 2, 10, 10) == it["decode n=2 ctx=10"]
    assert pt(2, 2, 12, 12) == it["decode n=2 ctx=12"]


def test_timelines_worked_by_hand(golden):
    for tl in golden["timelines"]:
        sp = toy_space(golden, tl["mem"], tl["kv_block"], [tl["max_batch"]])
        n = len(tl["arrival"])
        tr = {"arrival": np.array(tl["arrival"]), "in_len": np.zeros(n, np.uint32), "out_len": np.zeros(n, np.uint32)}
        out = oracle.simulate(sp, tr, per_request=True)
        assert out["status"][0] == 0, tl["name"]
        for k in ("latency", "ttft", "ttft_p50", "ttft_p99", "tpot"):
            assert out[k][0] == tl[k], (tl["name"], k)
        assert out["req_ttft"][0].tolist() == tl["req_ttft"]
        assert out["req_tpot"][0].tolist() == tl["req_tpot"]
        assert out["thr_decode"][0] == tl["dec_tok"] / tl["dec_time"]
        assert out["n_iters"][0] == tl["n_iters"] and out["n_req_iters"][0] == tl["n_req_iters"]
        assert out["n_preempt"][0] == tl["n_preempt"]
        if "bmax" in tl:
            assert out["bmax"][0] == tl["bmax"]


def test_trace_reduces_to_closed_form_prefill(golden):
    """All requests at t=0, identical, at most max-batch of them, ample memory: one prefill pass
    whose time is the closed form's TTFT bit for bit, then Lout-1 decode iterations."""
    ll = np.array([golden["llama7b_shape"]["model"]])
    hw, mem = I.seeded_hw(11, 1, mem_gb=[192])
    fw_f, fw_i = I.seeded_fw(11, 1)
    for b, lin, lout in [(4, 128, 16), (8, 512, 4), (1, 2048, 2)]:
        sp = I._space(ll, hw, mem, fw_f, fw_i, [b], [1, 2], [(lin, lout)])
        cf = oracle.simulate(sp)
        tr = {"arrival": np.zeros(b), "in_len": np.zeros(b, np.uint32), "out_len": np.zeros(b, np.uint32)}
        ts = oracle.simulate(sp, tr, per_request=True)
        assert ts["status"].tolist() == [0, 0]
        for c in range(2):
            assert np.all(ts["req_ttft"][c] == cf["ttft"][c])
            assert ts["n_iters"][c] == lout and ts["n_req_iters"][c] == b * lout
            # a sum of per-step maxima is never below the maximum of the sums
            assert ts["latency"][c] >= cf["latency"][c] * (1 - 1e-12)
            assert ts["latency"][c] == pytest.approx(cf["latency"][c], rel=0.05)


def test_status_bits(golden):
    ll = np.array([golden["llama7b_shape"]["model"]])
    hw, mem = I.seeded_hw(5, 2, mem_gb=[12, 24])
    fw_f, fw_i = I.seeded_fw(5, 1)
    sp = I._space(ll, hw, mem, fw_f, fw_i, [1, 4096], [1, 64], [(128, 128)])
    out = oracle.simulate(sp)
    st = out["status"].reshape(2, 2, 2)
    # 12 GB: fp16 weights (13.5 GB) do not fit on one GPU -> bit0 (+ bit1: no room for any batch)
    assert st[0, 0, 0] == oracle.ST_WEIGHTS | oracle.ST_KV
    # 64-way TP does not divide 32 heads -> bit2
    assert st[1, 0, 1] & oracle.ST_HEADS
    assert st[1, 0, 0] == 0 and st[1, 1, 0] == oracle.ST_KV


def test_invalid_inputs_rejected(golden):
    sp = toy_space(golden, 10**6, 1, [2], tp=(3,))
    with pytest.raises(ValueError):
        oracle.simulate(sp)
    sp = toy_space(golden, 10**6, 1, [2])
    tr = {"arrival": np.array([1.0, 0.5]), "in_len": np.zeros(2, np.uint32), "out_len": np.zeros(2, np.uint32)}
    with pytest.raises(ValueError):
        oracle.simulate(sp, tr)


def test_overflow_is_reported(golden):
    big = [200, 2**20, 32, 32, 2**22, 2**20, 1, 2, 2, 2]
    sp = I._space(np.array([big]), np.array([golden["hw"]]), np.array([2**62]), np.array([[1.0] * 7 + [0.0]]),
                  np.array([[1, 1, 0, 0]]), [2**10], [1], [(2**20, 2)])
    with pytest.raises(ValueError, match="overflow"):
        oracle.simulate(sp)


def test_iteration_cap_sets_status(golden):
    sp = toy_space(golden, 10**6, 1, [1])
    tr = {"arrival": np.array([0.0, 1.0]), "in_len": np.zeros(2, np.uint32), "out_len": np.zeros(2, np.uint32)}
    out = oracle.simulate(sp, tr, max_iters=5)     # the schedule needs 6 iterations
    assert out["status"][0] == oracle.ST_ITER and np.isinf(out["latency"][0])
    out = oracle.simulate(sp, tr, max_iters=6)
    assert out["status"][0] == 0


def test_percentile_ranks(golden):
    """p50 / p99 are order statistics at the nearest rank; request counts where a floor-based rank
    would pick a different element."""
    hw, mem = I.seeded_hw(21, 1, mem_gb=[1])
    fw_f, fw_i = I.seeded_fw(21, 1)
    small = [4, 256, 8, 4, 512, 1000, 1, 2, 2, 2]
    for case in golden["percentile_ranks"]["cases"]:
        n = case["n"]
        tr = I.make_trace(300 + n, n, 2.0e5, lengths=True, in_clip=48, out_clip=6)     # arrivals faster than service: queueing
        sp = I._space(np.array([small]), hw, mem, fw_f, fw_i, [2], [1], [(1, 1)])
        out = oracle.simulate(sp, tr, per_request=True)
        srt = np.sort(out["req_ttft"][0])
        assert len(np.unique(srt)) > n // 2          # distinct enough for the rank to matter
        assert out["ttft_p50"][0] == srt[case["p50"]], n
        assert out["ttft_p99"][0] == srt[case["p99"]], n
