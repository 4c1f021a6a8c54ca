"""Multi-GPU plumbing on CPU: two gloo ranks shard the hardware axis, select locally (here with the
oracle standing in for the kernels), all-gather their candidates and merge; the result must be the
single-process answer."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2412_04788_b200 import inputs as I, sharding


def test_hw_slices_cover_the_axis():
    for n, world in ((16, 1), (16, 2), (17, 4), (5, 5), (64, 8)):
        cuts = [sharding.hw_slice(n, r, world) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
        assert max(hi - lo for lo, hi in cuts) - min(hi - lo for lo, hi in cuts) <= 1


def test_local_to_global_indices():
    g = I.workload(2, scale=0.25)["space"]          # 4 hardware profiles
    for world in (2, 4):
        seen = []
        for r in range(world):
            loc, off = sharding.shard_space(g, r, world)
            n = I.space_size(loc)
            idx = np.arange(n, dtype=np.int64)
            gi = sharding.local_to_global(idx, loc, g, off)
            for j in (0, 1, n // 3, n - 1):
                m, h, f, b, t, l = I.decode_index(loc, j)
                assert I.decode_index(g, int(gi[j])) == (m, h + off, f, b, t, l)
            seen.append(gi)
        allg = np.sort(np.concatenate(seen))
        assert np.array_equal(allg, np.arange(I.space_size(g)))
    assert sharding.local_to_global(np.array([-1, 0]), loc, g, off)[0] == -1


def _oracle_selectors(key, x, y):
    """The oracle standing in for the library's selection calls over a gathered list (CPU tensors)."""
    name = {"throughput": "thr_decode"}

    def full(status, **arrays):
        n = status.numel()
        out = {k: np.zeros(n) for k in oracle.F64_FIELDS}
        out["status"] = status.numpy().copy()
        for k, v in arrays.items():
            out[name.get(k, k)] = v.numpy().copy()
        return out

    def select(status, values, k):
        idx, val, found = oracle.select_topk(full(status, **{key: values}), {}, key, k)
        return torch.from_numpy(idx.view(np.int64).copy()), torch.from_numpy(val.copy()), found

    def front(status, xs, ys, cap):
        idx, size = oracle.pareto(full(status, **{x: xs, y: ys}), {}, x, y, cap=cap)
        return torch.from_numpy(idx.view(np.int64).copy()), size

    return select, front


def _local_results(loc, key, k, x, y, cap):
    """One shard's candidates and front from the oracle: (idx, val, front idx, x, y, front size)."""
    out = oracle.simulate(loc)
    idx, val, _ = oracle.select_topk(out, {}, key, k)
    fidx, fsize = oracle.pareto(out, {}, x, y, cap=cap)
    pad = np.zeros(cap, dtype=np.int64)
    pad[:len(fidx)] = fidx.view(np.int64)
    sel = pad[:len(fidx)]
    name = {"throughput": "thr_decode"}
    fx, fy = np.zeros(cap), np.zeros(cap)
    fx[:len(fidx)] = out[name.get(x, x)][sel]
    fy[:len(fidx)] = out[name.get(y, y)][sel]
    return (torch.from_numpy(idx.view(np.int64).copy()), torch.from_numpy(val.copy()), torch.from_numpy(pad),
            torch.from_numpy(fx), torch.from_numpy(fy), fsize)


KEY, K, FX, FY, CAP = "cost_per_hr", 16, "ttft", "cost_per_token", 256


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        g = I.workload(2, scale=0.25)["space"]
        loc, off = sharding.shard_space(g, rank, world)
        idx, val, fidx, fx, fy, fsize = _local_results(loc, KEY, K, FX, FY, CAP)
        select, front = _oracle_selectors(KEY, FX, FY)
        top, _, found = sharding.merge_topk(sharding.local_to_global(idx, loc, g, off), val, K, select)
        fr, size = sharding.merge_front(sharding.local_to_global(fidx, loc, g, off), fx, fy, fsize, CAP, front)
        q.put((rank, top.tolist(), found, fr.tolist(), size))
    finally:
        dist.destroy_process_group()


def test_two_rank_selection_matches_single_process():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = {r[0]: r[1:] for r in (q.get(timeout=120) for _ in procs)}
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    g = I.workload(2, scale=0.25)["space"]
    whole = oracle.simulate(g)
    want_idx, _, found = oracle.select_topk(whole, {}, KEY, K)
    want_front, want_size = oracle.pareto(whole, {}, FX, FY, cap=CAP)
    assert found == K and want_size > 3
    # cost/hr has many ties: only the lowest-index rule makes the answer unique
    for r in (0, 1):
        top, got_found, fr, size = res[r]
        assert top == want_idx.view(np.int64).tolist() and got_found == found
        assert size == want_size and fr == want_front.view(np.int64).tolist()


def test_merge_in_one_process_with_three_shards():
    """The same merges without a process group (the shards' lists concatenated in rank order), on an
    uneven split and with a throughput key (descending order)."""
    g = I.workload(2, scale=0.25)["space"]
    g = dict(g)
    g["batch"] = g["batch"][:4]
    key, k, x, y, cap = "throughput", 7, "ttft", "throughput", 64
    parts = []
    for r in range(3):
        loc, off = sharding.shard_space(g, r, 3)
        idx, val, fidx, fx, fy, fsize = _local_results(loc, key, k, x, y, cap)
        used = torch.arange(cap) < fsize
        parts.append((sharding.local_to_global(idx, loc, g, off), val,
                      torch.where(used, sharding.local_to_global(fidx, loc, g, off), torch.full_like(fidx, -1)), fx, fy))
    select, front = _oracle_selectors(key, x, y)
    pick = lambda i: (lambda t: sharding.concat_gather(p[i] for p in parts))
    top, _, found = sharding.merge_topk(None, None, k, select, gather=_SeqGather([pick(0), pick(1)]))
    fr, size = sharding.merge_front(torch.zeros(0, dtype=torch.int64), None, None, 0, cap, front,
                                    gather=_SeqGather([pick(2), pick(3), pick(4)]))
    whole = oracle.simulate(g)
    want_idx, _, want_found = oracle.select_topk(whole, {}, key, k)
    want_front, want_size = oracle.pareto(whole, {}, x, y, cap=cap)
    assert found == want_found and top.tolist() == want_idx.view(np.int64).tolist()
    assert size == want_size and fr.tolist() == want_front.view(np.int64).tolist()


class _SeqGather:
    """gather stand-in that returns prepared concatenations in call order."""

    def __init__(self, fns):
        self.fns = list(fns)

    def __call__(self, t):
        return self.fns.pop(0)(t)
