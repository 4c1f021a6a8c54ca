"""Multi-GPU plumbing: configs are independent, so the space is cut along the hardware axis, each
rank evaluates its slice with the single-GPU kernels, and the only exchange is an all-gather of
each rank's k best candidates and of its local front before a final merge with the same selection
calls (guide_select_topk / guide_pareto over the gathered lists).

Everything here is index arithmetic and torch.distributed calls; it runs unchanged on gloo/CPU
tensors (used by the tests) and on nccl/CUDA tensors.  The two `merge_*` functions take the
selection call as an argument: the library's binding on a GPU, and whatever stands in for it in a
CPU test of the plumbing.
"""
from __future__ import annotations

import numpy as np

AXES = ("models", "hw", "fw_f", "batch", "tp", "pairs")


def hw_slice(n_hw: int, rank: int, world: int):
    """Contiguous, near-even slice [lo, hi) of the hardware axis for this rank."""
    base, extra = divmod(n_hw, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_space(space: dict, rank: int, world: int):
    """This rank's sub-space (same axes, a slice of the hardware profiles) and its hardware offset."""
    lo, hi = hw_slice(len(space["hw"]), rank, world)
    if hi == lo:
        raise ValueError(f"rank {rank} of {world} gets no hardware profile ({len(space['hw'])} in all)")
    local = dict(space)
    local["hw"] = np.ascontiguousarray(space["hw"][lo:hi])
    local["hw_mem"] = np.ascontiguousarray(space["hw_mem"][lo:hi])
    return local, lo


def dims(space: dict):
    return [len(space[k]) for k in AXES]


def local_to_global(idx_local, local_space: dict, global_space: dict, hw_offset: int):
    """Config indices of the sub-space -> indices of the whole space (numpy or torch int64 arrays).
    Entries equal to -1 / 2^64-1 (unused slots) are passed through."""
    n_m, n_h, n_f, n_b, n_t, n_l = dims(local_space)
    n_hg = len(global_space["hw"])
    inner = n_f * n_b * n_t * n_l
    idx = idx_local
    unused = idx < 0
    rest = idx % inner
    mh = idx // inner
    h = mh % n_h
    m = mh // n_h
    out = (m * n_hg + h + hw_offset) * inner + rest
    if hasattr(out, "masked_fill"):
        return out.masked_fill(unused, -1)
    return np.where(unused, -1, out)


def all_gather_concat(t, group=None):
    """All-gather equal-length 1-D tensors and concatenate them in rank order."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    bufs = [torch.empty_like(t) for _ in range(world)]
    dist.all_gather(bufs, t.contiguous(), group=group)
    return torch.cat(bufs)


def order_for_merge(global_idx):
    """Permutation that puts gathered candidates in ascending global config index, unused slots
    last, so that position order equals index order and the merge kernel's lowest-position
    tie-break is the lowest-index tie-break of the single-GPU result."""
    import torch
    key = torch.where(global_idx < 0, torch.full_like(global_idx, torch.iinfo(torch.int64).max), global_idx)
    return torch.argsort(key, stable=True)


def concat_gather(parts):
    """Stand-in for all_gather_concat when the shards live in one process: `parts` holds every
    shard's tensor in rank order."""
    import torch
    return torch.cat(list(parts))


def merge_topk(gidx, val, k, select, gather=all_gather_concat):
    """Global top-k from every shard's k candidates.

    gidx: this shard's candidates as *global* config indices (int64, -1 = unused slot); val: their
    key values.  The gathered lists are put in global-index order, so that the selection call's
    lowest-position tie-break is the single-space lowest-index tie-break.  `select(status, values,
    k)` runs the top-k selection over the gathered list (status 0 = candidate, 1 = unused slot) and
    returns (positions int64[k] with -1 for unused, values[k], count).  Returns (global indices
    int64[k], values[k], count)."""
    import torch
    all_idx, all_val = gather(gidx), gather(val)
    order = order_for_merge(all_idx)
    all_idx, all_val = all_idx[order], all_val[order].contiguous()
    status = (all_idx < 0).to(torch.uint8)
    pos, vals, count = select(status, all_val, k)
    found = pos >= 0
    out = torch.full_like(pos, -1)
    out[found] = all_idx[pos[found]]                 # positions in the gathered list -> config indices
    return out, vals, count


def merge_front(gidx, x, y, count, cap, front, gather=all_gather_concat):
    """Global Pareto front from every shard's local front (a point no shard's point dominates is on
    its own shard's front, so the union of the local fronts contains the global one).

    gidx / x / y: this shard's front as global config indices and the two metric values, padded to
    `cap` entries; count: how many are real.  `front(status, xs, ys, cap)` runs the front selection
    over the gathered points and returns (positions int64[<=cap] in ascending x, size).  Returns
    (global indices of the front in ascending x, size)."""
    import torch
    used = torch.arange(gidx.numel(), device=gidx.device) < count
    gidx = torch.where(used, gidx, torch.full_like(gidx, -1))
    all_idx, all_x, all_y = gather(gidx), gather(x), gather(y)
    order = order_for_merge(all_idx)
    all_idx, all_x, all_y = all_idx[order], all_x[order].contiguous(), all_y[order].contiguous()
    status = (all_idx < 0).to(torch.uint8)
    pos, size = front(status, all_x, all_y, cap)
    return all_idx[pos], size


_ARRAY_OF = {"throughput": "thr_decode"}          # metric name -> name of the guide_outputs array that holds it


def kernel_selectors(guide, sp, key, x="latency", y="cost_per_hr"):
    """The merge steps through the library: (select, front) callables for merge_topk / merge_front that
    run guide_select_topk / guide_pareto over the gathered lists (CUDA tensors), with the gathered
    values standing in as the metric arrays of the call.  `sp` is any guide.Space handle at least as
    large as the gathered lists (the calls only use it to check the range)."""
    import torch

    def select(status, values, k):
        m = status.numel()
        out = {"status": status, _ARRAY_OF.get(key, key): values}
        idx = torch.empty(k, dtype=torch.int64, device=values.device)
        val = torch.empty(k, dtype=torch.float64, device=values.device)
        cnt = torch.zeros(1, dtype=torch.int32, device=values.device)
        ws = torch.empty(guide.guide_select_workspace_bytes(sp, k), dtype=torch.uint8, device=values.device)
        guide.guide_select_topk(sp, None, out, {}, key, k, idx, val, cnt, ws, count=m)
        return idx, val, int(cnt.item())           # unused slots come back as 2^64 - 1 = -1

    def front(status, xs, ys, cap):
        m = status.numel()
        out = {"status": status, _ARRAY_OF.get(x, x): xs, _ARRAY_OF.get(y, y): ys}
        idx = torch.empty(cap, dtype=torch.int64, device=xs.device)
        cnt = torch.zeros(1, dtype=torch.int32, device=xs.device)
        ws = torch.empty(guide.guide_pareto_workspace_bytes(sp), dtype=torch.uint8, device=xs.device)
        guide.guide_pareto(sp, None, out, {}, x, y, idx, cnt, ws, count=m)
        size = int(cnt.item())
        return idx[:min(size, cap)], size

    return select, front
