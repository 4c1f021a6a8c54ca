"""Multi-GPU plumbing: configs are independent, so the space is cut along the hardware axis, each
rank evaluates its slice with the single-GPU kernels, and the only exchange is an all-gather of
each rank's k best candidates (and its local front) before a final merge with the same kernels.

Everything here is index arithmetic and torch.distributed calls; it runs unchanged on gloo/CPU
tensors (used by the tests) and on nccl/CUDA tensors.
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
