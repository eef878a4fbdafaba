"""Request-level sharding for N > 1 GPUs.

Requests of a `forward` batch are independent (each reads only its own page list), so the path
shards by request with no data-path collective: rank k plans and runs its own contiguous slice
of the batch on its own GPU and pool.  The only cross-rank traffic is the timing reduction.
"""
from __future__ import annotations

import numpy as np


def shard_bounds(n_requests: int, world: int, rank: int):
    """Contiguous, balanced slice [lo, hi) of the request ids for `rank`."""
    base, rem = divmod(n_requests, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def shard_batch(qo_indptr, page_indptr, page_indices, last_page_len, world, rank, mask_indptr=None, mask=None):
    """The CSR arrays of this rank's slice of a batch, re-based to start at 0."""
    qo_indptr, page_indptr = np.asarray(qo_indptr), np.asarray(page_indptr)
    lo, hi = shard_bounds(len(qo_indptr) - 1, world, rank)
    out = {
        "requests": (lo, hi),
        "qo_indptr": (qo_indptr[lo:hi + 1] - qo_indptr[lo]).astype(np.int32),
        "page_indptr": (page_indptr[lo:hi + 1] - page_indptr[lo]).astype(np.int32),
        "page_indices": np.asarray(page_indices)[page_indptr[lo]:page_indptr[hi]].astype(np.int32),
        "last_page_len": np.asarray(last_page_len)[lo:hi].astype(np.int32),
        "token_range": (int(qo_indptr[lo]), int(qo_indptr[hi])),
        "mask_indptr": None, "mask": None,
    }
    if mask_indptr is not None:
        mask_indptr = np.asarray(mask_indptr)
        out["mask_indptr"] = (mask_indptr[lo:hi + 1] - mask_indptr[lo]).astype(np.int64)
        out["mask"] = np.asarray(mask)[mask_indptr[lo]:mask_indptr[hi]]
    return out


def aggregate(tokens: int, ms: float, group=None):
    """Whole-job figures: total tokens over all ranks and the slowest rank's time (torch.distributed
    must be initialised when world > 1).  Returns (total_tokens, max_ms)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return tokens, ms
    dev = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    t = torch.tensor([float(tokens)], dtype=torch.float64, device=dev)
    m = torch.tensor([float(ms)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    dist.all_reduce(m, op=dist.ReduceOp.MAX, group=group)
    return int(round(t.item())), float(m.item())
