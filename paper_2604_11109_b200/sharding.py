"""Candidate sharding across ranks (one process per GPU) and the one exchange step it needs.

Candidates are independent given the fitted factor, so a pool is split into contiguous shards, every
rank fits the (small) history itself -- the fit is deterministic -- and scores its own shard.  The only
communication is the merge of the per-rank top-k lists: one all-gather of k (value, global index)
pairs per rank, after which every rank holds the global top-k.  Batched workloads shard whole GPs the
same way and need no exchange at all.
"""
from __future__ import annotations


def shard_bounds(m: int, world: int, rank: int):
    """Contiguous shard [lo, hi) of ``m`` items for ``rank`` of ``world``; sizes differ by at most one."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(m, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def merge_topk(local_val, local_idx, k: int, shard_lo: int, group=None, topk_fn=None):
    """All-gather the ranks' local top-k lists and select the global top-k on every rank.

    local_val [k] float32 sorted descending (ties by ascending local index), local_idx [k] int32 local
    to the shard starting at ``shard_lo``.  Every rank must pass the same k.  ``topk_fn(values, k)``
    returns the positions of the k largest values, ties to the lower position (``binding.r3_topk`` on
    a GPU; any exact stand-in on CPU).  Because shards are contiguous and gathered in rank order, "lower
    position" is also "lower global index", so ties resolve as in the single-GPU call.
    Returns (values [k], global indices [k] int64).
    """
    import torch
    import torch.distributed as dist

    world = dist.get_world_size(group)
    gidx = local_idx.to(torch.int64) + int(shard_lo)
    vals = [torch.empty_like(local_val) for _ in range(world)]
    idxs = [torch.empty_like(gidx) for _ in range(world)]
    dist.all_gather(vals, local_val.contiguous(), group=group)
    dist.all_gather(idxs, gidx.contiguous(), group=group)
    allv, alli = torch.cat(vals), torch.cat(idxs)
    pos = topk_fn(allv, min(k, allv.numel())).to(torch.int64)
    return allv[pos], alli[pos]
