"""The multi-rank host logic on CPU: two gloo ranks shard a pool, build local top-k lists with the
oracle's ordering, and merge them; the result equals the single-process top-k."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_11109_b200.sharding import merge_topk, shard_bounds


def test_shard_bounds_cover_exactly():
    for m, world in ((10, 3), (7, 8), (1 << 20, 8), (5, 1)):
        spans = [shard_bounds(m, world, r) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == m
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        sizes = [hi - lo for lo, hi in spans]
        assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_bounds(4, 2, 2)


def _exact_topk(values, k):
    v = values.numpy().astype(np.float64)
    return torch.from_numpy(np.lexsort((np.arange(v.size), -v))[:k].copy())


def _worker(rank, world, port, m, k, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rng = np.random.default_rng(5)
        ei = rng.random(m).astype(np.float32)
        ei[[3, m // 2 + 1, m - 2]] = 2.0       # a tie that spans both shards
        lo, hi = shard_bounds(m, world, rank)
        local = ei[lo:hi]
        order = np.lexsort((np.arange(local.size), -local.astype(np.float64)))[:k]
        val, idx = merge_topk(torch.from_numpy(local[order].copy()), torch.from_numpy(order.astype(np.int32)), k, lo,
                              topk_fn=_exact_topk)
        ref = np.lexsort((np.arange(m), -ei.astype(np.float64)))[:k]
        ok = np.array_equal(idx.numpy(), ref) and np.array_equal(val.numpy(), ei[ref])
        q.put((rank, bool(ok)))
    finally:
        dist.destroy_process_group()


def test_two_rank_merge_equals_single_process_topk():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, 1001, 16, q)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    results = dict(q.get(timeout=10) for _ in range(2))
    assert results == {0: True, 1: True}
