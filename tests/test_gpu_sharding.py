"""The exchange step of the multi-GPU path on a GPU: a one-rank NCCL group gathers the local top-k list and
`merge_topk` selects with the library's own `r3_topk`, as `bench.py --gpus N` does on every rank."""
import os
import socket

import numpy as np
import pytest

from paper_2604_11109_b200 import binding as b
from paper_2604_11109_b200.sharding import merge_topk

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def test_merge_topk_with_nccl_and_the_library_topk():
    import torch.distributed as dist

    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        rng = np.random.default_rng(9)
        m, k, shard_lo = 5000, 32, 123456
        ei = rng.random(m).astype(np.float32)
        ei[[7, 4000]] = 2.0   # a tie: the lower index comes first
        idx, val = b.r3_topk(torch.from_numpy(ei).cuda(), k)
        gval, gidx = merge_topk(val, idx, k, shard_lo, topk_fn=lambda v, kk: b.r3_topk(v, kk)[0])
        ref = np.lexsort((np.arange(m), -ei.astype(np.float64)))[:k]
        assert np.array_equal(gidx.cpu().numpy(), ref + shard_lo)
        assert np.array_equal(gval.cpu().numpy(), ei[ref])
        # the barrier and the max-reduction of the timing that the benchmark uses
        dist.barrier()
        t = torch.tensor([1.5], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert float(t.item()) == 1.5
    finally:
        dist.destroy_process_group()
