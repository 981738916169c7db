"""r3_topk_noalloc, the entry point for callers that cannot allocate device memory at call time
(a proposal loop inside a replay server, a host whose device memory belongs to another framework's
arena): its workspace is a fixed array inside the library.  It must return exactly what r3_topk
returns, call after call, because every call reuses that one array.

Collected last on purpose: a run that stops at the first failure has then already run everything else.
"""
import ctypes

import numpy as np
import pytest

from oracle import gp_oracle as o
from paper_2604_11109_b200 import binding as b

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _values(seed, batch, m):
    rng = np.random.default_rng(seed)
    e = rng.random((batch, m)).astype(np.float32)
    e[:, [1, m // 3, m - 1]] = 1.5          # ties at the top: the lower index must win in both entry points
    return torch.from_numpy(e).cuda()


@pytest.mark.parametrize("batch,m,k", [(1, 1 << 20, 128), (64, 65536, 16), (3, 10001, 7)])
def test_noalloc_equals_topk_on_two_calls_in_a_row(batch, m, k):
    idx = torch.empty((batch, k), dtype=torch.int32, device="cuda")
    val = torch.empty((batch, k), dtype=torch.float32, device="cuda")
    for call in range(2):                    # the second call finds the first call's keys in the array
        e = _values(100 * k + call, batch, m)
        ref_idx, ref_val = b.r3_topk(e, k)
        b.r3_topk_noalloc(e, k, (idx, val))
        torch.cuda.synchronize()
        assert torch.equal(idx, ref_idx)     # integer work: bit-exact
        assert torch.equal(val, ref_val)
        # and against the oracle's definition of the selection itself
        e_h, idx_h = e.cpu().numpy(), idx.cpu().numpy()
        for q in range(batch):
            oidx, oval = o.topk(e_h[q], k)
            assert np.array_equal(idx_h[q], oidx)
            assert np.array_equal(val.cpu().numpy()[q], oval.astype(np.float32))


def test_noalloc_rejects_requests_beyond_its_fixed_capacity():
    e = _values(5, 1, 1 << 20)
    idx = torch.empty((1, 1024), dtype=torch.int32, device="cuda")
    with pytest.raises(b.R3Error) as err:   # 256 chunks * 1024 keys > 65536
        b.r3_topk_noalloc(e, 1024, (idx, None))
    assert err.value.status == 7 and "capacity" in str(err.value)
    # and still works afterwards, values omitted
    idx = torch.empty((1, 8), dtype=torch.int32, device="cuda")
    b.r3_topk_noalloc(e, 8, (idx, None))
    assert torch.equal(idx, b.r3_topk(e, 8)[0])
