"""GPU parity of r3_gp_lml against the oracle's log marginal likelihood and gradient (both FP64; the
device sums in another order, so agreement is to rounding: relative 1e-9 of the largest term)."""
import numpy as np
import pytest

from oracle import gp_oracle as o
from paper_2604_11109_b200 import binding as b
from paper_2604_11109_b200 import workloads as w

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def check(g):
    gp = b.r3_gp_fit(dev(g["X"]), dev(g["y"]), g["ell"], g["sf2"], g["sn2"])
    lml, grad = b.r3_gp_lml(gp)
    for q in range(g["X"].shape[0]):
        v, gr = o.lml(g["X"][q], g["y"][q], g["ell"][q], g["sf2"][q], g["sn2"][q])
        assert lml[q] == pytest.approx(v, rel=1e-10, abs=1e-9)
        np.testing.assert_allclose(grad[q], gr, rtol=1e-8, atol=1e-9 * max(1.0, np.abs(gr).max()))
    gp.close()


@pytest.mark.parametrize("batch,n,d", [(1, 1, 1), (1, 7, 2), (2, 33, 5), (1, 100, 40), (3, 257, 9), (1, 600, 70)])
def test_random_problems(batch, n, d):
    rng = np.random.default_rng(300 + n)
    check({
        "X": rng.uniform(0, 1, (batch, n, d)).astype(np.float32),
        "y": rng.normal(0, 1, (batch, n)).astype(np.float32),
        "ell": rng.uniform(0.3, 1.5, (batch, d)).astype(np.float32),
        "sf2": rng.uniform(0.5, 2.0, batch).astype(np.float32),
        "sn2": rng.uniform(1e-3, 1e-1, batch).astype(np.float32),
    })


@pytest.mark.parametrize("cfg", [1, 2])
def test_workload_histories(cfg):
    c = w.get_config(cfg, m=16)
    check(w.generate(c))


def test_after_append_equals_fit_of_the_whole_history():
    rng = np.random.default_rng(5)
    X = rng.uniform(0, 1, (1, 90, 4)).astype(np.float32)
    y = rng.normal(0, 1, (1, 90)).astype(np.float32)
    ell, sf2, sn2 = np.full((1, 4), 0.6, np.float32), np.ones(1, np.float32), np.full(1, 1e-2, np.float32)
    gp = b.r3_gp_fit(dev(X[:, :60]), dev(y[:, :60]), ell, sf2, sn2)
    b.r3_gp_append(gp, dev(X[:, 60:]), dev(y[:, 60:]))
    lml, grad = b.r3_gp_lml(gp)
    v, gr = o.lml(X[0], y[0], ell[0], sf2[0], sn2[0])
    assert lml[0] == pytest.approx(v, rel=1e-10)
    np.testing.assert_allclose(grad[0], gr, rtol=1e-8, atol=1e-9)
    gp.close()
