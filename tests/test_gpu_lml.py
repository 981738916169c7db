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


def _lml_extended(X, y, ell, sf2, sn2):
    """The evidence in 80-bit arithmetic by the textbook recurrences (a reference for ill-conditioned cases, where
    any FP64 factorisation has lost digits): unblocked Cholesky, forward substitution, sum of log pivots."""
    LD = np.longdouble
    X, y, ell = X.astype(LD), y.astype(LD), ell.astype(LD)
    n = X.shape[0]
    D = (X[:, None, :] - X[None, :, :]) / ell
    s = np.sqrt(LD(5)) * np.sqrt((D * D).sum(-1))
    K = LD(sf2) * (1 + s + s * s / 3) * np.exp(-s) + LD(sn2) * np.eye(n, dtype=LD)
    L = np.zeros((n, n), dtype=LD)
    for j in range(n):
        L[j, j] = np.sqrt(K[j, j] - (L[j, :j] ** 2).sum())
        L[j + 1:, j] = (K[j + 1:, j] - L[j + 1:, :j] @ L[j, :j]) / L[j, j]
    z = np.zeros(n, dtype=LD)
    for i in range(n):
        z[i] = (y[i] - L[i, :i] @ z[:i]) / L[i, i]
    return float(-0.5 * (z @ z) - np.log(np.diag(L)).sum() - 0.5 * n * np.log(2 * LD(np.pi)))


@pytest.mark.parametrize("seed,n,d", [(1, 90, 6), (2, 115, 1), (3, 160, 9)])
def test_ill_conditioned_history_is_as_accurate_as_the_oracle(seed, n, d):
    """Noise-free linear data at the corner the hyper-parameter fit runs into on such data (lengthscales 1000, signal
    variance 1e6, noise 1e-8): the last digits of the small pivots are gone in FP64 whoever factors, and both the
    library and the LAPACK-based oracle are off by 0.1 to 1 in an evidence of 500 to 1000.  Against an 80-bit
    reference the library must not be further off than a few times the oracle (a panel solved with a diagonal
    block's explicit inverse was 5 to 60 times further off; the blocked factorisation uses forward substitution)."""
    if np.finfo(np.longdouble).eps > 2e-19:
        pytest.skip("no 80-bit long double on this platform")
    rng = np.random.default_rng(7000 + seed)
    X = rng.uniform(0, 1, (1, n, d)).astype(np.float32)
    y = (3.0 * X.sum(-1)).astype(np.float32)
    ell = np.full((1, d), 1000.0, np.float32)
    sf2, sn2 = np.full(1, 1e6, np.float32), np.full(1, 1e-8, np.float32)
    gp = b.r3_gp_fit(dev(X), dev(y), ell, sf2, sn2)
    lml, _ = b.r3_gp_lml(gp)
    gp.close()
    ref = _lml_extended(X[0], y[0], ell[0], sf2[0], sn2[0])
    v, _ = o.lml(X[0], y[0], ell[0], sf2[0], sn2[0])
    err_lib, err_oracle = abs(lml[0] - ref), abs(v - ref)
    assert err_lib <= 4.0 * err_oracle + 1e-7 * abs(ref), (lml[0], v, ref)
    assert err_lib <= 2e-3 * abs(ref)
