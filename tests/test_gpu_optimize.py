"""GPU tests of r3_gp_refit and r3_gp_optimize.

The optimiser is host logic around two device computations that have their own parity tests (the fit and the
log marginal likelihood), so what is checked here is the result: the value it reports is the oracle's evidence at
the hyper-parameters it returns, the oracle's gradient there is small, it is no worse than the start and agrees
with SciPy's L-BFGS-B run on the oracle's evidence from the same start, and the handle it leaves behind is the fit
at those hyper-parameters.
"""
import numpy as np
import pytest
from scipy import optimize

from oracle import gp_oracle as o
from paper_2604_11109_b200 import binding as b

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def sample_problem(seed, n, d, ell_true, sf2_true, sn2_true):
    """A history drawn from the GP prior with known hyper-parameters (so the evidence has a clear maximum)."""
    rng = np.random.default_rng(seed)
    X = rng.uniform(0, 1, (n, d)).astype(np.float32)
    K = o.gram(X, np.asarray(ell_true, dtype=np.float32), sf2_true, sn2_true)
    y = (np.linalg.cholesky(K) @ rng.standard_normal(n)).astype(np.float32)
    return X, y


def scipy_optimum(X, y, ell0, sf20, sn20):
    d = X.shape[1]
    theta0 = np.concatenate([np.log(ell0), [np.log(sf20), np.log(sn20)]])

    def negative(theta):
        v, g = o.lml(X, y, np.exp(theta[:d]), np.exp(theta[d]), np.exp(theta[d + 1]))
        return -v, -g

    bounds = [(np.log(1e-3), np.log(1e3))] * d + [(np.log(1e-6), np.log(1e6)), (np.log(1e-8), np.log(1e2))]
    res = optimize.minimize(negative, theta0, jac=True, method="L-BFGS-B", bounds=bounds,
                            options={"maxiter": 200, "ftol": 1e-12, "gtol": 1e-6})
    return -res.fun


@pytest.mark.parametrize("seed,n,d", [(0, 120, 1), (1, 150, 2), (2, 200, 3)])
def test_optimum_matches_scipy_on_the_oracle(seed, n, d):
    ell_true = [0.25, 0.6, 0.4][:d]
    X, y = sample_problem(seed, n, d, ell_true, 1.5, 0.02)
    ell0, sf20, sn20 = np.ones(d, np.float32), np.float32(1.0), np.float32(0.1)
    gp = b.r3_gp_fit(dev(X), dev(y), ell0, sf20, sn20)
    start = b.r3_gp_lml(gp)[0][0]
    ell, sf2, sn2, lml, used = b.r3_gp_optimize(gp, max_evals=120, gtol=1e-3)
    assert 1 <= used <= 120
    v, g = o.lml(X, y, ell[0], sf2[0], sn2[0])
    assert lml[0] == pytest.approx(v, rel=1e-9, abs=1e-7)          # the reported value is the evidence at the result
    assert lml[0] >= start
    assert np.abs(g).max() <= 2e-2                                    # a stationary point (gtol 1e-3 at FP32 parameters)
    ref = scipy_optimum(X, y, ell0, sf20, sn20)
    assert lml[0] >= ref - 1e-3 * max(1.0, abs(ref))
    # the handle is the fit at the returned hyper-parameters
    alpha, L = b.r3_gp_get_factor(gp)
    f = o.fit(X, y, ell[0], sf2[0], sn2[0])
    assert np.allclose(L[0], f.L, rtol=1e-9, atol=1e-11)
    assert np.allclose(alpha[0], f.alpha, rtol=1e-7, atol=1e-9 * np.abs(f.alpha).max())
    gp.close()


def test_batch_members_are_optimised_independently():
    probs = [sample_problem(10 + q, 100, 2, [0.3, 0.7], 1.0 + q, 0.01) for q in range(3)]
    X = np.stack([p[0] for p in probs])
    y = np.stack([p[1] for p in probs])
    ell0, sf20, sn20 = np.ones((3, 2), np.float32), np.ones(3, np.float32), np.full(3, 0.1, np.float32)
    gp = b.r3_gp_fit(dev(X), dev(y), ell0, sf20, sn20)
    ell, sf2, sn2, lml, used = b.r3_gp_optimize(gp, max_evals=150, gtol=1e-3)
    for q in range(3):
        single = b.r3_gp_fit(dev(X[q]), dev(y[q]), ell0[q], sf20[q], sn20[q])
        e1, s1, n1, l1, _ = b.r3_gp_optimize(single, max_evals=150, gtol=1e-3)
        assert lml[q] == pytest.approx(l1[0], rel=1e-6, abs=1e-5)
        np.testing.assert_allclose(ell[q], e1[0], rtol=1e-3)
        single.close()
    gp.close()


def test_refit_and_its_errors():
    rng = np.random.default_rng(4)
    X = rng.uniform(0, 1, (1, 60, 3)).astype(np.float32)
    X[0, 1] = X[0, 0]                                                 # duplicate rows: singular without noise
    y = rng.normal(0, 1, (1, 60)).astype(np.float32)
    ell, sf2, sn2 = np.full((1, 3), 0.5, np.float32), np.ones(1, np.float32), np.full(1, 1e-2, np.float32)
    gp = b.r3_gp_fit(dev(X), dev(y), ell, sf2, sn2)
    new_ell = np.array([[0.2, 0.9, 0.4]], np.float32)
    b.r3_gp_refit(gp, new_ell, np.float32(2.0), np.float32(0.05))
    alpha, L = b.r3_gp_get_factor(gp)
    f = o.fit(X[0], y[0], new_ell[0], 2.0, 0.05)
    assert np.allclose(L[0], f.L, rtol=1e-9, atol=1e-11)
    with pytest.raises(b.R3Error) as e:
        b.r3_gp_refit(gp, new_ell, np.float32(1.0), np.float32(0.0))   # rows 0 and 1 coincide: the second pivot is 1 - 1
    assert e.value.status == 3
    alpha2, L2 = b.r3_gp_get_factor(gp)                               # the previous hyper-parameters were kept
    assert np.allclose(L2[0], f.L, rtol=1e-12, atol=1e-14)
    with pytest.raises(b.R3Error) as e:
        b.r3_gp_refit(gp, -new_ell, np.float32(2.0), np.float32(0.1))
    assert e.value.status == 1
    with pytest.raises(b.R3Error) as e:
        b.r3_gp_optimize(gp, max_evals=0)
    assert e.value.status == 1
    gp.close()
