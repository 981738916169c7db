"""Pins of the oracle's log marginal likelihood and its gradient (CPU only): a closed form, central
finite differences of the value, and scikit-learn's GaussianProcessRegressor with the same kernel
(an independent implementation of both the value and the gradient in log-parameters)."""
import math

import numpy as np
import pytest
from sklearn.gaussian_process import GaussianProcessRegressor
from sklearn.gaussian_process.kernels import ConstantKernel, Matern, WhiteKernel

from oracle import gp_oracle as o


def problem(seed, n, d):
    rng = np.random.default_rng(seed)
    X = rng.uniform(0, 1, (n, d)).astype(np.float32)
    y = rng.normal(0, 1, n).astype(np.float32)
    ell = rng.uniform(0.2, 1.5, d).astype(np.float32)
    return X, y, ell, np.float32(rng.uniform(0.5, 2.0)), np.float32(rng.uniform(1e-3, 1e-1))


def test_single_observation_closed_form():
    X = np.array([[0.3, 0.7]], dtype=np.float32)
    y = np.array([1.5], dtype=np.float32)
    sf2, sn2 = np.float32(2.0), np.float32(0.5)
    v, g = o.lml(X, y, [0.4, 0.9], sf2, sn2)
    k = 2.5
    assert v == pytest.approx(-0.5 * 1.5 ** 2 / k - 0.5 * math.log(k) - 0.5 * math.log(2 * math.pi), rel=1e-14)
    # d/dlog sf2 = sf2 * d/dk, d/dlog sn2 = sn2 * d/dk with d lml/dk = y^2/(2 k^2) - 1/(2 k)
    dk = 1.5 ** 2 / (2 * k * k) - 1 / (2 * k)
    np.testing.assert_allclose(g, [0.0, 0.0, 2.0 * dk, 0.5 * dk], rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("seed,n,d", [(0, 12, 1), (1, 40, 3), (2, 90, 7)])
def test_gradient_is_the_derivative_of_the_value(seed, n, d):
    X, y, ell, sf2, sn2 = problem(seed, n, d)
    _, g = o.lml(X, y, ell, sf2, sn2)
    theta = np.concatenate([np.log(ell.astype(np.float64)), [math.log(float(sf2)), math.log(float(sn2))]])

    def value(t):
        # parameters are FP32 at the oracle's boundary: evaluate on a grid coarse enough not to notice
        return o.lml(X, y, np.exp(t[:d]), np.exp(t[d]), np.exp(t[d + 1]))[0]

    h = 2e-2
    for p in range(d + 2):
        tp, tm = theta.copy(), theta.copy()
        tp[p] += h
        tm[p] -= h
        t2p, t2m = theta.copy(), theta.copy()
        t2p[p] += 2 * h
        t2m[p] -= 2 * h
        fd = (8 * (value(tp) - value(tm)) - (value(t2p) - value(t2m))) / (12 * h)   # fourth-order central difference
        assert g[p] == pytest.approx(fd, rel=2e-4, abs=2e-4 * np.abs(g).max())


@pytest.mark.parametrize("seed,n,d", [(5, 30, 2), (6, 120, 6)])
def test_against_scikit_learn(seed, n, d):
    X, y, ell, sf2, sn2 = problem(seed, n, d)
    kernel = ConstantKernel(float(sf2)) * Matern(length_scale=ell.astype(np.float64), nu=2.5) + WhiteKernel(float(sn2))
    gpr = GaussianProcessRegressor(kernel=kernel, optimizer=None, alpha=0.0).fit(X.astype(np.float64),
                                                                                 y.astype(np.float64))
    ref_v, ref_g = gpr.log_marginal_likelihood(gpr.kernel_.theta, eval_gradient=True)
    # scikit-learn's theta: (log constant, log length scales, log noise)
    v, g = o.lml(X, y, ell, sf2, sn2)
    assert v == pytest.approx(ref_v, rel=1e-10)
    np.testing.assert_allclose(g[d], ref_g[0], rtol=1e-8, atol=1e-9)
    np.testing.assert_allclose(g[:d], ref_g[1:1 + d], rtol=1e-8, atol=1e-9)
    np.testing.assert_allclose(g[d + 1], ref_g[1 + d], rtol=1e-8, atol=1e-9)


def test_value_agrees_with_the_factor_of_the_fit():
    X, y, ell, sf2, sn2 = problem(9, 60, 4)
    f = o.fit(X, y, ell, sf2, sn2)
    v, _ = o.lml(X, y, ell, sf2, sn2)
    ref = -0.5 * float(y.astype(np.float64) @ f.alpha) - np.log(np.diag(f.L)).sum() - 30 * math.log(2 * math.pi)
    assert v == pytest.approx(ref, rel=1e-12)
