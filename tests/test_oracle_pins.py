"""Pins of the FP64 CPU oracle against things other than itself.

Closed forms (40-digit values in tests/golden/closed_forms.json, written by a
script that uses mpmath only), exact identities of GP regression, limits,
invariances, an independent explicit-inverse implementation for tiny n, and a
library Gaussian-process regressor.  Each test names the step of the oracle's
header it pins.
"""
import json
import math
import os

import numpy as np
import pytest

from oracle import brute_force, gp_oracle as o

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "closed_forms.json")))


def _rand_problem(seed, n, d, m, sn2=1e-3, sf2=1.0):
    rng = np.random.default_rng(seed)
    X = rng.uniform(0, 1, (n, d)).astype(np.float32)
    y = rng.normal(0, 1, n).astype(np.float32)
    ell = rng.uniform(0.2, 1.5, d).astype(np.float32)
    Xc = rng.uniform(-0.2, 1.2, (m, d)).astype(np.float32)
    return X, y, ell, np.float32(sf2), np.float32(sn2), Xc


# ------------------------------------------------------------------ step (1): covariance
def test_matern52_closed_form_values():
    for s, v in GOLD["matern52_of_s"].items():
        s = float(s)
        assert o.matern52(s * s / 5.0) == pytest.approx(float(v), rel=1e-13, abs=0)
    # 7/(3e) at s = 1
    assert o.matern52(0.2) == pytest.approx(7.0 / (3.0 * math.e), rel=2e-15)


def test_kernel_is_ard_lengthscale_not_squared_not_inverse():
    # s = sqrt(5) * |dx| / ell ; with dx = 1, ell = sqrt(5): s = 1
    v = o.kernel([0.0], [1.0], [math.sqrt(5.0)], 2.0)
    assert v == pytest.approx(2.0 * float(GOLD["matern52_of_s"]["1"]), rel=1e-6)
    # two features with different lengthscales: r^2 = (1/0.5)^2 + (1/2)^2 = 4.25
    v = o.kernel([0.0, 0.0], [1.0, 1.0], [0.5, 2.0], 1.0)
    s = math.sqrt(5 * 4.25)
    assert v == pytest.approx((1 + s + s * s / 3) * math.exp(-s), rel=1e-12)
    # symmetric, maximal at zero distance
    assert o.kernel([0.3, 0.1], [0.3, 0.1], [0.5, 2.0], 1.7) == pytest.approx(1.7, rel=1e-15)


def test_gram_symmetric_noise_on_diagonal_only():
    X, y, ell, sf2, sn2, _ = _rand_problem(1, 9, 3, 1, sn2=0.05, sf2=1.3)
    K = o.gram(X, ell, sf2, sn2)
    assert np.array_equal(K, K.T)
    assert np.allclose(np.diag(K), float(sf2) + float(sn2), rtol=1e-15)
    K0 = o.gram(X, ell, sf2, 0.0)
    assert np.allclose(K - K0, float(sn2) * np.eye(9), atol=1e-15)


# ------------------------------------------------------------------ step (2): Cholesky
def test_cholesky_reconstructs_and_matches_lapack():
    X, y, ell, sf2, sn2, _ = _rand_problem(2, 40, 4, 1)
    K = o.gram(X, ell, sf2, sn2)
    L = o.cholesky(K)
    assert np.all(np.triu(L, 1) == 0)
    assert np.allclose(L @ L.T, K, rtol=0, atol=1e-13)
    assert np.allclose(L, np.linalg.cholesky(K), rtol=0, atol=1e-12)


def test_cholesky_rejects_singular_matrix():
    X = np.array([[0.1, 0.2], [0.1, 0.2], [0.7, 0.3]], dtype=np.float32)  # duplicate row, no noise
    with pytest.raises(o.NotPositiveDefinite):
        o.fit(X, np.zeros(3, np.float32), np.ones(2, np.float32), 1.0, 0.0)


def test_fit_rejects_non_finite():
    X = np.array([[0.1], [np.nan]], dtype=np.float32)
    with pytest.raises(ValueError):
        o.fit(X, np.zeros(2, np.float32), np.ones(1, np.float32), 1.0, 0.1)


# ------------------------------------------------------------------ step (3): weights
def test_alpha_solves_the_linear_system():
    X, y, ell, sf2, sn2, _ = _rand_problem(3, 30, 5, 1)
    f = o.fit(X, y, ell, sf2, sn2)
    K = o.gram(X, ell, sf2, sn2)
    assert np.allclose(K @ f.alpha, y.astype(np.float64), rtol=0, atol=1e-10)
    assert f.best == float(y.min())


# ------------------------------------------------------------------ step (5): EI
def test_ei_closed_form_values():
    for z, v in GOLD["h_of_z"].items():
        z = float(z)
        # sigma = 1, best = 0, mu = -z  ->  EI = h(z)
        assert o.ei(-z, 1.0, 0.0) == pytest.approx(float(v), rel=5e-13)
        # EI = sigma * h(z) for any sigma and shift
        assert o.ei(2.0 - 0.3 * z, 0.3, 2.0) == pytest.approx(0.3 * float(v), rel=1e-11)


def test_ei_reflection_identity_and_limits():
    for z in (0.1, 0.7, 2.5, 5.0):
        assert o.ei(-z, 1.0, 0.0) - o.ei(z, 1.0, 0.0) == pytest.approx(z, rel=1e-12)
    # sigma = 0: plain improvement
    assert o.ei(0.25, 0.0, 1.0) == 0.75
    assert o.ei(1.25, 0.0, 1.0) == 0.0
    # sigma -> 0 approaches max(best - mu, 0); EI >= max(best - mu, 0) >= 0
    assert o.ei(0.25, 1e-9, 1.0) == pytest.approx(0.75, rel=1e-12)
    assert o.ei(1.25, 1e-3, 1.0) >= 0.0
    for mu, sd in ((0.3, 0.2), (-1.0, 0.5), (2.0, 1.5)):
        assert o.ei(mu, sd, 0.5) >= max(0.5 - mu, 0.0)


def test_ei_partial_derivatives():
    # dEI/dsigma = phi(z) > 0 ; dEI/dmu = -Phi(z) < 0
    mu, sd, best, h = 0.4, 0.7, 0.1, 1e-6
    z = (best - mu) / sd
    phi = math.exp(-0.5 * z * z) / math.sqrt(2 * math.pi)
    Phi = 0.5 * math.erfc(-z / math.sqrt(2))
    dsd = (o.ei(mu, sd + h, best) - o.ei(mu, sd - h, best)) / (2 * h)
    dmu = (o.ei(mu + h, sd, best) - o.ei(mu - h, sd, best)) / (2 * h)
    assert dsd == pytest.approx(phi, rel=1e-7)
    assert dmu == pytest.approx(-Phi, rel=1e-7)


# ------------------------------------------------------------------ steps (2)-(5) end to end
def test_single_observation_closed_form():
    c = GOLD["n1"]
    f = o.fit(np.array(c["X"]), np.array(c["y"]), np.array(c["ell"]), c["sf2"], c["sn2"])
    mu, sd, e = o.score(f, np.array([[1.0 / math.sqrt(5.0)]]))
    # inputs are rounded to FP32 before the oracle widens them, hence 1e-6
    assert mu[0] == pytest.approx(float(c["mu"]), rel=1e-6)
    assert sd[0] == pytest.approx(float(c["sigma"]), rel=1e-6)
    assert sd[0] ** 2 == pytest.approx(float(c["var"]), rel=1e-6)


def test_three_observation_ard_closed_form():
    c = GOLD["n3_ard"]
    X, y, ell = np.array(c["X"]), np.array(c["y"]), np.array(c["ell"])
    K = o.gram(X, ell, np.float32(c["sf2"]), np.float32(c["sn2"]))
    assert np.allclose(K, np.array(c["K"], dtype=float), rtol=1e-6)
    f = o.fit(X, y, ell, c["sf2"], c["sn2"])
    assert np.allclose(f.alpha, np.array(c["alpha"], dtype=float), rtol=2e-5)
    for p in c["points"]:
        mu, sd, e = o.score(f, np.array([p["xstar"]]))
        assert mu[0] == pytest.approx(float(p["mu"]), rel=2e-5, abs=1e-9)
        assert sd[0] == pytest.approx(float(p["sigma"]), rel=2e-5)
        assert e[0] == pytest.approx(float(p["ei"]), rel=2e-4)
    # far point: prior
    far = c["points"][2]
    assert float(far["sigma"]) == pytest.approx(math.sqrt(1.5), rel=1e-12)


def test_training_point_identities():
    # mu(x_i) = y_i - sn2*alpha_i ; var(x_i) = sn2 - sn2^2 [K^-1]_ii ; 0 < sigma(x_i) <= sqrt(sn2)
    X, y, ell, sf2, sn2, _ = _rand_problem(4, 24, 3, 1, sn2=1e-2)
    f = o.fit(X, y, ell, sf2, sn2)
    mu, sd, _ = o.score(f, X)
    Kinv = np.linalg.inv(o.gram(X, ell, sf2, sn2))
    s2 = float(sn2)
    assert np.allclose(mu, y.astype(np.float64) - s2 * f.alpha, rtol=0, atol=1e-10)
    assert np.allclose(sd ** 2, s2 - s2 * s2 * np.diag(Kinv), rtol=1e-7, atol=1e-12)
    assert np.all(sd > 0) and np.all(sd <= math.sqrt(s2) * (1 + 1e-12))


def test_far_field_is_the_prior():
    X, y, ell, sf2, sn2, _ = _rand_problem(5, 12, 2, 1, sf2=2.5)
    f = o.fit(X, y, ell, sf2, sn2)
    mu, sd, e = o.score(f, np.full((1, 2), 500.0, dtype=np.float32))
    sf = math.sqrt(float(sf2))
    assert abs(mu[0]) < 1e-200 or mu[0] == 0.0
    assert sd[0] == pytest.approx(sf, rel=1e-15)
    z = f.best / sf
    hz = z * 0.5 * math.erfc(-z / math.sqrt(2)) + math.exp(-0.5 * z * z) / math.sqrt(2 * math.pi)
    assert e[0] == pytest.approx(sf * hz, rel=1e-12)


@pytest.mark.parametrize("seed,n,d", [(10, 1, 1), (11, 5, 2), (12, 16, 6), (13, 13, 3)])
def test_agrees_with_explicit_inverse_brute_force(seed, n, d):
    X, y, ell, sf2, sn2, Xc = _rand_problem(seed, n, d, 7, sn2=5e-3, sf2=1.4)
    f = o.fit(X, y, ell, sf2, sn2)
    mu, sd, e = o.score(f, Xc)
    bmu, bsd, bei = brute_force.posterior(X.tolist(), y.tolist(), ell.tolist(), float(sf2), float(sn2),
                                          Xc.tolist())
    assert np.allclose(mu, bmu, rtol=1e-9, atol=1e-11)
    assert np.allclose(sd, bsd, rtol=1e-8, atol=1e-11)
    assert np.allclose(e, bei, rtol=1e-7, atol=1e-13)


def test_invariances():
    X, y, ell, sf2, sn2, Xc = _rand_problem(6, 20, 4, 11)
    f = o.fit(X, y, ell, sf2, sn2)
    mu, sd, e = o.score(f, Xc)
    # permuting the training rows changes nothing
    p = np.random.default_rng(0).permutation(20)
    mu2, sd2, e2 = o.score(o.fit(X[p], y[p], ell, sf2, sn2), Xc)
    assert np.allclose(mu, mu2, atol=1e-11) and np.allclose(sd, sd2, atol=1e-11)
    # permuting the candidates permutes the outputs
    q = np.random.default_rng(1).permutation(11)
    mu3, sd3, e3 = o.score(f, Xc[q])
    assert np.array_equal(mu3, mu[q]) and np.array_equal(sd3, sd[q]) and np.array_equal(e3, e[q])
    # scaling feature j and its lengthscale by the same power of two changes nothing
    Xs, Xcs, ells = X.copy(), Xc.copy(), ell.copy()
    Xs[:, 2] *= 4
    Xcs[:, 2] *= 4
    ells[2] *= 4
    mu4, sd4, e4 = o.score(o.fit(Xs, y, ells, sf2, sn2), Xcs)
    assert np.allclose(mu, mu4, atol=1e-12) and np.allclose(sd, sd4, atol=1e-12)
    # (y, sf2, sn2) -> (c y, c^2 sf2, c^2 sn2) scales mu, sigma, EI by c  (c = 2: exact in FP32)
    mu5, sd5, e5 = o.score(o.fit(X, 2 * y, ell, 4 * sf2, 4 * sn2), Xc)
    assert np.allclose(mu5, 2 * mu, rtol=1e-10, atol=1e-12)
    assert np.allclose(sd5, 2 * sd, rtol=1e-10)
    assert np.allclose(e5, 2 * e, rtol=1e-9, atol=1e-15)


def test_duplicated_data_equals_averaged_data_with_half_noise():
    X, ya, ell, sf2, _, Xc = _rand_problem(7, 10, 3, 9)
    yb = np.random.default_rng(70).normal(0, 1, 10).astype(np.float32)
    sn2 = np.float32(2.0 ** -6)
    f2 = o.fit(np.concatenate([X, X]), np.concatenate([ya, yb]), ell, sf2, sn2)
    ybar = ((ya.astype(np.float64) + yb.astype(np.float64)) / 2).astype(np.float32)
    f1 = o.fit(X, ybar, ell, sf2, sn2 / 2)
    mu2, sd2, _ = o.score(f2, Xc)
    mu1, sd1, _ = o.score(f1, Xc)
    assert np.allclose(mu2, mu1, rtol=0, atol=2e-6)     # ybar is rounded to FP32
    assert np.allclose(sd2, sd1, rtol=1e-9, atol=1e-10)


def test_variance_bounds_and_monotonicity():
    X, y, ell, sf2, sn2, Xc = _rand_problem(8, 30, 3, 200)
    f = o.fit(X, y, ell, sf2, sn2)
    _, sd, e = o.score(f, Xc)
    assert np.all(sd >= 0) and np.all(sd <= math.sqrt(float(sf2)) * (1 + 1e-15))
    assert np.all(e >= 0)
    # one more observation never increases the variance anywhere
    _, sd_less, _ = o.score(o.fit(X[:-1], y[:-1], ell, sf2, sn2), Xc)
    assert np.all(sd <= sd_less + 1e-12)


def test_library_gaussian_process_second_opinion():
    sk = pytest.importorskip("sklearn.gaussian_process")
    from sklearn.gaussian_process.kernels import ConstantKernel, Matern
    X, y, ell, sf2, sn2, Xc = _rand_problem(9, 50, 5, 40, sn2=1e-3, sf2=1.7)
    kern = ConstantKernel(float(sf2), "fixed") * Matern(length_scale=ell.astype(np.float64),
                                                       length_scale_bounds="fixed", nu=2.5)
    gpr = sk.GaussianProcessRegressor(kernel=kern, alpha=float(sn2), optimizer=None)
    gpr.fit(X.astype(np.float64), y.astype(np.float64))
    m_ref, s_ref = gpr.predict(Xc.astype(np.float64), return_std=True)
    mu, sd, _ = o.score(o.fit(X, y, ell, sf2, sn2), Xc)
    assert np.allclose(mu, m_ref, rtol=1e-8, atol=1e-10)
    assert np.allclose(sd, s_ref, rtol=1e-6, atol=1e-9)


# ------------------------------------------------------------------ step (6): top-k
def test_topk_is_truncated_lexsort_with_lower_index_winning_ties():
    rng = np.random.default_rng(20)
    e = rng.random(5000)
    e[[7, 4000, 123]] = 2.0          # planted ties at the top
    e[[9, 10]] = e[11]               # and somewhere inside
    idx, val = o.topk(e, 50)
    ref = np.lexsort((np.arange(e.size), -e))[:50]
    assert np.array_equal(idx, ref)
    assert list(idx[:3]) == [7, 123, 4000]
    assert np.array_equal(val, e[ref])
    assert np.array_equal(o.topk(e, e.size)[0], np.lexsort((np.arange(e.size), -e)))
    with pytest.raises(ValueError):
        o.topk(e, e.size + 1)


def test_batch_helpers_match_single_calls():
    X, y, ell, sf2, sn2, Xc = _rand_problem(30, 8, 2, 5)
    fits = o.fit_batch(np.stack([X, X[::-1]]), np.stack([y, y[::-1]]), np.stack([ell, ell]), sf2, sn2)
    mu, sd, e = o.score_batch(fits, np.stack([Xc, Xc]))
    assert mu.shape == (2, 5)
    assert np.allclose(mu[0], mu[1], atol=1e-12) and np.allclose(sd[0], sd[1], atol=1e-12)
