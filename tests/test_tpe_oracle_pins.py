"""Pins of the TPE oracle against things other than itself (CPU only).

The estimator's definition is this build's own (the paper names TPE in Section VII-C without a
formula), so the pins are: hand-worked examples of each rule, the mathematics every density must
satisfy, an independent library's truncated normal, and a brute-force restatement in plain loops.
"""
import json
import math
import os

import numpy as np
import pytest
from scipy import integrate, stats

from oracle import tpe_oracle as T

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "tpe_hand_worked.json")))


@pytest.mark.parametrize("case", GOLD["split"])
def test_split_hand_worked(case):
    order, n_good = T.split(np.array(case["y"]), case["gamma"])
    assert n_good == case["n_good"]
    assert order.tolist() == case["order"]


@pytest.mark.parametrize("case", GOLD["bandwidth"])
def test_bandwidth_hand_worked(case):
    mix = T.parzen(np.array(case["values"], dtype=np.float64), 1.0)
    s = len(case["values"])
    assert mix.mu.shape == (s + 1,)
    np.testing.assert_allclose(mix.mu[:s], case["values"], rtol=0, atol=0)
    assert mix.mu[s] == 0.5 and mix.sigma[s] == 1.0          # the prior
    np.testing.assert_allclose(mix.sigma[:s], case["sigma"], rtol=1e-13)
    np.testing.assert_allclose(mix.weight, np.full(s + 1, 1.0 / (s + 1)), rtol=1e-15)


def test_bandwidth_floor_is_one_hundredth_for_large_sets():
    rng = np.random.default_rng(3)
    v = rng.integers(0, 16, size=400) / 15.0          # many duplicates: zero gaps
    mix = T.parzen(v, 1.0)
    assert mix.sigma[:-1].min() == pytest.approx(0.01, rel=1e-15)
    assert mix.sigma.max() == 1.0


def test_prior_weight_enters_the_mixture_weights():
    mix = T.parzen(np.array([0.1, 0.2, 0.7]), 2.5)
    np.testing.assert_allclose(mix.weight, np.array([1, 1, 1, 2.5]) / 5.5, rtol=1e-15)


@pytest.mark.parametrize("case", GOLD["categorical"])
def test_categorical_hand_worked(case):
    mix = T.categorical(np.array(case["values"], dtype=np.float32), case["C"], case["prior_weight"])
    np.testing.assert_allclose(mix.prob, case["prob"], rtol=1e-14)
    assert mix.prob.sum() == pytest.approx(1.0, rel=1e-14)


def test_level_of_rounds_to_nearest_level():
    C = 16
    x = np.arange(C, dtype=np.float64) / (C - 1)
    assert T.level_of(x, C).tolist() == list(range(C))
    assert T.level_of(np.array([-0.2, 1.7, 0.49, 0.51]), 2).tolist() == [0, 1, 0, 1]


@pytest.mark.parametrize("seed,s", [(0, 0), (1, 1), (2, 7), (3, 60), (4, 300)])
def test_mixture_integrates_to_one(seed, s):
    rng = np.random.default_rng(seed)
    v = rng.random(s) if seed % 2 else rng.integers(0, 8, size=s) / 7.0
    mix = T.parzen(v, 1.0 + seed)
    pts = sorted(set(np.clip(mix.mu, 0, 1).tolist()))
    total, err = integrate.quad(lambda t: float(T.density(mix, np.array([t]))[0]), 0.0, 1.0, points=pts[:40],
                                limit=400, epsabs=1e-11, epsrel=1e-11)
    assert total == pytest.approx(1.0, abs=1e-8)


def test_components_are_scipy_truncated_normals():
    rng = np.random.default_rng(11)
    mix = T.parzen(rng.random(25), 0.7)
    x = np.linspace(0.0, 1.0, 101)
    ref = np.zeros_like(x)
    for mu, sg, w in zip(mix.mu, mix.sigma, mix.weight):
        ref += w * stats.truncnorm.pdf(x, (0.0 - mu) / sg, (1.0 - mu) / sg, loc=mu, scale=sg)
    np.testing.assert_allclose(T.density(mix, x), ref, rtol=1e-12)


def test_single_observation_closed_form():
    # one ordinal dimension, one observation: good = {0.3}, bad = {} (prior only)
    X = np.array([[0.3]], dtype=np.float32)
    model = T.tpe_fit(X, np.array([1.0]), [0], gamma=0.25, prior_weight=1.0)
    x = np.array([[0.1], [0.3], [0.95]], dtype=np.float32)
    got = T.tpe_score(model, x)
    x64 = x[:, 0].astype(np.float64)
    mu = float(np.float32(0.3))
    sg = 0.5                                              # gap to the prior mean 0.2 -> floor 1/2
    f_obs = stats.norm.pdf(x64, mu, sg) / (stats.norm.cdf(1, mu, sg) - stats.norm.cdf(0, mu, sg))
    f_pri = stats.norm.pdf(x64, 0.5, 1.0) / (stats.norm.cdf(1, 0.5, 1.0) - stats.norm.cdf(0, 0.5, 1.0))
    want = np.log(0.5 * f_obs + 0.5 * f_pri) - np.log(f_pri)
    np.testing.assert_allclose(got, want, rtol=1e-12)


def test_identical_sets_score_zero():
    rng = np.random.default_rng(5)
    half = np.concatenate([rng.random((6, 2)), rng.integers(0, 2, size=(6, 2)).astype(np.float64)], axis=1)
    X = np.concatenate([half, half]).astype(np.float32)
    y = np.concatenate([np.zeros(6), np.ones(6)])         # first copy good, second copy bad
    model = T.tpe_fit(X, y, [0, 0, 2, 2], gamma=0.5)
    assert model.n_good == 6
    cand = np.concatenate([rng.random((50, 2)), rng.integers(0, 2, size=(50, 2))], axis=1).astype(np.float32)
    np.testing.assert_allclose(T.tpe_score(model, cand), 0.0, atol=1e-13)


def test_score_prefers_the_good_cluster():
    rng = np.random.default_rng(9)
    good = 0.2 + 0.02 * rng.standard_normal((20, 1))
    bad = 0.8 + 0.02 * rng.standard_normal((60, 1))
    X = np.clip(np.concatenate([good, bad]), 0, 1).astype(np.float32)
    y = np.concatenate([np.zeros(20), np.ones(60)])
    model = T.tpe_fit(X, y, [0], gamma=0.25)
    s = T.tpe_score(model, np.array([[0.2], [0.8]], dtype=np.float32))
    assert s[0] > 1.0 and s[1] < -1.0


def _brute_force(X, y, levels, gamma, w0, cand):
    """The definition again in plain loops and scalars (tiny inputs only)."""
    n, d = len(X), len(X[0])
    n_good = min(max(1, math.ceil(float(np.float32(gamma)) * n)), n)   # gamma is FP32 at the boundary
    order = sorted(range(n), key=lambda i: (y[i], i))
    sets = [order[:n_good], order[n_good:]]
    out = []
    for x in cand:
        total = 0.0
        for j in range(d):
            logs = []
            for S in sets:
                vals = [float(X[i][j]) for i in S]
                if levels[j]:
                    C = levels[j]
                    lvl = lambda t: int(min(max(math.floor(float(np.float32(np.float32(t) * np.float32(C - 1)
                                                                              + np.float32(0.5)))), 0), C - 1))
                    cnt = sum(1 for t in vals if lvl(t) == lvl(x[j]))
                    logs.append(math.log((cnt + w0 / C) / (len(vals) + w0)))
                    continue
                comps = [(v, 1.0, k) for k, v in enumerate(vals)] + [(0.5, w0, len(vals))]
                srt = sorted(comps, key=lambda c: (c[0], c[2]))
                dens = 0.0
                for pos, (mu, w, k) in enumerate(srt):
                    if k == len(vals):
                        sg = 1.0
                    else:
                        gaps = []
                        if pos > 0:
                            gaps.append(mu - srt[pos - 1][0])
                        if pos < len(srt) - 1:
                            gaps.append(srt[pos + 1][0] - mu)
                        sg = min(max(max(gaps), 1.0 / min(100.0, len(vals) + 1.0)), 1.0)
                    Phi = lambda z: 0.5 * (1.0 + math.erf(z / math.sqrt(2.0)))
                    Z = Phi((1.0 - mu) / sg) - Phi((0.0 - mu) / sg)
                    t = (float(x[j]) - mu) / sg
                    dens += w * math.exp(-0.5 * t * t) / (math.sqrt(2 * math.pi) * sg * Z)
                logs.append(math.log(dens / (len(vals) + w0)))
            total += logs[0] - logs[1]
        out.append(total)
    return np.array(out)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_brute_force_tiny(seed):
    rng = np.random.default_rng(100 + seed)
    n, m = 9 + seed, 12
    levels = [0, 3, 0, 2]
    cols = [rng.integers(0, 5, size=n) / 4.0, rng.integers(0, 3, size=n) / 2.0, rng.random(n),
            rng.integers(0, 2, size=n).astype(float)]
    X = np.stack(cols, axis=1).astype(np.float32)
    y = rng.integers(0, 4, size=n).astype(np.float64)      # ties in y
    cand = np.stack([rng.integers(0, 5, size=m) / 4.0, rng.integers(0, 3, size=m) / 2.0, rng.random(m),
                     rng.integers(0, 2, size=m).astype(float)], axis=1).astype(np.float32)
    model = T.tpe_fit(X, y, levels, gamma=0.3, prior_weight=1.5)
    np.testing.assert_allclose(T.tpe_score(model, cand), _brute_force(X, y, levels, 0.3, 1.5, cand), rtol=1e-11,
                               atol=1e-12)


def test_grid_dimension_equals_the_mixture_on_grid_and_snaps_off_grid():
    rng = np.random.default_rng(21)
    L = 16
    X = (rng.integers(0, L, size=(40, 1)) / (L - 1)).astype(np.float32)
    y = rng.normal(size=40)
    cont = T.tpe_fit(X, y, [0], gamma=0.25)
    grid = T.tpe_fit(X, y, [-L], gamma=0.25)
    on = (np.arange(L) / (L - 1)).astype(np.float32)[:, None]
    np.testing.assert_array_equal(T.tpe_score(grid, on), T.tpe_score(cont, on))      # on the grid: identical
    off = (on + np.float32(0.3 / (L - 1))).astype(np.float32)                          # nearer to the same level
    np.testing.assert_array_equal(T.tpe_score(grid, off), T.tpe_score(cont, on))
    assert np.abs(T.tpe_score(cont, off) - T.tpe_score(cont, on)).max() > 1e-3         # the mixture itself differs there


def test_topk_ties_take_the_lower_index():
    s = np.array([0.5, 2.0, 2.0, -1.0, 2.0, 0.5])
    assert T.tpe_topk(s, 4).tolist() == [1, 2, 4, 0]
