"""Pins of the oracle's greedy batch proposal (fantasies) against things other than itself (CPU only).

The rule itself is a reading (the paper only says that the search is "parallel"); what can be pinned
is that the oracle's loop does what the rule says: against an independent explicit-inverse posterior
in plain Python on tiny problems, against the single-point selection for q = 1, and against the
identities that conditioning on a fantasised value must satisfy.
"""
import math

import numpy as np
import pytest

from oracle import brute_force as bf
from oracle import gp_oracle as o


def problem(seed, n, d, m):
    rng = np.random.default_rng(seed)
    X = rng.uniform(0, 1, (n, d)).astype(np.float32)
    y = rng.normal(0, 1, n).astype(np.float32)
    ell = rng.uniform(0.3, 1.0, d).astype(np.float32)
    Xc = rng.uniform(0, 1, (m, d)).astype(np.float32)
    return X, y, ell, np.float32(1.3), np.float32(1e-2), Xc


def ei_fixed_incumbent(mu, sd, best):
    if sd > 0.0:
        z = (best - mu) / sd
        return sd * (z * 0.5 * (1.0 + math.erf(z / math.sqrt(2.0))) + math.exp(-0.5 * z * z) / math.sqrt(2 * math.pi))
    return max(best - mu, 0.0)


def brute_force_propose(X, y, ell, sf2, sn2, Xc, q, lie):
    Xa = [list(map(float, r)) for r in X]
    ya = [float(v) for v in y]
    best0 = min(ya)
    picked, vals = [], []
    for _ in range(q):
        mus, sds, _ = bf.posterior(Xa, ya, ell, float(sf2), float(sn2), Xc)
        e = [ei_fixed_incumbent(mu, sd, best0) for mu, sd in zip(mus, sds)]
        cand = [i for i in range(len(Xc)) if i not in picked]
        j = max(cand, key=lambda i: (e[i], -i))
        picked.append(j)
        vals.append(e[j])
        Xa.append(list(map(float, Xc[j])))
        ya.append(float(np.float32(mus[j] if lie == "believer" else best0)))
    return picked, vals


@pytest.mark.parametrize("seed,lie", [(0, "believer"), (1, "believer"), (2, "liar"), (3, "liar")])
def test_against_explicit_inverse_brute_force(seed, lie):
    X, y, ell, sf2, sn2, Xc = problem(seed, 8, 2, 30)
    idx, val = o.propose(X, y, ell, sf2, sn2, Xc, 5, lie)
    ridx, rval = brute_force_propose(X, y, ell, sf2, sn2, Xc, 5, lie)
    assert idx.tolist() == ridx
    np.testing.assert_allclose(val, rval, rtol=1e-7, atol=1e-12)


def test_single_pick_is_the_top_candidate():
    X, y, ell, sf2, sn2, Xc = problem(7, 40, 4, 500)
    f = o.fit(X, y, ell, sf2, sn2)
    _, _, e = o.score(f, Xc)
    idx, val = o.propose(X, y, ell, sf2, sn2, Xc, 1)
    tidx, tval = o.topk(e, 1)
    assert idx[0] == tidx[0] and val[0] == tval[0]


def test_picks_are_distinct_and_first_pick_does_not_depend_on_the_lie():
    X, y, ell, sf2, sn2, Xc = problem(11, 30, 3, 200)
    a, _ = o.propose(X, y, ell, sf2, sn2, Xc, 12, "believer")
    b, _ = o.propose(X, y, ell, sf2, sn2, Xc, 12, "liar")
    assert len(set(a.tolist())) == 12 and len(set(b.tolist())) == 12
    assert a[0] == b[0]


def test_believer_keeps_the_mean_and_shrinks_variance_and_ei():
    """Conditioning on the posterior mean changes no mean; variances and (fixed incumbent) EI only drop.
    This is what lets an implementation shortlist candidates by their initial EI."""
    X, y, ell, sf2, sn2, Xc = problem(13, 50, 3, 400)
    f0 = o.fit(X, y, ell, sf2, sn2)
    mu0, sd0, e0 = o.score(f0, Xc)
    j = int(np.argmax(e0))
    Xa = np.concatenate([X, Xc[j:j + 1]])
    ya = np.concatenate([y, np.array([mu0[j]], dtype=np.float32)])
    f1 = o.fit(Xa, ya, ell, sf2, sn2)
    mu1, sd1, e1 = o.score(f1, Xc, best=f0.best)
    # the fantasised value is rounded to FP32, hence 1e-7 instead of exact
    np.testing.assert_allclose(mu1, mu0, atol=3e-7 * max(1.0, np.abs(mu0).max()))
    assert np.all(sd1 <= sd0 + 1e-12)
    assert np.all(e1 <= e0 + 1e-9)
    # the rank-one formulas: sigma1^2 = sigma0^2 - c^2 / (sigma0_j^2 + noise)
    fj = o.fit(np.concatenate([X, Xc[j:j + 1]]), np.concatenate([y, [0.0]]).astype(np.float32), ell, sf2, sn2)
    assert sd1[j] ** 2 == pytest.approx(sd0[j] ** 2 * float(sn2) / (sd0[j] ** 2 + float(sn2)), rel=1e-8)
    assert np.allclose(o.score(fj, Xc, best=0.0)[1], sd1, rtol=1e-12)     # variances do not depend on y


def test_liar_uses_the_incumbent_as_value():
    X, y, ell, sf2, sn2, Xc = problem(17, 20, 2, 100)
    idx, _ = o.propose(X, y, ell, sf2, sn2, Xc, 2, "liar")
    f0 = o.fit(X, y, ell, sf2, sn2)
    Xa = np.concatenate([X, Xc[idx[0]:idx[0] + 1]])
    ya = np.concatenate([y, np.array([y.min()], dtype=np.float32)])
    _, _, e = o.score(o.fit(Xa, ya, ell, sf2, sn2), Xc, best=f0.best)
    e[idx[0]] = -np.inf
    assert int(np.argmax(e)) == idx[1]
