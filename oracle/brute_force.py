"""Explicit-inverse GP posterior for tiny problems (n <= 16).

TEST INFRASTRUCTURE ONLY.  A second, independent statement of the posterior used
to pin ``r3_oracle.c``: it shares nothing with it -- no Cholesky, no
substitution, not even the same kernel routine.  Everything is pure Python floats, with the inverse taken by Gauss-Jordan elimination
with partial pivoting, and the normal CDF by ``math.erf``:

    mu      = k*^T K^-1 y
    sigma^2 = sf2 - k*^T K^-1 k*
    EI      = sigma * (z Phi(z) + phi(z)),  z = (min y - mu)/sigma
"""
from __future__ import annotations

import math


def _k52(x, z, ell, sf2):
    r = math.sqrt(sum(((float(a) - float(b)) / float(l)) ** 2 for a, b, l in zip(x, z, ell)))
    s = math.sqrt(5.0) * r
    return sf2 * (1.0 + s + s * s / 3.0) * math.exp(-s)


def _inverse(A):
    n = len(A)
    M = [list(map(float, A[i])) + [1.0 if i == j else 0.0 for j in range(n)] for i in range(n)]
    for c in range(n):
        p = max(range(c, n), key=lambda r: abs(M[r][c]))
        if M[p][c] == 0.0:
            raise ArithmeticError("singular matrix")
        M[c], M[p] = M[p], M[c]
        piv = M[c][c]
        M[c] = [v / piv for v in M[c]]
        for r in range(n):
            if r != c and M[r][c] != 0.0:
                f = M[r][c]
                M[r] = [a - f * b for a, b in zip(M[r], M[c])]
    return [row[n:] for row in M]


def posterior(X, y, ell, sf2, sn2, Xcand):
    """Return lists (mu, sigma, ei) for every row of Xcand; n <= 16 only."""
    n = len(X)
    if n > 16:
        raise ValueError("brute force is for n <= 16")
    sf2 = float(sf2)
    sn2 = float(sn2)
    K = [[_k52(X[i], X[j], ell, sf2) + (sn2 if i == j else 0.0) for j in range(n)] for i in range(n)]
    Kinv = _inverse(K)
    yv = [float(v) for v in y]
    best = min(yv)
    Kinv_y = [sum(Kinv[i][j] * yv[j] for j in range(n)) for i in range(n)]
    mus, sigmas, eis = [], [], []
    for xs in Xcand:
        ks = [_k52(X[i], xs, ell, sf2) for i in range(n)]
        mu = sum(ks[i] * Kinv_y[i] for i in range(n))
        quad = sum(ks[i] * Kinv[i][j] * ks[j] for i in range(n) for j in range(n))
        var = max(sf2 - quad, 0.0)
        sd = math.sqrt(var)
        if sd > 0.0:
            z = (best - mu) / sd
            Phi = 0.5 * (1.0 + math.erf(z / math.sqrt(2.0)))
            phi = math.exp(-0.5 * z * z) / math.sqrt(2.0 * math.pi)
            e = sd * (z * Phi + phi)
        else:
            e = max(best - mu, 0.0)
        mus.append(mu)
        sigmas.append(sd)
        eis.append(e)
    return mus, sigmas, eis
