"""Writes ``closed_forms.json``: 40-digit evaluations of the closed forms that pin the CPU oracle.

Uses mpmath only -- neither the oracle nor the CUDA library is imported -- so the
stored values are independent of both.  Every entry is a direct consequence of
the textbook definitions (zero-mean GP posterior, ARD Matern-5/2 covariance,
Expected Improvement for minimisation); the paper prints no worked example.

    python tests/golden/make_closed_forms.py
"""
import json
import os

import mpmath as mp

mp.mp.dps = 40


def m52(s):
    s = mp.mpf(s)
    return (1 + s + s * s / 3) * mp.e ** (-s)


def h(z):
    z = mp.mpf(z)
    return z * mp.ncdf(z) + mp.npdf(z)


def kern(x, z, ell, sf2):
    r2 = sum(((mp.mpf(a) - mp.mpf(b)) / mp.mpf(l)) ** 2 for a, b, l in zip(x, z, ell))
    return mp.mpf(sf2) * m52(mp.sqrt(5) * mp.sqrt(r2))


def posterior(X, y, ell, sf2, sn2, xs):
    n = len(X)
    K = mp.matrix(n, n)
    for i in range(n):
        for j in range(n):
            K[i, j] = kern(X[i], X[j], ell, sf2) + (mp.mpf(sn2) if i == j else 0)
    Kinv = K ** -1
    yv = mp.matrix([mp.mpf(v) for v in y])
    ks = mp.matrix([kern(X[i], xs, ell, sf2) for i in range(n)])
    alpha = Kinv * yv
    mu = (ks.T * alpha)[0]
    var = mp.mpf(sf2) - (ks.T * Kinv * ks)[0]
    sd = mp.sqrt(var)
    best = min(mp.mpf(v) for v in y)
    ei = sd * h((best - mu) / sd)
    return K, alpha, ks, mu, sd, ei


def f(v):
    return mp.nstr(v, 25)


out = {
    "_source": "closed forms evaluated with mpmath at 40 digits; see make_closed_forms.py",
    "matern52_of_s": {str(s): f(m52(s)) for s in ("0", "0.5", "1", "2", "5", "10", "20")},
    "h_of_z": {str(z): f(h(z)) for z in ("0", "1", "-1", "-2", "-3", "-4", "-6")},
}

# one observation, one feature: x1 = 0, y1 = 1, ell = 1, sf2 = 1, sn2 = 0.1, x* = 1/sqrt(5)
xs = 1 / mp.sqrt(5)
ks = m52(1)
out["n1"] = {
    "X": [[0.0]], "y": [1.0], "ell": [1.0], "sf2": 1.0, "sn2": 0.1, "xstar_is": "1/sqrt(5)",
    "kstar": f(ks), "mu": f(ks / mp.mpf("1.1")), "var": f(1 - ks * ks / mp.mpf("1.1")),
    "sigma": f(mp.sqrt(1 - ks * ks / mp.mpf("1.1"))),
}

# three observations, two ARD features
X = [["0", "0"], ["1", "0"], ["0.5", "1"]]
y = ["0.3", "-0.7", "0.4"]
ell = ["0.5", "2"]
sf2, sn2 = "1.5", "0.01"
case = {"X": [[float(a) for a in r] for r in X], "y": [float(v) for v in y],
        "ell": [float(v) for v in ell], "sf2": float(sf2), "sn2": float(sn2), "points": []}
for xs in (["0.25", "0.5"], ["1", "0"], ["10", "10"]):
    K, alpha, ks, mu, sd, ei = posterior(X, y, ell, sf2, sn2, xs)
    case["points"].append({"xstar": [float(v) for v in xs], "kstar": [f(v) for v in ks],
                           "mu": f(mu), "sigma": f(sd), "ei": f(ei)})
case["K"] = [[f(K[i, j]) for j in range(3)] for i in range(3)]
case["alpha"] = [f(v) for v in alpha]
out["n3_ard"] = case

path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "closed_forms.json")
with open(path, "w") as fh:
    json.dump(out, fh, indent=1)
print("wrote", path)
