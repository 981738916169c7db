"""ctypes front end of the FP64 CPU oracle (``r3_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA package never imports this module and
this module never imports the CUDA package.

The arithmetic lives in ``r3_oracle.c`` (steps (1)-(6) of its header); this file
only builds the shared object with gcc, marshals numpy arrays and loops over the
GPs of a batch.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "r3_oracle.c")
_LIB = os.path.join(_HERE, "libr3_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile ``r3_oracle.c`` into ``libr3_oracle.so`` beside it (gcc, OpenMP)."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O3", "-march=x86-64-v3", "-fopenmp", "-fPIC", "-shared", "-std=c11",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True, capture_output=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is not None:
            return _lib
        build()
        try:
            lib = ctypes.CDLL(_LIB)
        except OSError:
            build(force=True)
            lib = ctypes.CDLL(_LIB)
        c_fp = ctypes.POINTER(ctypes.c_float)
        c_dp = ctypes.POINTER(ctypes.c_double)
        c_lp = ctypes.POINTER(ctypes.c_longlong)
        lib.r3o_matern52.restype = ctypes.c_double
        lib.r3o_matern52.argtypes = [ctypes.c_double]
        lib.r3o_kernel.restype = ctypes.c_double
        lib.r3o_kernel.argtypes = [c_fp, c_fp, c_fp, ctypes.c_int, ctypes.c_double]
        lib.r3o_gram.restype = None
        lib.r3o_gram.argtypes = [c_fp, c_fp, ctypes.c_double, ctypes.c_double, ctypes.c_int,
                                 ctypes.c_int, c_dp]
        lib.r3o_cholesky.restype = ctypes.c_int
        lib.r3o_cholesky.argtypes = [c_dp, ctypes.c_int]
        lib.r3o_alpha.restype = None
        lib.r3o_alpha.argtypes = [c_dp, c_fp, ctypes.c_int, c_dp]
        lib.r3o_fit.restype = ctypes.c_int
        lib.r3o_fit.argtypes = [c_fp, c_fp, c_fp, ctypes.c_double, ctypes.c_double, ctypes.c_int,
                                ctypes.c_int, c_dp, c_dp, c_dp]
        lib.r3o_ei.restype = ctypes.c_double
        lib.r3o_ei.argtypes = [ctypes.c_double] * 3
        lib.r3o_score.restype = None
        lib.r3o_score.argtypes = [c_fp, c_dp, c_dp, ctypes.c_double, c_fp, ctypes.c_double,
                                  ctypes.c_int, ctypes.c_int, c_fp, ctypes.c_longlong, c_dp, c_dp, c_dp]
        lib.r3o_topk.restype = ctypes.c_int
        lib.r3o_topk.argtypes = [c_dp, ctypes.c_longlong, ctypes.c_int, c_lp, c_dp]
        lib.r3o_threads.restype = ctypes.c_int
        lib.r3o_threads.argtypes = []
        _lib = lib
        return lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _fp(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def _dp(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


class NotPositiveDefinite(ArithmeticError):
    """A Cholesky pivot was not a positive finite number (step (2))."""


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().r3o_threads())


def matern52(r2: float) -> float:
    """Step (1): (1 + s + s^2/3) exp(-s) with s = sqrt(5 r2)."""
    return float(_load().r3o_matern52(float(r2)))


def kernel(x, z, ell, sf2: float) -> float:
    """Step (1): ARD Matern-5/2 covariance of two feature rows."""
    x, z, ell = _f32(x), _f32(z), _f32(ell)
    return float(_load().r3o_kernel(_fp(x), _fp(z), _fp(ell), x.shape[0], float(sf2)))


def gram(X, ell, sf2: float, sn2: float) -> np.ndarray:
    """Step (2): K(X,X) + sn2*I, FP64 [n][n]."""
    X, ell = _f32(X), _f32(ell)
    n, d = X.shape
    K = np.empty((n, n), dtype=np.float64)
    _load().r3o_gram(_fp(X), _fp(ell), float(sf2), float(sn2), n, d, _dp(K))
    return K


def cholesky(K: np.ndarray) -> np.ndarray:
    """Step (2): lower Cholesky factor of an FP64 matrix (copy)."""
    L = np.array(K, dtype=np.float64, order="C", copy=True)
    st = _load().r3o_cholesky(_dp(L), L.shape[0])
    if st:
        raise NotPositiveDefinite(f"pivot {st - 1} is not positive")
    return L


def ei(mu: float, sigma: float, best: float) -> float:
    """Step (5): closed-form Expected Improvement (minimisation)."""
    return float(_load().r3o_ei(float(mu), float(sigma), float(best)))


@dataclass
class Fit:
    """Everything step (4) needs for one GP; all FP64 except the FP32 inputs."""
    X: np.ndarray       # [n][d] float32, as given
    ell: np.ndarray     # [d] float32, as given
    sf2: float
    sn2: float
    L: np.ndarray       # [n][n] float64 lower
    alpha: np.ndarray   # [n] float64
    best: float


def fit(X, y, ell, sf2: float, sn2: float) -> Fit:
    """Steps (2)-(3) for one GP."""
    X, y, ell = _f32(X), _f32(y), _f32(ell)
    n, d = X.shape
    if y.shape != (n,) or ell.shape != (d,):
        raise ValueError("shape mismatch")
    # the C-ABI takes the hyper-parameters as FP32: widen exactly those values
    sf2 = float(np.float32(sf2))
    sn2 = float(np.float32(sn2))
    L = np.empty((n, n), dtype=np.float64)
    alpha = np.empty(n, dtype=np.float64)
    best = ctypes.c_double(0.0)
    st = _load().r3o_fit(_fp(X), _fp(y), _fp(ell), sf2, sn2, n, d, _dp(L), _dp(alpha),
                         ctypes.byref(best))
    if st == -1:
        raise ValueError("non-finite input")
    if st:
        raise NotPositiveDefinite(f"pivot {st - 1} is not positive")
    return Fit(X, ell, sf2, sn2, L, alpha, float(best.value))


def score(f: Fit, Xcand, best: float | None = None):
    """Steps (4)-(5): (mu, sigma, EI), each FP64 [m]."""
    Xcand = _f32(Xcand)
    m, d = Xcand.shape
    if d != f.X.shape[1]:
        raise ValueError("feature dimension mismatch")
    mu = np.empty(m, dtype=np.float64)
    sigma = np.empty(m, dtype=np.float64)
    e = np.empty(m, dtype=np.float64)
    b = f.best if best is None else float(best)
    _load().r3o_score(_fp(f.X), _dp(f.L), _dp(f.alpha), b, _fp(f.ell), f.sf2, f.X.shape[0], d,
                      _fp(Xcand), m, _dp(mu), _dp(sigma), _dp(e))
    return mu, sigma, e


def topk(ei_values, k: int):
    """Step (6): indices (int64 [k]) and values of the k largest EI, ties to the lower index."""
    e = np.ascontiguousarray(ei_values, dtype=np.float64)
    idx = np.empty(k, dtype=np.int64)
    val = np.empty(k, dtype=np.float64)
    st = _load().r3o_topk(_dp(e), e.shape[0], int(k),
                          idx.ctypes.data_as(ctypes.POINTER(ctypes.c_longlong)), _dp(val))
    if st:
        raise ValueError("invalid k")
    return idx, val


def propose(X, y, ell, sf2: float, sn2: float, Xcand, q: int, lie: str = "believer"):
    """Greedy batch of q distinct pool members by fantasies ("parallel" BO, Section IV: several points of one
    search are replayed at once).  The paper gives no rule for choosing them; this is the usual sequential one,
    written as its definition:

      repeat q times:  fit the (augmented) history; score the pool with the incumbent fixed at the best
      OBSERVED value; pick the not-yet-picked candidate of largest EI (ties: lower index); append it to the
      history with a fantasised value -- its posterior mean ("believer") or the incumbent ("liar") -- rounded
      to FP32 like any observation.

    Returns (indices int64 [q], EI of each pick at the time it was picked, FP64 [q]).
    """
    if lie not in ("believer", "liar"):
        raise ValueError("lie must be 'believer' or 'liar'")
    Xa, ya, Xcand = _f32(X).copy(), _f32(y).copy(), _f32(Xcand)
    best0 = float(ya.min())
    picked, values = [], []
    for _ in range(q):
        f = fit(Xa, ya, ell, sf2, sn2)
        mu, _, e = score(f, Xcand, best=best0)
        e = e.copy()
        e[picked] = -np.inf
        j = int(np.argmax(e))          # first maximum: the lower index wins ties
        picked.append(j)
        values.append(float(e[j]))
        value = mu[j] if lie == "believer" else best0
        Xa = np.concatenate([Xa, Xcand[j:j + 1]])
        ya = np.concatenate([ya, np.array([value], dtype=np.float32)])
    return np.array(picked, dtype=np.int64), np.array(values)


def lml(X, y, ell, sf2: float, sn2: float):
    """Log marginal likelihood of the history and its gradient with respect to the LOGARITHMS of the
    hyper-parameters, in the order (log ell_1 .. log ell_d, log sf2, log sn2) -- what a hyper-parameter fit of
    the surrogate maximises (the paper passes no rule; this is the textbook evidence of a zero-mean GP):

        K = Kf + sn2 I,  alpha = K^-1 y,
        lml = -1/2 y.alpha - 1/2 log|K| - n/2 log(2 pi),
        d lml / d theta = 1/2 trace((alpha alpha^T - K^-1) dK/dtheta),
        dK/dlog ell_j = sf2 exp(-s) (5/3)(1 + s) u_j^2   (u_j = (x_j - z_j)/ell_j, s = sqrt(5 sum u^2)),
        dK/dlog sf2 = Kf,   dK/dlog sn2 = sn2 I.

    Plain numpy FP64 with LAPACK's Cholesky and inverse as steps; n^2 d memory, so for test sizes only.
    Returns (lml, gradient [d + 2]).
    """
    X, y, ell = _f32(X).astype(np.float64), _f32(y).astype(np.float64), _f32(ell).astype(np.float64)
    sf2, sn2 = float(np.float32(sf2)), float(np.float32(sn2))
    n, d = X.shape
    U = (X[:, None, :] - X[None, :, :]) / ell[None, None, :]
    s = np.sqrt(5.0 * (U * U).sum(axis=2))
    e = np.exp(-s)
    Kf = sf2 * (1.0 + s + s * s / 3.0) * e
    K = Kf + sn2 * np.eye(n)
    L = np.linalg.cholesky(K)
    alpha = np.linalg.solve(L.T, np.linalg.solve(L, y))
    value = -0.5 * float(y @ alpha) - float(np.log(np.diag(L)).sum()) - 0.5 * n * np.log(2.0 * np.pi)
    M = np.outer(alpha, alpha) - np.linalg.inv(K)
    G = sf2 * e * (5.0 / 3.0) * (1.0 + s)
    grad = np.empty(d + 2)
    for j in range(d):
        grad[j] = 0.5 * float((M * G * U[:, :, j] ** 2).sum())
    grad[d] = 0.5 * float((M * Kf).sum())
    grad[d + 1] = 0.5 * sn2 * float(np.trace(M))
    return value, grad


def fit_batch(X, y, ell, sf2, sn2):
    """Steps (2)-(3) for [batch] independent GPs; returns a list of Fit."""
    X, y, ell = _f32(X), _f32(y), _f32(ell)
    sf2 = np.broadcast_to(np.asarray(sf2, dtype=np.float32), (X.shape[0],))
    sn2 = np.broadcast_to(np.asarray(sn2, dtype=np.float32), (X.shape[0],))
    return [fit(X[g], y[g], ell[g], sf2[g], sn2[g]) for g in range(X.shape[0])]


def score_batch(fits, Xcand):
    """Steps (4)-(5) for a batch: Xcand [batch][m][d] -> three FP64 [batch][m] arrays."""
    out = [score(f, Xcand[g]) for g, f in enumerate(fits)]
    return tuple(np.stack([o[i] for o in out]) for i in range(3))
