"""FP64 CPU oracle of Tree-structured-Parzen-Estimator candidate scoring.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA package never imports this module and
this module never imports the CUDA package.

Where this sits in the paper.  Section VII-C states that the replay server tunes
pass order and launch parameters with parallel Tree Parzen Estimation for 30
iterations; it gives no formula, quantile, bandwidth rule or prior.  The
definition below is therefore THIS BUILD'S OWN statement of the estimator (the
usual one: split the history at a quantile of y, one Parzen mixture per
dimension for each side, score = log-density ratio); every free choice is
listed here and each function says which step it is.

Definition (features are normalised to [0, 1]; smaller y is better):

  (T1) split      n_good = min(max(1, ceil(gamma * n)), n), with gamma first rounded
                  to FP32 (the type it has at the library's boundary) and the
                  product taken in FP64.  Sort the history by y ascending, ties by
                  lower index; the first n_good observations are the "good" set,
                  the rest the "bad" set (possibly empty).
  (T2) ordinal / continuous dimension (levels == 0), for one set with values
                  p_1..p_s: the mixture has s + 1 components -- one per value
                  (weight 1, mean p_i) and a prior (weight prior_weight, mean
                  1/2, sigma 1).  Sort the s + 1 means ascending; a value's
                  sigma is the larger of the gaps to its neighbours in that
                  order (the only gap at either end), clipped to
                  [1 / min(100, s + 1), 1].  Each component is a normal density
                  truncated to [0, 1]:
                     f_c(x) = phi((x - mu_c)/sigma_c) / (sigma_c * Z_c),
                     Z_c = Phi((1 - mu_c)/sigma_c) - Phi((0 - mu_c)/sigma_c),
                  and the density is sum_c w_c f_c(x) / sum_c w_c.
  (T3) categorical dimension (levels == C >= 2): the level of x is
                  v = clamp(floor(x * (C - 1) + 1/2), 0, C - 1), that product and
                  sum taken in FP32 (the precision the device decides it in);
                  P(v) = (count_v + prior_weight / C) / (s + prior_weight).
  (T3g) ordinal dimension on a known grid (levels == -L, 2 <= L <= 64: the admissible
                  values are v/(L-1), v = 0..L-1, as for block sizes, unroll factors
                  or sixteen-level features): the mixture is (T2)'s, and a candidate is
                  evaluated at its nearest grid value -- level v as in (T3), value
                  v/(L-1) taken in FP64 and rounded to FP32, which is the FP32 number an
                  on-grid candidate holds.  For candidates on the grid this IS (T2); it
                  lets an implementation tabulate the L densities once.
  (T4) score      sum over dimensions of ln l_j(x_j) - ln g_j(x_j), l from the
                  good set and g from the bad set.  A larger score is a better
                  candidate (the ratio l/g is monotone in Expected Improvement
                  under the estimator's model).

Parity unpinned against the paper: it prints no formula or worked example for
this estimator, so the pins below tie the oracle to its stated definition and to
the mathematics only.

Pins (tests/test_tpe_oracle_pins.py): every mixture integrates to 1 over [0, 1]
by adaptive quadrature; the components equal SciPy's truncated normal; a
hand-worked split, bandwidth and clipping example; categorical probabilities
against counts done by hand; identical good and bad sets give score 0; a
pure-Python brute-force restatement on tiny inputs.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

_SQRT_2PI = math.sqrt(2.0 * math.pi)


def _Phi(z: float) -> float:
    return 0.5 * math.erfc(-z / math.sqrt(2.0))


@dataclass
class Mixture:
    """Parzen mixture of one dimension and one set (T2), or a probability table (T3)."""
    levels: int
    grid: int = 0                # (T3g): evaluate at the nearest of `grid` equally spaced values
    mu: np.ndarray = field(default_factory=lambda: np.zeros(0))      # [s + 1] component means, prior last
    sigma: np.ndarray = field(default_factory=lambda: np.zeros(0))   # [s + 1]
    weight: np.ndarray = field(default_factory=lambda: np.zeros(0))  # [s + 1], normalised to sum 1
    Z: np.ndarray = field(default_factory=lambda: np.zeros(0))       # [s + 1] truncation mass
    prob: np.ndarray = field(default_factory=lambda: np.zeros(0))    # [C] for a categorical dimension


@dataclass
class TpeModel:
    n: int
    d: int
    n_good: int
    order: np.ndarray            # [n] history indices by y ascending (ties: lower index)
    levels: np.ndarray           # [d]
    good: list                   # [d] Mixture
    bad: list                    # [d] Mixture


def split(y: np.ndarray, gamma: float):
    """(T1): the order of the history and the size of the good set."""
    y = np.asarray(y, dtype=np.float64)
    n = y.shape[0]
    n_good = min(max(1, int(math.ceil(float(np.float32(gamma)) * n))), n)
    order = np.argsort(y, kind="stable")
    return order, n_good


def parzen(values: np.ndarray, prior_weight: float) -> Mixture:
    """(T2): the truncated-normal mixture of one set's values in one dimension."""
    p = np.asarray(values, dtype=np.float64)
    s = p.shape[0]
    means = np.concatenate([p, [0.5]])
    is_prior = np.zeros(s + 1, dtype=bool)
    is_prior[s] = True
    srt = np.argsort(means, kind="stable")
    sm = means[srt]
    sig_sorted = np.ones(s + 1)
    if s >= 1:
        gaps = np.diff(sm)                       # gaps[t] = sm[t+1] - sm[t]
        for t in range(s + 1):
            left = gaps[t - 1] if t > 0 else -np.inf
            right = gaps[t] if t < s else -np.inf
            sig_sorted[t] = max(left, right)
        lo = 1.0 / min(100.0, s + 1.0)
        sig_sorted = np.clip(sig_sorted, lo, 1.0)
    sigma = np.empty(s + 1)
    sigma[srt] = sig_sorted
    sigma[is_prior] = 1.0
    w = np.ones(s + 1)
    w[s] = prior_weight
    w = w / w.sum()
    Z = np.array([_Phi((1.0 - means[c]) / sigma[c]) - _Phi((0.0 - means[c]) / sigma[c]) for c in range(s + 1)])
    return Mixture(levels=0, mu=means, sigma=sigma, weight=w, Z=Z)


def level_of(x: np.ndarray, C: int) -> np.ndarray:
    """(T3): categorical level of a normalised feature, decided in FP32."""
    x32 = np.asarray(x, dtype=np.float32)
    v = np.floor(x32 * np.float32(C - 1) + np.float32(0.5))
    return np.clip(v, 0, C - 1).astype(np.int64)


def categorical(values: np.ndarray, C: int, prior_weight: float) -> Mixture:
    """(T3): smoothed level frequencies of one set's values in one dimension."""
    s = values.shape[0]
    counts = np.bincount(level_of(values, C), minlength=C).astype(np.float64)
    prob = (counts + prior_weight / C) / (s + prior_weight)
    return Mixture(levels=C, prob=prob)


def tpe_fit(X: np.ndarray, y: np.ndarray, levels, gamma: float = 0.25, prior_weight: float = 1.0) -> TpeModel:
    """(T1)-(T3) for every dimension and both sets."""
    X = np.asarray(X)
    n, d = X.shape
    levels = np.asarray(levels, dtype=np.int64)
    if not (0.0 < gamma <= 1.0) or not prior_weight > 0.0:
        raise ValueError("gamma in (0, 1], prior_weight > 0")
    order, n_good = split(y, gamma)
    gi, bi = order[:n_good], order[n_good:]
    good, bad = [], []
    for j in range(d):
        col = X[:, j]
        if levels[j] <= 0:
            good.append(parzen(col[gi], prior_weight))
            bad.append(parzen(col[bi], prior_weight))
            good[-1].grid = bad[-1].grid = int(-levels[j])
        else:
            good.append(categorical(col[gi], int(levels[j]), prior_weight))
            bad.append(categorical(col[bi], int(levels[j]), prior_weight))
    return TpeModel(n=n, d=d, n_good=n_good, order=order, levels=levels, good=good, bad=bad)


def density(mix: Mixture, x: np.ndarray) -> np.ndarray:
    """Value of one dimension's mixture (T2) or level probability (T3) at the points x."""
    if mix.levels:
        return mix.prob[level_of(x, mix.levels)]
    if mix.grid:
        L = mix.grid
        x = (level_of(x, L).astype(np.float64) / (L - 1)).astype(np.float32)
    x = np.asarray(x, dtype=np.float64)[:, None]
    t = (x - mix.mu[None, :]) / mix.sigma[None, :]
    comp = np.exp(-0.5 * t * t) / (_SQRT_2PI * mix.sigma[None, :] * mix.Z[None, :])
    return comp @ mix.weight


def tpe_score(model: TpeModel, Xcand: np.ndarray, block: int = 2048) -> np.ndarray:
    """(T4): log-density ratio of every candidate, FP64."""
    Xc = np.asarray(Xcand)
    m = Xc.shape[0]
    out = np.zeros(m)
    for b0 in range(0, m, block):
        xb = Xc[b0:b0 + block]
        acc = np.zeros(xb.shape[0])
        for j in range(model.d):
            acc += np.log(density(model.good[j], xb[:, j])) - np.log(density(model.bad[j], xb[:, j]))
        out[b0:b0 + block] = acc
    return out


def tpe_topk(score: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest scores, ties by lower index."""
    order = np.lexsort((np.arange(score.shape[0]), -score))
    return order[:k]
