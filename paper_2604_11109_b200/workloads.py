"""Seeded synthetic tuning histories and candidate pools.

This module serves both the CUDA library's tests/benchmark and the CPU oracle's
tests.  It holds none of the method's arithmetic (no covariance, no posterior,
no acquisition): it only draws feature rows, a synthetic log-runtime response
and hyper-parameters.

The rows stand in for the search points of the paper's inner Bayesian
optimisation loop (Section V-B: a point is a compiler pipeline plus a launch
configuration, its value the replayed runtime; Section IV: runtimes are means of
several replays, hence small observation noise).  The paper publishes no tuning
histories, so five seeded workloads of the sizes named by the build contract
are generated instead:

  cfg 1  single GP, d=6 launch parameters, n=64,   m=4096,      k=8
  cfg 2  single GP, d=16 (+10 binary flags), n=256, m=262144,   k=32
  cfg 3  64 GPs,    d=32 (+26 binary),       n=512, m=65536 each, k=16
  cfg 4  pass ordering, d=128 one-hot,       n=1024, m=1048576, k=64
  cfg 5  large history, d=64 mixed,          n=4096, m=1048576, k=128

Feature encodings (all in [0, 1]):
  block size {32,64,..,1024} -> (v-32)/992; grid multiplier {1..8} -> (v-1)/7;
  unroll {1,2,4,8} -> log2(v)/3; maxrregcount {32..255} -> (v-32)/223;
  shared-memory carve-out {0,25,50,100}% -> v/100; booleans -> 0/1;
  cfg 5: 32 integer features with 16 levels (v/15) + 32 booleans;
  cfg 4: a candidate is a permutation of 32 passes; feature[4p + pos(p)//8]
  = 1/sqrt(32), so every row has unit L2 norm.

Response: three seeded sinusoids + a quadratic bowl (scaled by 6/d for d > 6)
+ for d >= 16 ten seeded pairwise products (weight 0.1) + Gaussian noise whose
standard deviation is sqrt(noise_var); cfg 4 instead sums seeded pass-pair
precedence rewards.  y is then standardised (zero mean, unit variance), as a
BO driver would do before fitting a zero-mean GP with signal variance 1.

Pools are iid uniform over the grid and made of distinct rows; observations are
not excluded from the pool.  ``stress=True`` gives the harder twin: lengthscales
multiplied by sqrt(d/6) and one eighth of the pool replaced by one- or two-step
grid neighbours of observed points (small posterior variance, worse
conditioning).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

BASE_SEED = 20260411 * 10


@dataclass(frozen=True)
class Config:
    cfg: int            # 1..5
    batch: int
    d: int
    n: int
    m: int
    k: int
    noise_var: float
    ell_lo: float
    ell_hi: float
    kind: str           # "grid" or "perm"
    stress: bool = False

    @property
    def name(self) -> str:
        return f"cfg{self.cfg}{'S' if self.stress else ''}"

    @property
    def seed(self) -> int:
        return BASE_SEED + self.cfg


CONFIGS = {
    1: Config(1, 1, 6, 64, 4096, 8, 1e-4, 0.1, 1.0, "grid"),
    2: Config(2, 1, 16, 256, 262144, 32, 1e-4, 0.1, 1.0, "grid"),
    3: Config(3, 64, 32, 512, 65536, 16, 1e-4, 0.1, 1.0, "grid"),
    4: Config(4, 1, 128, 1024, 1048576, 64, 4e-4, 0.1, 1.0, "perm"),
    5: Config(5, 1, 64, 4096, 1048576, 128, 1e-3, 0.05, 2.0, "grid"),
}


def get_config(cfg: int, *, m: int | None = None, n: int | None = None, batch: int | None = None,
               stress: bool = False) -> Config:
    """One of the five workloads, optionally shrunk (for tests) or in its stress form."""
    c = CONFIGS[cfg]
    kw = {"stress": stress}
    if m is not None:
        kw["m"] = int(m)
    if n is not None:
        kw["n"] = int(n)
    if batch is not None:
        kw["batch"] = int(batch)
    c = replace(c, **kw)
    return replace(c, k=min(c.k, c.m))


# ----------------------------------------------------------------------------- feature grids
_LAUNCH_LEVELS = [
    np.arange(32) / 31.0,                        # block size 32..1024 step 32
    np.arange(8) / 7.0,                          # grid multiplier 1..8
    np.arange(4) / 3.0,                          # unroll 1,2,4,8 (log2 / 3)
    np.arange(224) / 223.0,                      # maxrregcount 32..255
    np.array([0.0, 0.25, 0.5, 1.0]),             # shared-memory carve-out
    np.array([0.0, 1.0]),                        # one boolean
]


def feature_levels(c: Config):
    """Per-feature arrays of admissible (normalised) values for the grid workloads."""
    if c.cfg in (1, 2, 3):
        lv = list(_LAUNCH_LEVELS) + [np.array([0.0, 1.0])] * (c.d - 6)
    elif c.cfg == 5:
        lv = [np.arange(16) / 15.0] * 32 + [np.array([0.0, 1.0])] * 32
    else:
        raise ValueError("cfg 4 is a permutation workload")
    assert len(lv) == c.d
    return lv


def tpe_levels(c: Config, grid: bool = False) -> np.ndarray:
    """Kind of each feature for the Parzen estimator: 0 = ordinal (more than two admissible values),
    2 = a binary flag, treated as a two-level categorical.  The permutation features of config 4 are
    all ordinal.  With ``grid`` an ordinal feature whose admissible values are v/(L-1), L <= 64, is
    declared as such (-L)."""
    if c.cfg == 4:
        return np.zeros(c.d, dtype=np.int32)
    out = []
    for l in feature_levels(c):
        L = len(l)
        if L <= 2:
            out.append(2)
        elif grid and L <= 64 and np.allclose(l, np.arange(L) / (L - 1), rtol=0, atol=1e-12):
            out.append(-L)
        else:
            out.append(0)
    return np.array(out, dtype=np.int32)


def _draw_level_idx(rng, levels, count):
    return np.stack([rng.integers(0, len(l), size=count) for l in levels], axis=1)


def _row_hash(idx: np.ndarray, rng_hash) -> np.ndarray:
    w = rng_hash.integers(1, 2**61, size=idx.shape[1], dtype=np.int64)
    with np.errstate(over="ignore"):
        return (idx.astype(np.int64) * w).sum(axis=1)


def _distinct_level_rows(rng, levels, count):
    """``count`` distinct rows of level indices, iid uniform (duplicates redrawn)."""
    idx = _draw_level_idx(rng, levels, count)
    for _ in range(64):
        h = _row_hash(idx, np.random.default_rng(12345))
        _, first = np.unique(h, return_index=True)
        if first.size == count:
            return idx
        dup = np.ones(count, dtype=bool)
        dup[first] = False
        idx[dup] = _draw_level_idx(rng, levels, int(dup.sum()))
    raise RuntimeError("could not draw distinct rows")


def _levels_to_features(idx, levels):
    out = np.empty(idx.shape, dtype=np.float64)
    for j, l in enumerate(levels):
        out[:, j] = l[idx[:, j]]
    return out


def _neighbours(rng, base_idx, levels, count):
    """One- or two-step grid neighbours of rows of ``base_idx``."""
    src = base_idx[rng.integers(0, base_idx.shape[0], size=count)].copy()
    d = src.shape[1]
    sizes = np.array([len(l) for l in levels])
    for step in range(2):
        active = np.ones(count, dtype=bool) if step == 0 else rng.random(count) < 0.5
        j = rng.integers(0, d, size=count)
        delta = rng.choice([-1, 1], size=count)
        rows = np.nonzero(active)[0]
        v = src[rows, j[rows]] + delta[rows]
        hi = sizes[j[rows]] - 1
        v = np.where(v < 0, 1, v)
        v = np.where(v > hi, hi - 1, v)
        src[rows, j[rows]] = np.clip(v, 0, hi)
    return src


# ----------------------------------------------------------------------------- permutations (cfg 4)
def _draw_perms(rng, count, p=32):
    base = np.tile(np.arange(p, dtype=np.int8), (count, 1))
    return rng.permuted(base, axis=1)  # row r: pass at each position


def _perm_positions(perms):
    pos = np.empty_like(perms)
    rows = np.arange(perms.shape[0])[:, None]
    pos[rows, perms.astype(np.int64)] = np.arange(perms.shape[1], dtype=perms.dtype)[None, :]
    return pos  # pos[r, a] = position of pass a


def _perm_features(pos):
    m, p = pos.shape
    f = np.zeros((m, 4 * p), dtype=np.float32)
    cols = 4 * np.arange(p)[None, :] + (pos.astype(np.int64) // (p // 4))
    f[np.arange(m)[:, None], cols] = np.float32(1.0 / np.sqrt(p))
    return f


def _distinct_perms(rng, count):
    perms = _draw_perms(rng, count)
    for _ in range(64):
        w = np.random.default_rng(999).integers(1, 2**61, size=perms.shape[1], dtype=np.int64)
        with np.errstate(over="ignore"):
            h = ((perms.astype(np.int64) + 1) * w).sum(axis=1)
        _, first = np.unique(h, return_index=True)
        if first.size == count:
            return perms
        dup = np.ones(count, dtype=bool)
        dup[first] = False
        perms[dup] = _draw_perms(rng, int(dup.sum()))
    raise RuntimeError("could not draw distinct permutations")


# ----------------------------------------------------------------------------- response
def _response_grid(rng, X, d, noise_std):
    a = rng.uniform(0.5, 1.0, size=3)
    omega = rng.normal(0.0, 2.0 / np.sqrt(d), size=(3, d))
    phase = rng.uniform(0.0, 2.0 * np.pi, size=3)
    centre = rng.uniform(0.2, 0.8, size=d)
    y = np.zeros(X.shape[0])
    for t in range(3):
        y += a[t] * np.sin(2.0 * np.pi * (X @ omega[t]) + phase[t])
    bowl = ((X - centre) ** 2).sum(axis=1)
    y += bowl * (6.0 / d if d > 6 else 1.0)
    if d >= 16:
        for _ in range(10):
            p, q = rng.choice(d, size=2, replace=False)
            sgn = rng.choice([-1.0, 1.0])
            y += 0.1 * sgn * X[:, p] * X[:, q]
    y += rng.normal(0.0, noise_std, size=X.shape[0])
    return y


def _response_perm(rng, pos, noise_std):
    p = pos.shape[1]
    y = np.zeros(pos.shape[0])
    for _ in range(64):
        a, b = rng.choice(p, size=2, replace=False)
        w = rng.uniform(-1.0, 1.0)
        y += w * (pos[:, a] < pos[:, b])
    y += rng.normal(0.0, noise_std, size=pos.shape[0])
    return y


def _standardise(y):
    return (y - y.mean()) / y.std()


# ----------------------------------------------------------------------------- public
def generate_gp(c: Config, g: int = 0):
    """Inputs of GP number ``g`` of workload ``c``.

    Returns a dict of FP32 arrays: X [n][d], y [n], ell [d], Xcand [m][d] and the
    scalars sf2, sn2 (float32).  Generated in FP64 and rounded once to FP32.
    """
    rng = np.random.default_rng(c.seed + 1000 * g + (500 if c.stress else 0))
    noise_std = float(np.sqrt(c.noise_var))
    ell = rng.uniform(c.ell_lo, c.ell_hi, size=c.d)
    if c.stress:
        ell = ell * np.sqrt(c.d / 6.0)
    n_near = c.m // 8 if c.stress else 0
    if c.kind == "grid":
        levels = feature_levels(c)
        xi = _distinct_level_rows(rng, levels, c.n)
        X = _levels_to_features(xi, levels)
        y = _standardise(_response_grid(rng, X, c.d, noise_std))
        ci = _distinct_level_rows(rng, levels, c.m)
        if n_near:
            ci[rng.choice(c.m, size=n_near, replace=False)] = _neighbours(rng, xi, levels, n_near)
        Xc = _levels_to_features(ci, levels)
    else:
        perms = _distinct_perms(rng, c.n)
        pos = _perm_positions(perms)
        X = _perm_features(pos)
        y = _standardise(_response_perm(rng, pos, noise_std))
        cperm = _distinct_perms(rng, c.m)
        if n_near:
            rows = rng.choice(c.m, size=n_near, replace=False)
            src = perms[rng.integers(0, c.n, size=n_near)].copy()
            a = rng.integers(0, 32, size=n_near)
            b = (a + 1 + rng.integers(0, 31, size=n_near)) % 32
            r = np.arange(n_near)
            src[r, a], src[r, b] = src[r, b].copy(), src[r, a].copy()
            cperm[rows] = src
        Xc = _perm_features(_perm_positions(cperm))
    return {
        "X": np.ascontiguousarray(X, dtype=np.float32),
        "y": np.ascontiguousarray(y, dtype=np.float32),
        "ell": np.ascontiguousarray(ell, dtype=np.float32),
        "sf2": np.float32(1.0),
        "sn2": np.float32(c.noise_var),
        "Xcand": np.ascontiguousarray(Xc, dtype=np.float32),
    }


def generate(c: Config):
    """Inputs of the whole workload, batched.

    Returns FP32 arrays X [batch][n][d], y [batch][n], ell [batch][d], sf2 [batch],
    sn2 [batch], Xcand [batch][m][d].
    """
    gps = [generate_gp(c, g) for g in range(c.batch)]
    return {
        "X": np.stack([p["X"] for p in gps]),
        "y": np.stack([p["y"] for p in gps]),
        "ell": np.stack([p["ell"] for p in gps]),
        "sf2": np.array([p["sf2"] for p in gps], dtype=np.float32),
        "sn2": np.array([p["sn2"] for p in gps], dtype=np.float32),
        "Xcand": np.stack([p["Xcand"] for p in gps]),
    }


def sample_indices(c: Config, count: int) -> np.ndarray:
    """Seeded, sorted, distinct candidate indices in [0, m) for sampled parity checks."""
    rng = np.random.default_rng(c.seed + 77)
    count = min(count, c.m)
    return np.sort(rng.choice(c.m, size=count, replace=False))
