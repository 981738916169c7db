"""GPU parity of TPE candidate scoring: the CUDA library through its C ABI against the FP64 oracle.

Integer results (the order of the history, the good-set size, the selected top-k where the oracle's
gap exceeds the tolerance) must match exactly.  Floating point: the fitted model is computed in FP64
on both sides and stored in FP32 on the device (relative 2e-7 on a mean, bandwidth or coefficient);
the score is a sum over d dimensions of differences of log-sums evaluated in FP32 with MUFU
exponentials.  One log-sum is off by about 5e-7 (rounding of the exponents, 2^-24 of a magnitude
up to 10, and the MUFU results) plus 3e-8 * sqrt(n) (FP32 accumulation of up to n + 1 positive
terms); the 2 * d_ord log-sums of a score err independently, so the score is held to four standard
deviations of that,

    |score - oracle| <= 4 * sqrt(2 * d_ord) * (5e-7 + 3e-8 * sqrt(n)) + 5e-6 * |oracle|,

d_ord the number of ordinal dimensions (at least 1).
"""
import numpy as np
import pytest

from oracle import tpe_oracle as T
from paper_2604_11109_b200 import binding as b
from paper_2604_11109_b200 import workloads as w

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

RTOL = 5e-6


def atol(n, levels):
    d_ord = max(1, int((np.asarray(levels) == 0).sum()))
    return 4.0 * np.sqrt(2.0 * d_ord) * (5e-7 + 3e-8 * np.sqrt(n))


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def rand_case(seed, n, d, m, frac_cat=0.4, continuous=True):
    rng = np.random.default_rng(seed)
    levels = np.zeros(d, dtype=np.int32)
    X = np.empty((n, d))
    Xc = np.empty((m, d))
    for j in range(d):
        if rng.random() < frac_cat:
            C = int(rng.integers(2, 9))
            levels[j] = C
            X[:, j] = rng.integers(0, C, size=n) / (C - 1)
            Xc[:, j] = rng.integers(0, C, size=m) / (C - 1)
        elif continuous and rng.random() < 0.5:
            X[:, j] = rng.random(n)
            Xc[:, j] = rng.random(m)
        else:
            L = int(rng.integers(3, 17))
            X[:, j] = rng.integers(0, L, size=n) / (L - 1)
            Xc[:, j] = rng.integers(0, L, size=m) / (L - 1)
            if rng.random() < 0.5:
                levels[j] = -L          # declared as a grid: tabulated by the fit
                if rng.random() < 0.5:  # and some candidates slightly off the grid
                    Xc[:, j] += rng.uniform(-0.3, 0.3, m) / (L - 1)
    y = np.round(rng.normal(0, 1, n), 1)      # rounded: ties in y
    return X.astype(np.float32), y.astype(np.float32), levels, Xc.astype(np.float32)


def merged(mu, sigma, coef):
    """One (mean, sigma, summed coefficient) row per distinct (mean, sigma), sorted."""
    key = np.lexsort((sigma, mu))
    mu, sigma, coef = mu[key], sigma[key], coef[key]
    first = np.ones(mu.shape[0], dtype=bool)
    first[1:] = (mu[1:] != mu[:-1]) | (np.abs(sigma[1:] - sigma[:-1]) > 1e-6 * sigma[:-1])
    start = np.flatnonzero(first)
    return mu[start], sigma[start], np.add.reduceat(coef, start)


def check_model(tpe, model, n, d):
    n_good, order, comps, counts, table = b.r3_tpe_get_model(tpe)
    assert n_good == model.n_good
    assert order.tolist() == model.order.tolist()
    for j in range(d):
        if model.levels[j] > 0:
            C = int(model.levels[j])
            want = np.log(model.good[j].prob) - np.log(model.bad[j].prob)
            np.testing.assert_allclose(table[j, :C], want, rtol=1e-6, atol=1e-6)
            assert counts[j].tolist() == [0, 0]
            continue
        for set_, (mix, off) in enumerate(((model.good[j], 0), (model.bad[j], n_good + 1))):
            cnt = int(counts[j, set_])
            assert 1 <= cnt <= mix.mu.shape[0]
            got = comps[j, off:off + cnt].astype(np.float64)
            # each set stays sorted by mean
            assert (np.diff(got[:, 0]) >= 0).all()
            # the exponent's factor belongs to the stored sigma
            np.testing.assert_allclose(got[:, 1], np.log2(np.e) / (2 * got[:, 3] ** 2), rtol=3e-7)
            # equal (mean, sigma) components are one component with the summed coefficient: compare the
            # two sides after merging both completely (the device merges neighbours in its sorted order)
            ref_coef = mix.weight / (mix.sigma * mix.Z * np.sqrt(2 * np.pi))
            rmu, rsig, rcoef = merged(mix.mu.astype(np.float64), mix.sigma, ref_coef)
            gmu, gsig, gcoef = merged(got[:, 0], got[:, 3], np.exp2(got[:, 2]))
            np.testing.assert_array_equal(gmu, rmu)
            np.testing.assert_allclose(gsig, rsig, rtol=2e-7)
            np.testing.assert_allclose(gcoef, rcoef, rtol=1e-6)
            # a run of equal values gives at most three neighbour-gap bandwidths (its two ends and its
            # inside), and the prior can split one run in two
            assert cnt <= 3 * np.unique(mix.mu).shape[0] + 2
        if model.levels[j] < 0:
            L = int(-model.levels[j])
            xg = (np.arange(L) / (L - 1)).astype(np.float32)
            want = np.log(T.density(model.good[j], xg)) - np.log(T.density(model.bad[j], xg))
            np.testing.assert_allclose(table[j, :L], want, rtol=1e-6, atol=1e-6)
        else:
            assert not table[j].any()


def check_score(got, want, ATOL):
    err = np.abs(got.astype(np.float64) - want)
    tol = ATOL + RTOL * np.abs(want)
    worst = float((err / tol).max())
    assert worst <= 1.0, f"score error {worst:.2f} x tolerance (max abs {err.max():.3e})"
    return worst


def check_topk(score_gpu, idx_gpu, want, k, ATOL):
    """Exact where the oracle separates rank k from rank k + 1 by more than the tolerance."""
    ref = T.tpe_topk(want, min(k + 1, want.shape[0]))
    tol = ATOL + RTOL * np.abs(want[ref]).max()
    sel = want[idx_gpu]
    assert len(set(idx_gpu.tolist())) == k
    if ref.shape[0] > k and want[ref[k - 1]] - want[ref[k]] > 2 * tol:
        assert set(idx_gpu.tolist()) == set(ref[:k].tolist())
    # every selected candidate is within tolerance of belonging; order by the device's own scores
    assert sel.min() >= want[ref[k - 1]] - 2 * tol
    s = score_gpu[idx_gpu]
    assert np.all(s[:-1] >= s[1:])
    eq = s[:-1] == s[1:]
    assert np.all(idx_gpu[:-1][eq] < idx_gpu[1:][eq])


@pytest.mark.parametrize("seed,n,d,m,gamma,w0", [
    (0, 1, 1, 5, 0.25, 1.0),            # one observation: the bad set is the prior alone
    (1, 2, 3, 17, 1.0, 1.0),            # gamma = 1: everything is good
    (2, 37, 5, 1025, 0.25, 1.0),        # one candidate past a block's range
    (3, 200, 7, 4099, 0.15, 2.5),
    (4, 513, 13, 3000, 0.5, 0.3),
    (5, 4096, 3, 2048, 0.25, 1.0),      # largest history
])
def test_small_cases(seed, n, d, m, gamma, w0):
    X, y, levels, Xc = rand_case(seed, n, d, m)
    model = T.tpe_fit(X, y, levels, gamma, w0)
    tpe = b.r3_tpe_fit(dev(X), dev(y), levels, gamma, w0)
    check_model(tpe, model, n, d)
    got = b.r3_tpe_score(tpe, dev(Xc)).cpu().numpy()
    b.r3_tpe_check(tpe)
    want = T.tpe_score(model, Xc)
    check_score(got, want, atol(n, levels))
    k = min(8, m)
    idx, val = b.r3_topk(dev(got), k)
    check_topk(got, idx.cpu().numpy().astype(np.int64), want, k, atol(n, levels))
    tpe.close()


def test_all_categorical_and_all_ordinal():
    for frac in (0.0, 1.0):
        X, y, levels, Xc = rand_case(40 + int(frac), 150, 6, 777, frac_cat=frac)
        model = T.tpe_fit(X, y, levels, 0.25, 1.0)
        tpe = b.r3_tpe_fit(dev(X), dev(y), levels, 0.25, 1.0)
        check_model(tpe, model, 150, 6)
        check_score(b.r3_tpe_score(tpe, dev(Xc)).cpu().numpy(), T.tpe_score(model, Xc), atol(150, levels))
        tpe.close()


def test_repeated_values_are_merged_and_large_models_are_not_packed():
    """Unevenly spaced admissible values, one of them the prior's mean, repeated many times: a few components
    per value remain, and candidates anywhere in [0, 1] score as with the unmerged mixture.  A continuous
    feature beside them keeps all its components; with the longest history the model exceeds what a block
    holds in shared memory, so both scoring paths are taken."""
    rng = np.random.default_rng(77)
    values = np.array([0.0, 0.1, 0.12, 0.5, 0.55, 0.9, 1.0])
    for n, m in ((300, 5000), (4096, 3000)):
        X = values[rng.integers(0, values.shape[0], size=(n, 6))]
        X[:, 5] = rng.random(n)
        Xc = rng.random((m, 6))
        Xc[: m // 2] = values[rng.integers(0, values.shape[0], size=(m // 2, 6))]
        y = rng.normal(0, 1, n)
        X, y, Xc = X.astype(np.float32), y.astype(np.float32), Xc.astype(np.float32)
        levels = np.zeros(6, dtype=np.int32)
        model = T.tpe_fit(X, y, levels, 0.25, 1.0)
        tpe = b.r3_tpe_fit(dev(X), dev(y), levels, 0.25, 1.0)
        check_model(tpe, model, n, 6)
        counts = b.r3_tpe_get_model(tpe)[3]
        assert counts[:5].max() <= 3 * values.shape[0] + 2
        assert counts[5].sum() == n + 2
        check_score(b.r3_tpe_score(tpe, dev(Xc)).cpu().numpy(), T.tpe_score(model, Xc), atol(n, levels))
        b.r3_tpe_check(tpe)
        tpe.close()


@pytest.mark.parametrize("d,m", [(8, 40000), (12, 3000), (16, 300001), (10, 5000)])
def test_packed_model_pool_sizes_and_alignment(d, m):
    """Discrete ordinal features (a model that a block keeps in shared memory), pools large and small enough
    for both tile widths, and a pool that does not start on a 16-byte boundary: all give the oracle's
    scores."""
    rng = np.random.default_rng(500 + d)
    n = 400
    L = rng.integers(3, 20, size=d)
    X = np.stack([rng.integers(0, L[j], size=n) / (L[j] - 1) for j in range(d)], axis=1).astype(np.float32)
    Xc = np.stack([rng.integers(0, L[j], size=m) / (L[j] - 1) for j in range(d)], axis=1).astype(np.float32)
    levels = np.zeros(d, dtype=np.int32)
    levels[1] = 2
    X[:, 1], Xc[:, 1] = rng.integers(0, 2, n), rng.integers(0, 2, m)
    y = rng.normal(size=n).astype(np.float32)
    model = T.tpe_fit(X, y, levels, 0.25, 1.0)
    tpe = b.r3_tpe_fit(dev(X), dev(y), levels, 0.25, 1.0)
    want = T.tpe_score(model, Xc)
    check_score(b.r3_tpe_score(tpe, dev(Xc)).cpu().numpy(), want, atol(n, levels))
    shifted = torch.empty(m * d + 1, dtype=torch.float32, device="cuda")[1:].view(m, d)
    shifted.copy_(dev(Xc))
    check_score(b.r3_tpe_score(tpe, shifted).cpu().numpy(), want, atol(n, levels))
    b.r3_tpe_check(tpe)
    tpe.close()


@pytest.mark.parametrize("d,m", [(4, 1000), (8, 5000), (20, 3001), (64, 70000), (132, 2000)])
def test_all_tabulated_dimensions_take_the_streaming_kernel(d, m):
    """Every dimension categorical or on a grid and d a multiple of 4: scored by whole-row loads and look-ups."""
    rng = np.random.default_rng(d)
    n = 300
    levels = np.empty(d, dtype=np.int32)
    X, Xc = np.empty((n, d)), np.empty((m, d))
    for j in range(d):
        L = int(rng.integers(2, 33))
        levels[j] = L if rng.random() < 0.5 else -L
        X[:, j] = rng.integers(0, L, size=n) / (L - 1)
        Xc[:, j] = rng.integers(0, L, size=m) / (L - 1)
    X, Xc = X.astype(np.float32), Xc.astype(np.float32)
    y = rng.normal(size=n).astype(np.float32)
    model = T.tpe_fit(X, y, levels, 0.25, 1.0)
    tpe = b.r3_tpe_fit(dev(X), dev(y), levels, 0.25, 1.0)
    check_model(tpe, model, n, d)
    want = T.tpe_score(model, Xc)
    check_score(b.r3_tpe_score(tpe, dev(Xc)).cpu().numpy(), want, atol(n, levels))
    # a pool that does not start on a 16-byte boundary goes through the general kernel: same scores
    shifted = torch.empty(m * d + 1, dtype=torch.float32, device="cuda")[1:].view(m, d)
    shifted.copy_(dev(Xc))
    check_score(b.r3_tpe_score(tpe, shifted).cpu().numpy(), want, atol(n, levels))
    tpe.close()


def test_candidates_outside_the_unit_interval():
    X, y, levels, Xc = rand_case(50, 90, 4, 600, frac_cat=0.25)
    Xc = (Xc * 1.3 - 0.15).astype(np.float32)
    model = T.tpe_fit(X, y, levels, 0.25, 1.0)
    tpe = b.r3_tpe_fit(dev(X), dev(y), levels, 0.25, 1.0)
    check_score(b.r3_tpe_score(tpe, dev(Xc)).cpu().numpy(), T.tpe_score(model, Xc), atol(90, levels))
    tpe.close()


@pytest.mark.parametrize("cfg,sample,grid", [(1, 4096, False), (2, 8192, False), (3, 4096, False), (4, 4096, False),
                                             (5, 1024, False), (2, 8192, True), (3, 8192, True),
                                             (5, 8192, True)])
def test_workloads_full_size(cfg, sample, grid):
    """The launch configuration the benchmark times, on the whole pool; the oracle on a seeded sample."""
    c = w.get_config(cfg)
    g = w.generate_gp(c, 0)
    levels = w.tpe_levels(c, grid=grid)
    model = T.tpe_fit(g["X"], g["y"], levels, 0.25, 1.0)
    tpe = b.r3_tpe_fit(dev(g["X"]), dev(g["y"]), levels, 0.25, 1.0)
    check_model(tpe, model, c.n, c.d)
    got = b.r3_tpe_score(tpe, dev(g["Xcand"])).cpu().numpy()
    b.r3_tpe_check(tpe)
    assert np.isfinite(got).all()
    sel = w.sample_indices(c, sample)
    want = T.tpe_score(model, g["Xcand"][sel])
    worst = check_score(got[sel], want, atol(c.n, levels))
    print(f"tpe {c.name} grid={grid}: worst error/tolerance {worst:.3f}")
    # top-k of the sampled pool, decided by the device on its own scores of the same candidates
    k = min(c.k, 32)
    idx, _ = b.r3_topk(dev(got[sel]), k)
    check_topk(got[sel], idx.cpu().numpy().astype(np.int64), want, k, atol(c.n, levels))
    # the full pool's selection is sorted, distinct and at least as good as the sample's best
    idx_full, val_full = b.r3_topk(dev(got), k)
    v = val_full.cpu().numpy()
    assert np.all(v[:-1] >= v[1:]) and v[0] >= got[sel].max()
    tpe.close()


def test_errors():
    X, y, levels, Xc = rand_case(60, 20, 3, 50)
    ybad = y.copy()
    ybad[3] = np.nan
    with pytest.raises(b.R3Error) as e:
        b.r3_tpe_fit(dev(X), dev(ybad), levels)
    assert e.value.status == 2
    Xbad = X.copy()
    Xbad[5, 1] = np.inf
    with pytest.raises(b.R3Error) as e:
        b.r3_tpe_fit(dev(Xbad), dev(y), levels)
    assert e.value.status == 2
    for bad_levels in ([1, 0, 0], [0, 65, 0], [0, -1, 0], [0, -65, 0]):
        with pytest.raises(b.R3Error) as e:
            b.r3_tpe_fit(dev(X), dev(y), np.array(bad_levels, dtype=np.int32))
        assert e.value.status == 1
    for gamma, w0 in ((0.0, 1.0), (1.5, 1.0), (0.25, 0.0)):
        with pytest.raises(b.R3Error) as e:
            b.r3_tpe_fit(dev(X), dev(y), levels, gamma, w0)
        assert e.value.status == 1
    tpe = b.r3_tpe_fit(dev(X), dev(y), levels)
    Xc[7, 0] = np.nan
    b.r3_tpe_score(tpe, dev(Xc))
    with pytest.raises(b.R3Error) as e:
        b.r3_tpe_check(tpe)
    assert e.value.status == 2
    b.r3_tpe_score(tpe, dev(np.nan_to_num(Xc)))
    b.r3_tpe_check(tpe)      # the latch was cleared
    tpe.close()
