"""GPU parity of r3_gp_append: extending the factor by k observations must give what a fit of the
concatenated history gives.  The oracle is exactly that definition -- its own fit on the concatenated
data -- so the factor, the weights, the incumbent and every score computed afterwards are compared
with it (same tolerances as for r3_gp_fit and r3_gp_score).
"""
import numpy as np
import pytest

from oracle import gp_oracle as o
from paper_2604_11109_b200 import binding as b
from paper_2604_11109_b200 import workloads as w
from tests.parity import check_scores

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def problem(seed, batch, n, d, m):
    rng = np.random.default_rng(seed)
    return {
        "X": rng.uniform(0, 1, (batch, n, d)).astype(np.float32),
        "y": rng.normal(0, 1, (batch, n)).astype(np.float32),
        "ell": rng.uniform(0.3, 1.5, (batch, d)).astype(np.float32),
        "sf2": rng.uniform(0.5, 2.0, batch).astype(np.float32),
        "sn2": np.full(batch, 1e-3, np.float32),
        "Xcand": rng.uniform(-0.1, 1.1, (batch, m, d)).astype(np.float32),
    }


def check_handle(gp, g, n_total):
    """Factor, weights and incumbent of the handle against the oracle's fit of the first n_total rows."""
    alpha, L = b.r3_gp_get_factor(gp)
    best = b.r3_gp_get_best(gp)
    assert b.r3_gp_size(gp) == n_total and gp.n == n_total
    fits = o.fit_batch(g["X"][:, :n_total], g["y"][:, :n_total], g["ell"], g["sf2"], g["sn2"])
    for q, f in enumerate(fits):
        assert np.allclose(L[q], f.L, rtol=1e-9, atol=1e-11)
        assert np.allclose(alpha[q], f.alpha, rtol=1e-7, atol=1e-9 * np.abs(f.alpha).max())
        assert best[q] == np.float32(f.best)
    return fits


def check_scoring(gp, g, fits):
    mu, sd, ei = (t.cpu().numpy() for t in b.r3_gp_score(gp, dev(g["Xcand"])))
    b.r3_gp_check(gp)
    for q, f in enumerate(fits):
        mu_r, sd_r, ei_r = o.score(f, g["Xcand"][q])
        check_scores(mu[q], sd[q], ei[q], mu_r, sd_r, ei_r, float(np.abs(g["y"][q]).max()), float(g["sf2"][q]),
                     what="after append")


@pytest.mark.parametrize("batch,n0,steps,d", [
    (1, 1, [1, 1, 2], 3),            # from a single observation
    (1, 30, [1, 1, 1], 5),           # crossing the padding boundary at 32 one row at a time
    (2, 64, [33, 128], 8),           # aligned start, ragged and maximal steps, two GPs
    (1, 250, [7, 128, 100], 20),     # tensor engine shapes (d > 16)
    (3, 100, [28, 4], 40),
])
def test_append_matches_fit_of_concatenated_history(batch, n0, steps, d):
    n_all = n0 + sum(steps)
    g = problem(500 + n0, batch, n_all, d, 700)
    gp = b.r3_gp_fit(dev(g["X"][:, :n0]), dev(g["y"][:, :n0]), g["ell"], g["sf2"], g["sn2"])
    n = n0
    for k in steps:
        b.r3_gp_append(gp, dev(g["X"][:, n:n + k]), dev(g["y"][:, n:n + k]))
        n += k
        fits = check_handle(gp, g, n)
    check_scoring(gp, g, fits)
    gp.close()


@pytest.mark.parametrize("engine", [b.ENGINE_SIMT, b.ENGINE_TENSOR])
def test_append_then_score_both_engines(engine):
    g = problem(77, 1, 400, 24, 3000)
    gp = b.r3_gp_fit(dev(g["X"][:, :300]), dev(g["y"][:, :300]), g["ell"], g["sf2"], g["sn2"])
    b.r3_gp_append(gp, dev(g["X"][:, 300:400]), dev(g["y"][:, 300:400]))
    b.r3_gp_set_engine(gp, engine)
    fits = check_handle(gp, g, 400)
    check_scoring(gp, g, fits)
    gp.close()


def test_append_on_workload_history():
    """Config 5's history grown from 3968 to 4096 observations in one step of 128 (the k of that config)."""
    c = w.get_config(5, m=4096)
    g = w.generate(c)
    n0 = c.n - 128
    gp = b.r3_gp_fit(dev(g["X"][:, :n0]), dev(g["y"][:, :n0]), g["ell"], g["sf2"], g["sn2"])
    b.r3_gp_append(gp, dev(g["X"][:, n0:]), dev(g["y"][:, n0:]))
    fits = check_handle(gp, g, c.n)
    check_scoring(gp, g, fits)
    gp.close()


def test_append_errors_leave_the_handle_usable():
    g = problem(9, 1, 40, 4, 200)
    gz = dict(g, sn2=np.zeros(1, np.float32))
    gp = b.r3_gp_fit(dev(gz["X"][:, :30]), dev(gz["y"][:, :30]), gz["ell"], gz["sf2"], gz["sn2"])
    # a duplicate of an observed row with zero noise: the extended matrix is singular
    dup = gz["X"][:, 3:4].copy()
    with pytest.raises(b.R3Error) as e:
        b.r3_gp_append(gp, dev(dup), dev(np.zeros((1, 1), np.float32)))
    assert e.value.status == 3 and "pivot 30" in str(e.value)
    bad = gz["X"][:, 30:32].copy()
    bad[0, 1, 2] = np.nan
    with pytest.raises(b.R3Error) as e:
        b.r3_gp_append(gp, dev(bad), dev(gz["y"][:, 30:32]))
    assert e.value.status == 2
    with pytest.raises(b.R3Error) as e:
        b.r3_gp_append(gp, dev(np.zeros((1, 129, 4), np.float32)), dev(np.zeros((1, 129), np.float32)))
    assert e.value.status == 1
    # unchanged and still usable: same factor as before, and a valid append still works
    fits = check_handle(gp, gz, 30)
    b.r3_gp_append(gp, dev(gz["X"][:, 30:40]), dev(gz["y"][:, 30:40]))
    fits = check_handle(gp, gz, 40)
    check_scoring(gp, gz, fits)
    gp.close()


def test_append_on_an_ill_conditioned_history_matches_a_fit():
    """Noise-free linear data at lengthscales 1000, signal variance 1e6 and noise 1e-8 (where the hyper-parameter
    fit ends on such data): the product with the explicit inverse alone made the Schur complement of the new rows
    indefinite; with the refinement step the append succeeds and its evidence is as close to an 80-bit reference
    as that of a fit of the whole history, within a small factor."""
    from tests.test_gpu_lml import _lml_extended
    if np.finfo(np.longdouble).eps > 2e-19:
        pytest.skip("no 80-bit long double on this platform")
    for seed, n, d, k in ((2, 115, 1, 32), (3, 160, 9, 64)):
        rng = np.random.default_rng(7000 + seed)
        X = rng.uniform(0, 1, (1, n, d)).astype(np.float32)
        y = (3.0 * X.sum(-1)).astype(np.float32)
        ell = np.full((1, d), 1000.0, np.float32)
        sf2, sn2 = np.full(1, 1e6, np.float32), np.full(1, 1e-8, np.float32)
        ref = _lml_extended(X[0], y[0], ell[0], sf2[0], sn2[0])
        gp = b.r3_gp_fit(dev(X), dev(y), ell, sf2, sn2)
        full, _ = b.r3_gp_lml(gp)
        gp.close()
        gp = b.r3_gp_fit(dev(X[:, :n - k]), dev(y[:, :n - k]), ell, sf2, sn2)
        b.r3_gp_append(gp, dev(X[:, n - k:]), dev(y[:, n - k:]))
        app, _ = b.r3_gp_lml(gp)
        gp.close()
        assert abs(app[0] - ref) <= 4.0 * abs(full[0] - ref) + 1e-7 * abs(ref), (app[0], full[0], ref)
