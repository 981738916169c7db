"""GPU parity: the CUDA library, called through its C ABI, against the FP64 CPU oracle.

Small cases compare every output element; the five workloads run at their full sizes on the GPU and
are compared on every candidate where the oracle finishes in seconds, else on a seeded sample of
candidates, with top-k checked against the oracle's EI on the sample pool or a stored full-pool
top list.  Tolerances are the ones in tests/parity.py.
"""
import json
import os

import numpy as np
import pytest

from oracle import gp_oracle as o
from paper_2604_11109_b200 import binding as b
from paper_2604_11109_b200 import workloads as w
from tests.parity import check_scores, check_topk

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
ENGINES = [b.ENGINE_SIMT, b.ENGINE_TENSOR]


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def fit_gpu(g, engine=None):
    gp = b.r3_gp_fit(dev(g["X"]), dev(g["y"]), g["ell"], g["sf2"], g["sn2"])
    if engine is not None:
        try:
            b.r3_gp_set_engine(gp, engine)
        except b.R3Error as e:
            if e.status == 7:
                gp.close()
                pytest.skip("engine does not serve this shape")
            raise
    return gp


def rand_problem(seed, batch, n, d, m, sn2=1e-3, sf2=1.0, spread=1.0):
    rng = np.random.default_rng(seed)
    return {
        "X": rng.uniform(0, 1, (batch, n, d)).astype(np.float32),
        "y": rng.normal(0, 1, (batch, n)).astype(np.float32),
        "ell": (rng.uniform(0.3, 1.5, (batch, d)) * spread).astype(np.float32),
        "sf2": np.full(batch, sf2, np.float32) * rng.uniform(0.5, 2.0, batch).astype(np.float32),
        "sn2": np.full(batch, sn2, np.float32),
        "Xcand": rng.uniform(-0.1, 1.1, (batch, m, d)).astype(np.float32),
    }


def oracle_all(g):
    fits = o.fit_batch(g["X"], g["y"], g["ell"], g["sf2"], g["sn2"])
    mu, sd, ei = o.score_batch(fits, g["Xcand"])
    return fits, mu, sd, ei


def compare_everything(g, gp, k, what):
    fits, mu_r, sd_r, ei_r = oracle_all(g)
    mu, sd, ei, idx, val = b.r3_gp_score_topk(gp, dev(g["Xcand"]), k)
    b.r3_gp_check(gp)
    mu, sd, ei, idx, val = (t.cpu().numpy() for t in (mu, sd, ei, idx, val))
    for q in range(g["X"].shape[0]):
        check_scores(mu[q], sd[q], ei[q], mu_r[q], sd_r[q], ei_r[q], float(np.abs(g["y"][q]).max()),
                     float(g["sf2"][q]), what=f"{what} gp{q}")
        ridx, rval = o.topk(ei_r[q], min(k + 1, ei_r[q].size))
        nxt = rval[k] if rval.size > k else -np.inf
        check_topk(idx[q], lambda i, q=q: ei_r[q][i], ridx[:k], rval[:k], nxt, ei_r[q].max(), what=f"{what} gp{q}")
        # the returned values are the EI entries at the returned indices, in descending order
        assert np.array_equal(val[q], ei[q][idx[q]])
        assert np.all(np.diff(val[q]) <= 0)


# ------------------------------------------------------------------------------------------ fit
@pytest.mark.parametrize("batch,n,d", [(1, 1, 1), (1, 7, 2), (2, 33, 5), (1, 64, 6), (3, 100, 17), (1, 257, 40)])
def test_fit_factor_and_weights_match_oracle(batch, n, d):
    g = rand_problem(100 + n, batch, n, d, 4)
    gp = fit_gpu(g)
    alpha, L = b.r3_gp_get_factor(gp)
    best = b.r3_gp_get_best(gp)
    for q, f in enumerate(o.fit_batch(g["X"], g["y"], g["ell"], g["sf2"], g["sn2"])):
        assert np.allclose(L[q], f.L, rtol=1e-9, atol=1e-11)
        assert np.allclose(alpha[q], f.alpha, rtol=1e-7, atol=1e-9 * np.abs(f.alpha).max())
        assert best[q] == np.float32(f.best)
    gp.close()


def test_fit_reports_not_positive_definite_and_non_finite():
    X = np.array([[[0.1, 0.2], [0.1, 0.2], [0.7, 0.3]]], dtype=np.float32)
    y = np.zeros((1, 3), np.float32)
    with pytest.raises(b.R3Error) as e:
        b.r3_gp_fit(dev(X), dev(y), np.ones((1, 2)), 1.0, 0.0)
    assert e.value.status == 3
    X[0, 1, 0] = np.nan
    with pytest.raises(b.R3Error) as e:
        b.r3_gp_fit(dev(X), dev(y), np.ones((1, 2)), 1.0, 0.1)
    assert e.value.status == 2
    # the context stays usable
    g = rand_problem(1, 1, 8, 2, 4)
    fit_gpu(g).close()


# ------------------------------------------------------------------------------------------ small, element by element
SMALL = [  # batch, n, d, m, k: several tiles and ragged tails in every dimension
    (1, 1, 1, 1, 1),
    (1, 5, 1, 3, 2),
    (1, 50, 3, 333, 8),
    (2, 64, 6, 1000, 16),
    (1, 130, 33, 1500, 32),
    (3, 200, 16, 777, 5),
    (1, 300, 70, 2049, 64),
    (1, 520, 128, 640, 128),
]


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("batch,n,d,m,k", SMALL)
def test_small_cases_every_element(engine, batch, n, d, m, k):
    g = rand_problem(7 * n + d, batch, n, d, m)
    gp = fit_gpu(g, engine)
    compare_everything(g, gp, k, f"small n{n} d{d} m{m}")
    gp.close()


@pytest.mark.parametrize("engine", ENGINES)
def test_candidates_on_and_near_observations_are_rescued(engine):
    # sigma ~ sqrt(noise) at observed points: the regime where sf2 - q cancels
    g = rand_problem(55, 1, 96, 6, 512, sn2=1e-4, spread=2.0)
    g["Xcand"][0, :96] = g["X"][0]
    g["Xcand"][0, 96:192] = g["X"][0] + np.float32(1e-3)
    gp = fit_gpu(g, engine)
    compare_everything(g, gp, 8, "near-observation")
    gp.close()


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("batch,m,k", [(1, 33, 1), (2, 40, 40), (1, 1500, 1024), (3, 5000, 300), (1, 70000, 1000)])
def test_selection_sizes_through_the_scoring_call(engine, batch, m, k):
    """The first level of the selection is taken by the guard's kernel, a block per slice of candidates: k larger
    than a slice, k equal to the pool, slices with a ragged tail, several GPs."""
    g = rand_problem(300 + m, batch, 90, 5, m)
    gp = fit_gpu(g, engine)
    compare_everything(g, gp, k, f"selection m{m} k{k}")
    gp.close()


@pytest.mark.parametrize("spread,sn2", [(1.0, 1e-3), (3.0, 1e-4)])
def test_long_history_with_fp8_cross_terms_near_observations(spread, sn2):
    """From eight passes on (n > 1792) the variance product's cross terms are FP8 MMAs; their error estimate has to
    send the candidates for which that matters -- on and next to observations, long lengthscales -- to the FP64
    pass.  Every element and the top-k against the oracle."""
    n, d, m = 2100, 20, 700
    g = rand_problem(2100 + int(spread), 1, n, d, m, sn2=sn2, spread=spread * np.sqrt(d) / 2)
    g["Xcand"][0, :200] = g["X"][0, :200]
    g["Xcand"][0, 200:400] = g["X"][0, 200:400] + np.float32(2e-3)
    gp = fit_gpu(g, b.ENGINE_TENSOR)
    assert b.r3_gp_tensor_info(gp)["f8_cross_terms"] == 1
    compare_everything(g, gp, 32, f"fp8 cross terms, spread {spread}")
    assert b.r3_gp_last_rescued(gp) >= 200          # the candidates on observations at the least
    gp.close()


def test_incumbent_override_and_engine_query():
    g = rand_problem(77, 2, 40, 4, 300)
    gp = fit_gpu(g)
    assert b.r3_gp_engine(gp) in (b.ENGINE_SIMT, b.ENGINE_TENSOR)
    best = b.r3_gp_get_best(gp) - np.float32(0.5)
    b.r3_gp_set_best(gp, best)
    assert np.array_equal(b.r3_gp_get_best(gp), best)
    mu, sd, ei = (t.cpu().numpy() for t in b.r3_gp_score(gp, dev(g["Xcand"])))
    fits = o.fit_batch(g["X"], g["y"], g["ell"], g["sf2"], g["sn2"])
    for q, f in enumerate(fits):
        mu_r, sd_r, ei_r = o.score(f, g["Xcand"][q], best=float(best[q]))
        check_scores(mu[q], sd[q], ei[q], mu_r, sd_r, ei_r, float(np.abs(g["y"][q]).max()), float(g["sf2"][q]))
    gp.close()


def test_non_finite_candidate_is_latched_not_fatal():
    g = rand_problem(78, 1, 20, 3, 100)
    gp = fit_gpu(g)
    xc = g["Xcand"].copy()
    xc[0, 17, 1] = np.inf
    b.r3_gp_score(gp, dev(xc))
    with pytest.raises(b.R3Error) as e:
        b.r3_gp_check(gp)
    assert e.value.status == 2
    b.r3_gp_score(gp, dev(g["Xcand"]))
    b.r3_gp_check(gp)  # cleared
    gp.close()


def test_host_buffer_form_equals_device_form():
    g = rand_problem(79, 2, 70, 9, 1234)
    gp = fit_gpu(g)
    k = 10
    mu, sd, ei, idx, val = (t.cpu() for t in b.r3_gp_score_topk(gp, dev(g["Xcand"]), k))
    xh = torch.from_numpy(g["Xcand"]).pin_memory()
    out = (torch.empty(2, 1234).pin_memory(), torch.empty(2, 1234).pin_memory(), torch.empty(2, 1234).pin_memory(),
           torch.empty(2, k, dtype=torch.int32).pin_memory(), torch.empty(2, k).pin_memory())
    b.r3_gp_score_topk_host(gp, xh, k, out)
    for a, c in zip((mu, sd, ei, idx, val), out):
        assert torch.equal(a, c)
    gp.close()


@pytest.mark.parametrize("batch,m,pinned", [(1, 148 * 7 * 128 * 2 + 777, True), (1, 148 * 7 * 128 + 5, False),
                                            (3, 70000, True), (5, 3000 * 128, False)])
def test_host_buffer_form_in_pieces_equals_device_form(batch, m, pinned):
    """On the tensor engine a pool of more than about seven waves of tiles is copied in pieces (ranges of one GP's
    tiles, or whole GPs of a batched handle) while earlier pieces are scored; the outputs are bit-identical to the
    device-buffer call.  Some candidates sit on observations so that the guard has work."""
    k = 50
    g = rand_problem(81 + batch, batch, 300, 8, m)
    g["Xcand"][:, 5:25] = g["X"][:, :20]
    gp = fit_gpu(g, b.ENGINE_TENSOR)
    mu, sd, ei, idx, val = (t.cpu() for t in b.r3_gp_score_topk(gp, dev(g["Xcand"]), k))
    xh = torch.from_numpy(g["Xcand"])
    out = [torch.empty(batch, m), torch.empty(batch, m), torch.empty(batch, m),
           torch.empty(batch, k, dtype=torch.int32), torch.empty(batch, k)]
    if pinned:
        xh, out = xh.pin_memory(), [t.pin_memory() for t in out]
    for _ in range(2):   # the second call reuses the staging buffer that the first one's kernels read
        b.r3_gp_score_topk_host(gp, xh, k, tuple(out))
        for a, c in zip((mu, sd, ei, idx, val), out):
            assert torch.equal(a, c)
    b.r3_gp_check(gp)
    gp.close()


# ------------------------------------------------------------------------------------------ top-k alone (bit-exact)
@pytest.mark.parametrize("batch,m,k", [(1, 1, 1), (1, 100, 100), (2, 4096, 7), (1, 4097, 1024), (3, 70001, 33),
                                       (1, 1 << 20, 128), (64, 65536, 16)])
def test_topk_matches_oracle_exactly(batch, m, k):
    rng = np.random.default_rng(m + k)
    e = rng.random((batch, m)).astype(np.float32)
    if m > 50:
        e[:, [3, m // 2, m - 1]] = 2.0                    # ties at the top: lower index first
        e[:, 10:20] = e[:, 5:6]                           # a run of equal values
    if m > 4200:
        e[0, 4095] = e[0, 4096] = 3.0                     # a tie across a chunk boundary
    idx, val = b.r3_topk(dev(e), k)
    idx, val = idx.cpu().numpy(), val.cpu().numpy()
    for q in range(batch):
        ridx, rval = o.topk(e[q], k)
        assert np.array_equal(idx[q], ridx)
        assert np.array_equal(val[q], rval.astype(np.float32))


def test_topk_degenerate_pools():
    """Pools that defeat a selection by value alone: every value equal (the indices decide), a handful of distinct
    values, values that differ in their last mantissa bits only, mostly NaN, signed values with an odd k above the
    size from which the survivors go through the sorting network."""
    rng = np.random.default_rng(77)
    for k in (50, 300, 1024):
        idx, val = b.r3_topk(dev(np.zeros((2, 10000), dtype=np.float32)), k)
        assert np.array_equal(idx.cpu().numpy(), np.tile(np.arange(k), (2, 1)))
        assert not val.cpu().numpy().any()
    cases = [
        (rng.choice(np.array([0.0, 1e-30, 0.5], dtype=np.float32), size=(1, 70001)), 600),
        ((1.0 + rng.integers(0, 64, size=(2, 20000)) * 2.0 ** -23).astype(np.float32), 129),
        (rng.normal(size=(3, 8191)).astype(np.float32), 257),
        (np.full((1, 4096), 7.0, dtype=np.float32), 4096 // 4),
    ]
    for e, k in cases:
        idx, val = b.r3_topk(dev(e), k)
        for q in range(e.shape[0]):
            ridx, rval = o.topk(e[q], k)
            assert np.array_equal(idx[q].cpu().numpy(), ridx)
            assert np.array_equal(val[q].cpu().numpy(), rval.astype(np.float32))
    # NaN ranks below every number, ties among NaN by index
    e = np.full((1, 5000), np.nan, dtype=np.float32)
    numbers = rng.choice(5000, size=10, replace=False)
    e[0, numbers] = rng.normal(size=10).astype(np.float32)
    idx, _ = b.r3_topk(dev(e), 64)
    idx = idx.cpu().numpy()[0]
    assert np.array_equal(idx[:10], o.topk(np.where(np.isnan(e[0]), -np.inf, e[0]), 10)[0])
    rest = np.setdiff1d(np.arange(5000), numbers)
    assert np.array_equal(idx[10:], rest[:54])


def test_topk_special_values():
    e = np.array([[0.0, -0.0, np.nan, -np.inf, 1.0, np.inf, -1.0, 0.0]], dtype=np.float32)
    idx, val = b.r3_topk(dev(e), 8)
    assert idx.cpu().numpy().tolist() == [[5, 4, 0, 1, 7, 6, 3, 2]]   # -0 ties with +0; NaN last
    idx, _ = b.r3_topk(dev(e[0]), 3)
    assert idx.cpu().numpy().tolist() == [5, 4, 0]


# ------------------------------------------------------------------------------------------ the five workloads
def _run_full(c, engine):
    g = w.generate(c)
    gp = fit_gpu(g, engine)
    xc = dev(g["Xcand"])
    out = b.r3_gp_score_topk(gp, xc, c.k)
    b.r3_gp_check(gp)
    out = tuple(t.cpu().numpy() for t in out)
    gp.close()
    del xc
    torch.cuda.empty_cache()
    return g, out


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("cfg", [1, 2])
def test_workload_full_pool_every_candidate(cfg, engine):
    c = w.get_config(cfg)
    g, (mu, sd, ei, idx, val) = _run_full(c, engine)
    fits, mu_r, sd_r, ei_r = oracle_all(g)
    check_scores(mu[0], sd[0], ei[0], mu_r[0], sd_r[0], ei_r[0], float(np.abs(g["y"]).max()), 1.0, what=c.name)
    ridx, rval = o.topk(ei_r[0], c.k + 1)
    check_topk(idx[0], lambda i: ei_r[0][i], ridx[:c.k], rval[:c.k], rval[c.k], ei_r[0].max(), what=c.name)


@pytest.mark.parametrize("engine", ENGINES)
def test_workload_cfg1_stress_twin(engine):
    c = w.get_config(1, stress=True)
    g, (mu, sd, ei, idx, val) = _run_full(c, engine)
    fits, mu_r, sd_r, ei_r = oracle_all(g)
    check_scores(mu[0], sd[0], ei[0], mu_r[0], sd_r[0], ei_r[0], float(np.abs(g["y"]).max()), 1.0, what=c.name)


def _sampled_check(c, g, out, per_gp):
    mu, sd, ei, idx, val = out
    sample = w.sample_indices(c, per_gp)
    for q in range(c.batch):
        f = o.fit(g["X"][q], g["y"][q], g["ell"][q], g["sf2"][q], g["sn2"][q])
        # the sample, plus whatever the GPU chose, scored one by one by the oracle
        pick = np.unique(np.concatenate([sample, idx[q].astype(np.int64)]))
        mu_r, sd_r, ei_r = o.score(f, g["Xcand"][q][pick])
        check_scores(mu[q][pick], sd[q][pick], ei[q][pick], mu_r, sd_r, ei_r, float(np.abs(g["y"][q]).max()),
                     float(g["sf2"][q]), what=f"{c.name} gp{q}")
        # the library's own top-k is exactly the top-k of the EI it wrote
        order = np.lexsort((np.arange(c.m), -ei[q].astype(np.float64)))[:c.k]
        assert np.array_equal(idx[q], order)
        assert np.array_equal(val[q], ei[q][order])
        yield q, f, pick, ei_r


_CFG3_ORACLE = {}


def _cfg3_oracle(c, g):
    """The oracle's mu, sigma, EI of every candidate of all 64 pools (scored once, shared by both engines)."""
    if not _CFG3_ORACLE:
        _CFG3_ORACLE["scores"] = oracle_all(g)[1:]
    return _CFG3_ORACLE["scores"]


@pytest.mark.parametrize("engine", ENGINES)
def test_workload_cfg3_batched_full_size_every_candidate(engine):
    """All 64 GPs at full size: every candidate of every pool against the oracle, and each GP's top-k under the
    top-k rule, against the oracle's EI of the whole pool and against the stored top list."""
    c = w.get_config(3)
    g, (mu, sd, ei, idx, val) = _run_full(c, engine)
    mu_r, sd_r, ei_r = _cfg3_oracle(c, g)
    gold = json.load(open(os.path.join(GOLDEN, f"topk_{c.name}.json")))
    assert gold["m"] == c.m and gold["n"] == c.n and gold["seed"] == c.seed and gold["batch"] == c.batch
    for q in range(c.batch):
        check_scores(mu[q], sd[q], ei[q], mu_r[q], sd_r[q], ei_r[q], float(np.abs(g["y"][q]).max()),
                     float(g["sf2"][q]), what=f"{c.name} gp{q}")
        ridx, rval = o.topk(ei_r[q], c.k + 1)
        check_topk(idx[q], lambda i, q=q: ei_r[q][i], ridx[:c.k], rval[:c.k], rval[c.k], ei_r[q].max(),
                   what=f"{c.name} gp{q}")
        # the stored list is this oracle's
        gq = gold["gps"][q]
        assert gq["idx"][:c.k + 1] == ridx.tolist() and float(gq["ei_max"]) == float(ei_r[q].max())
        assert np.array_equal(val[q], ei[q][idx[q]])


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("cfg", [4, 5])
def test_workload_full_size_sampled_and_full_pool_topk(cfg, engine):
    c = w.get_config(cfg)
    g, out = _run_full(c, engine)
    idx = out[3]
    for q, f, pick, ei_r in _sampled_check(c, g, out, 8192):
        path = os.path.join(GOLDEN, f"topk_{c.name}.json")
        if not os.path.exists(path):
            pytest.skip(f"{path} not generated")
        gold = json.load(open(path))
        assert gold["m"] == c.m and gold["n"] == c.n and gold["seed"] == c.seed
        ref_idx = np.array(gold["idx"], dtype=np.int64)
        ref_val = np.array([float(v) for v in gold["ei"]])
        known = dict(zip(ref_idx.tolist(), ref_val.tolist()))
        known.update(zip(pick.tolist(), ei_r.tolist()))
        check_topk(idx[q], lambda i: known[i], ref_idx[:c.k], ref_val[:c.k], ref_val[c.k], float(gold["ei_max"]),
                   what=c.name)


# ------------------------------------------------------------------------------------------ the paired tensor kernel
@pytest.mark.parametrize("batch,n,d,m,k", [
    (1, 300, 7, 700, 8),        # two passes: one super-pass, both CTAs busy
    (2, 520, 33, 1000, 16),     # three passes: the last super-pass has a pass for one CTA only
    (1, 1100, 64, 515, 8),      # five passes, ragged last tile
    (1, 2050, 20, 260, 4),      # nine passes
])
def test_paired_tensor_kernel_every_element(monkeypatch, batch, n, d, m, k):
    """R3_TC_PAIR=1 sends histories of two or more passes through the kernel that runs a tile on a cluster of
    two CTAs; its results meet the same tolerances."""
    monkeypatch.setenv("R3_TC_PAIR", "1")
    g = rand_problem(900 + n, batch, n, d, m)
    gp = fit_gpu(g, b.ENGINE_TENSOR)
    compare_everything(g, gp, k, f"paired n{n} d{d} m{m}")
    gp.close()


def test_paired_tensor_kernel_on_the_largest_workload(monkeypatch):
    monkeypatch.setenv("R3_TC_PAIR", "1")
    c = w.get_config(5)
    g, out = _run_full(c, b.ENGINE_TENSOR)
    for _ in _sampled_check(c, g, out, 2048):
        pass


# ------------------------------------------------------------------------------------------ the library's size limits
@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("d", [256, 128])
def test_maximum_history_and_feature_count(engine, d):
    """n = 8192 with d = 256 (the limits of r3_gp_fit; served by the CUDA-core engine) and with d = 128 (the
    widest the tensor engine takes): factor, weights and scores against the oracle."""
    rng = np.random.default_rng(8192)
    n, m = 8192, 200
    g = {
        "X": rng.uniform(0, 1, (1, n, d)).astype(np.float32),
        "y": rng.normal(0, 1, (1, n)).astype(np.float32),
        "ell": np.full((1, d), 0.25 * np.sqrt(d), np.float32),   # sqrt(d)-sized lengthscales: correlated neighbours
        "sf2": np.ones(1, np.float32),
        "sn2": np.full(1, 1e-2, np.float32),
        "Xcand": rng.uniform(0, 1, (1, m, d)).astype(np.float32),
    }
    try:
        gp = fit_gpu(g, engine)
    except b.R3Error as e:                                   # pragma: no cover
        pytest.fail(f"fit at the size limits failed: {e}")
    f = o.fit(g["X"][0], g["y"][0], g["ell"][0], g["sf2"][0], g["sn2"][0])
    alpha, L = b.r3_gp_get_factor(gp)
    assert np.allclose(L[0], f.L, rtol=1e-9, atol=1e-11)
    assert np.allclose(alpha[0], f.alpha, rtol=1e-6, atol=1e-8 * np.abs(f.alpha).max())
    mu, sd, ei = (t.cpu().numpy() for t in b.r3_gp_score(gp, dev(g["Xcand"])))
    b.r3_gp_check(gp)
    mu_r, sd_r, ei_r = o.score(f, g["Xcand"][0])
    check_scores(mu[0], sd[0], ei[0], mu_r, sd_r, ei_r, float(np.abs(g["y"]).max()), 1.0, what=f"n=8192 d={d}")
    gp.close()


# ------------------------------------------------------------------------------------------ seeded random shapes
@pytest.mark.parametrize("engine", ENGINES)
def test_random_shapes_and_conditioning(engine):
    """Thirty seeded problems with random batch, n, d, m, lengthscale spread and noise, a third of them with
    candidates on or next to observations: every element and the top-k against the oracle."""
    rng = np.random.default_rng(2604)
    for it in range(30):
        batch, n, d, m = int(rng.integers(1, 4)), int(rng.integers(1, 600)), int(rng.integers(1, 129)), int(rng.integers(1, 2500))
        spread = float(rng.choice([0.3, 1.0, 3.0])) * np.sqrt(d) / 2
        g = {
            "X": rng.uniform(0, 1, (batch, n, d)).astype(np.float32),
            "y": rng.normal(0, 1, (batch, n)).astype(np.float32),
            "ell": (rng.uniform(0.5, 1.5, (batch, d)) * spread).astype(np.float32),
            "sf2": rng.uniform(0.5, 2, batch).astype(np.float32),
            "sn2": np.full(batch, float(rng.choice([1e-2, 1e-3, 1e-5])), np.float32),
            "Xcand": rng.uniform(-0.1, 1.1, (batch, m, d)).astype(np.float32),
        }
        if rng.random() < 0.33 and m > 4 and n > 2:
            kk = min(n, m // 2)
            g["Xcand"][:, :kk] = g["X"][:, :kk] + np.float32(rng.choice([0.0, 1e-3]))
        gp = b.r3_gp_fit(dev(g["X"]), dev(g["y"]), g["ell"], g["sf2"], g["sn2"])
        try:
            b.r3_gp_set_engine(gp, engine)
        except b.R3Error as e:
            assert e.status == 7
            gp.close()
            continue
        compare_everything(g, gp, min(m, int(rng.integers(1, 65))), f"random #{it} n{n} d{d} m{m}")
        gp.close()


def test_calls_on_a_side_stream_give_the_same_results():
    """Everything a call enqueues goes to the stream it is given: results computed on a side stream (with the
    default stream busy with unrelated work) are bit-identical to those of the default stream."""
    g = rand_problem(91, 2, 150, 20, 5000)
    gp = fit_gpu(g)
    xc = dev(g["Xcand"])
    ref = [t.clone() for t in b.r3_gp_score_topk(gp, xc, 16)]
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    busy = torch.empty(1 << 26, device="cuda")
    with torch.cuda.stream(side):
        for _ in range(3):
            busy.normal_()                      # keeps the default stream's neighbour occupied; no dependency
        out = b.r3_gp_score_topk(gp, xc, 16)
        b.r3_gp_check(gp)
    side.synchronize()
    for a, c in zip(ref, out):
        assert torch.equal(a, c)
    gp.close()


def test_scoring_step_replays_from_a_cuda_graph():
    """Once the handle's workspace has its size (a first call), r3_gp_score_topk only enqueues work on the stream it
    is given -- kernels, two small memsets, one small copy to pinned memory -- so a step can be captured in a CUDA
    graph and replayed: the results are bit-identical to a direct call."""
    g = rand_problem(93, 2, 300, 12, 3000)
    gp = fit_gpu(g)
    xc = dev(g["Xcand"])
    k = 24
    out = (torch.empty((2, 3000), device="cuda"), torch.empty((2, 3000), device="cuda"), torch.empty((2, 3000), device="cuda"),
           torch.empty((2, k), dtype=torch.int32, device="cuda"), torch.empty((2, k), device="cuda"))
    b.r3_gp_score_topk(gp, xc, k, out)
    torch.cuda.synchronize()
    ref = [t.clone() for t in out]
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        b.r3_gp_score_topk(gp, xc, k, out)
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            b.r3_gp_score_topk(gp, xc, k, out)
    for rep in range(3):
        for t in out:
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for a, r in zip(out, ref):
            assert torch.equal(a, r)
    b.r3_gp_check(gp)
    gp.close()

