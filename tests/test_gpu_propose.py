"""GPU parity of r3_gp_propose (greedy batch by fantasies) against the oracle's definition: refit the
augmented history and rescore the pool before every pick.

The picks are integers, so they must be the oracle's, in order -- except where the oracle itself
cannot separate two candidates: if at some pick the GPU's choice and the oracle's differ, the oracle's
EI of the two at that step must agree within the EI tolerance (1e-5 of the pool's largest EI), and the
comparison stops there (later picks depend on the earlier ones).
"""
import numpy as np
import pytest

from oracle import gp_oracle as o
from paper_2604_11109_b200 import binding as b
from paper_2604_11109_b200 import workloads as w
from tests.parity import EI_ABS_FLOOR

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def problem(seed, batch, n, d, m, sn2=1e-3):
    rng = np.random.default_rng(seed)
    return {
        "X": rng.uniform(0, 1, (batch, n, d)).astype(np.float32),
        "y": rng.normal(0, 1, (batch, n)).astype(np.float32),
        "ell": rng.uniform(0.3, 1.2, (batch, d)).astype(np.float32),
        "sf2": rng.uniform(0.5, 2.0, batch).astype(np.float32),
        "sn2": np.full(batch, sn2, np.float32),
        "Xcand": rng.uniform(0, 1, (batch, m, d)).astype(np.float32),
    }


def oracle_ei_at_step(g, q_, picks, lie):
    """The oracle's EI over the pool of GP q_ after conditioning on `picks` (in order)."""
    X, y = g["X"][q_], g["y"][q_]
    best0 = float(y.min())
    Xa, ya = X.copy(), y.copy()
    for j in picks:
        f = o.fit(Xa, ya, g["ell"][q_], g["sf2"][q_], g["sn2"][q_])
        mu, _, _ = o.score(f, g["Xcand"][q_][j:j + 1], best=best0)
        value = mu[0] if lie == "believer" else best0
        Xa = np.concatenate([Xa, g["Xcand"][q_][j:j + 1]])
        ya = np.concatenate([ya, np.array([value], dtype=np.float32)])
    f = o.fit(Xa, ya, g["ell"][q_], g["sf2"][q_], g["sn2"][q_])
    return o.score(f, g["Xcand"][q_], best=best0)[2]


def check_sequence(g, q_, got_idx, got_val, q, lie):
    ref_idx, ref_val = o.propose(g["X"][q_], g["y"][q_], g["ell"][q_], g["sf2"][q_], g["sn2"][q_], g["Xcand"][q_], q,
                                 lie)
    tol = max(1e-5 * ref_val.max(), EI_ABS_FLOOR)      # EI comes back in FP32
    assert len(set(got_idx.tolist())) == q
    for t in range(q):
        if got_idx[t] == ref_idx[t]:
            assert abs(got_val[t] - ref_val[t]) <= tol + 1e-6 * ref_val[t]
            continue
        e = oracle_ei_at_step(g, q_, list(ref_idx[:t]), lie)
        assert abs(e[got_idx[t]] - e[ref_idx[t]]) <= tol, f"pick {t}: {got_idx[t]} vs {ref_idx[t]}"
        return t
    return q


@pytest.mark.parametrize("lie", ["believer", "liar"])
@pytest.mark.parametrize("batch,n,d,m,q", [(1, 20, 2, 50, 10), (2, 150, 6, 900, 24), (1, 300, 24, 1000, 16)])
def test_whole_pool_shortlist_matches_oracle(batch, n, d, m, q, lie):
    g = problem(900 + n, batch, n, d, m)
    gp = b.r3_gp_fit(dev(g["X"]), dev(g["y"]), g["ell"], g["sf2"], g["sn2"])
    idx, val, cert = b.r3_gp_propose(gp, dev(g["Xcand"]), q, shortlist=min(m, 1023), lie=lie)
    b.r3_gp_check(gp)
    idx, val = idx.cpu().numpy(), val.cpu().numpy()
    for q_ in range(batch):
        assert check_sequence(g, q_, idx[q_], val[q_], q, lie) == q
        assert cert[q_] == (m <= 1023)
    gp.close()


def test_believer_shortlist_is_certified_and_exact_on_a_large_pool():
    g = problem(31, 1, 200, 5, 60000)
    gp = b.r3_gp_fit(dev(g["X"]), dev(g["y"]), g["ell"], g["sf2"], g["sn2"])
    idx, val, cert = b.r3_gp_propose(gp, dev(g["Xcand"]), 16)          # automatic shortlist of 256
    b.r3_gp_check(gp)
    assert cert[0]
    assert check_sequence(g, 0, idx.cpu().numpy()[0], val.cpu().numpy()[0], 16, "believer") == 16
    # EI of the picks never increases under the believer
    v = val.cpu().numpy()[0]
    assert np.all(v[1:] <= v[:-1] * (1 + 1e-6))
    gp.close()


def test_too_small_a_shortlist_is_not_certified():
    g = problem(32, 1, 100, 3, 5000)
    gp = b.r3_gp_fit(dev(g["X"]), dev(g["y"]), g["ell"], g["sf2"], g["sn2"])
    idx, val, cert = b.r3_gp_propose(gp, dev(g["Xcand"]), 64, shortlist=64)
    assert not cert[0]                       # all 64 shortlisted get picked: the last EI is far below the bound
    assert sorted(idx.cpu().numpy()[0].tolist()) == sorted(b.r3_topk(b.r3_gp_score(gp, dev(g["Xcand"]))[2], 64)[0]
                                                           .cpu().numpy()[0].tolist())
    idx, val, cert = b.r3_gp_propose(gp, dev(g["Xcand"]), 8, lie="liar")
    assert not cert[0]                       # the liar moves means: a shortlist is a heuristic
    gp.close()


def test_workload_config_1():
    c = w.get_config(1)
    g = w.generate(c)
    gp = b.r3_gp_fit(dev(g["X"]), dev(g["y"]), g["ell"], g["sf2"], g["sn2"])
    idx, val, cert = b.r3_gp_propose(gp, dev(g["Xcand"]), c.k, shortlist=1023)
    b.r3_gp_check(gp)
    assert cert[0]
    assert check_sequence(g, 0, idx.cpu().numpy()[0], val.cpu().numpy()[0], c.k, "believer") == c.k
    gp.close()


def test_errors():
    g = problem(33, 1, 30, 3, 100, sn2=0.0)
    gp = b.r3_gp_fit(dev(g["X"]), dev(g["y"]), g["ell"], g["sf2"], g["sn2"])
    for q, sl in ((0, 0), (101, 0), (10, 5), (10, 2000)):
        with pytest.raises(b.R3Error) as e:
            b.r3_gp_propose(gp, dev(g["Xcand"]), q, shortlist=sl)
        assert e.value.status == 1
    # zero noise is fine as long as no pick duplicates an observation
    idx, val, cert = b.r3_gp_propose(gp, dev(g["Xcand"]), 3)
    b.r3_gp_check(gp)
    assert check_sequence(g, 0, idx.cpu().numpy()[0], val.cpu().numpy()[0], 3, "believer") == 3
    # a pool whose best candidate IS an observation, with zero noise: nothing to condition on
    pool = g["Xcand"].copy()
    pool[0, 0] = g["X"][0, int(np.argmin(g["y"][0]))]
    mu, sd, ei = (t.cpu().numpy()[0] for t in b.r3_gp_score(gp, dev(pool)))
    if ei[0] >= ei.max():
        with pytest.raises(b.R3Error) as e:
            b.r3_gp_propose(gp, dev(pool), 2)
        assert e.value.status == 3
        b.r3_gp_check(gp)        # the handle stays usable
    gp.close()
