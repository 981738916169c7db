"""Failure paths of the CUDA library that can be exercised without faulting a GPU.

* a device-side wait that runs out: the tensor-core kernel's bounded waits, provoked by withholding one stage
  of its operand stream under a short limit; the kernel returns by itself, the status is reported, the handle
  keeps working;
* allocation failures injected on the host; the device-memory cache across fits;
* status bits latched by one call do not leak into the next call's own checks;
* two live handles of different shapes that share a kernel instantiation.
"""
import numpy as np
import pytest

from oracle import gp_oracle as o
from paper_2604_11109_b200 import binding as b
from tests.parity import check_scores
from tests.test_gpu_parity import compare_everything, dev, fit_gpu, rand_problem

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

SHORT_LIMIT = 2_000_000     # cycles: about a millisecond


def _scores_match(g, gp, what):
    mu, sd, ei = (t.cpu().numpy() for t in b.r3_gp_score(gp, dev(g["Xcand"])))
    b.r3_gp_check(gp)
    for q, f in enumerate(o.fit_batch(g["X"], g["y"], g["ell"], g["sf2"], g["sn2"])):
        mu_r, sd_r, ei_r = o.score(f, g["Xcand"][q])
        check_scores(mu[q], sd[q], ei[q], mu_r, sd_r, ei_r, float(np.abs(g["y"][q]).max()), float(g["sf2"][q]),
                     what=what)


@pytest.mark.parametrize("n,m,chunk,pair", [
    (100, 128, 2, False),      # one pass of four chunks, one tile: the third chunk of W never arrives
    (250, 300, 0, False),      # the very first chunk is withheld; three tiles on three thread blocks
    (600, 1000, 11, False),    # three passes; the stream stops inside the second
    (300, 256, 5, True),       # the kernel that runs a tile on a cluster of two thread blocks
])
def test_a_wait_that_runs_out_is_reported_and_the_handle_stays_usable(monkeypatch, n, m, chunk, pair):
    if pair:
        monkeypatch.setenv("R3_TC_PAIR", "1")
    g = rand_problem(4000 + n, 1, n, 12, m)
    gp = fit_gpu(g, b.ENGINE_TENSOR)
    _scores_match(g, gp, "before")
    b.r3_gp_set_wait_limit(gp, SHORT_LIMIT)
    b.r3_gp_test_withhold(gp, chunk)
    b.r3_gp_score(gp, dev(g["Xcand"]))            # returns by itself: every wait is bounded
    with pytest.raises(b.R3Error) as e:
        b.r3_gp_check(gp)
    assert e.value.status == 6                    # R3_ERR_DEVICE_TIMEOUT
    # the latch is cleared, the hook was for one call, and the same handle scores correctly again
    _scores_match(g, gp, "after the timeout")
    b.r3_gp_set_wait_limit(gp, 4_000_000_000)
    _scores_match(g, gp, "default limit")
    gp.close()


def test_wait_limit_and_withhold_arguments():
    g = rand_problem(1, 1, 20, 3, 10)
    gp = fit_gpu(g)
    for bad in (0, 99_999, -5):
        with pytest.raises(b.R3Error) as e:
            b.r3_gp_set_wait_limit(gp, bad)
        assert e.value.status == 1
    with pytest.raises(b.R3Error) as e:
        b.r3_gp_test_withhold(gp, -1)
    assert e.value.status == 1
    gp.close()


def test_allocation_failure_in_fit_is_reported_and_leaves_nothing_behind():
    g = rand_problem(2, 2, 150, 10, 64)
    X, y = dev(g["X"]), dev(g["y"])
    b.r3_trim_cache()
    # count the allocations of one successful fit, then fail each of them in turn
    b.r3_test_fail_allocation(-1)
    b.r3_gp_fit(X, y, g["ell"], g["sf2"], g["sn2"]).close()
    total = b.r3_test_fail_allocation(-1)
    assert total >= 15
    for after in range(total):
        b.r3_test_fail_allocation(after)
        try:
            gp = b.r3_gp_fit(X, y, g["ell"], g["sf2"], g["sn2"])
        except b.R3Error as e:
            assert e.status == 4, f"allocation {after}: {e}"       # R3_ERR_ALLOC
            continue
        # allocations of temporaries that the fit can do without (none today) would land here
        gp.close()
    b.r3_test_fail_allocation(-1)
    gp = fit_gpu(g)
    compare_everything(g, gp, 8, "after the injected failures")
    gp.close()


def test_allocation_failure_in_append_leaves_the_handle_unchanged():
    g = rand_problem(3, 1, 200, 6, 500)
    k = 16
    gp = b.r3_gp_fit(dev(g["X"][:, :-k]), dev(g["y"][:, :-k]), g["ell"], g["sf2"], g["sn2"])
    xc = dev(g["Xcand"])
    before = [t.clone() for t in b.r3_gp_score(gp, xc)]
    xn, yn = dev(g["X"][:, -k:]), dev(g["y"][:, -k:])
    for after in (0, 3, 9):
        b.r3_test_fail_allocation(after)
        with pytest.raises(b.R3Error) as e:
            b.r3_gp_append(gp, xn, yn)
        assert e.value.status == 4
        assert b.r3_gp_size(gp) == 200 - k
        for a, c in zip(before, b.r3_gp_score(gp, xc)):
            assert torch.equal(a, c)
    b.r3_test_fail_allocation(-1)
    b.r3_gp_append(gp, xn, yn)
    assert b.r3_gp_size(gp) == 200
    compare_everything(g, gp, 8, "append after the injected failures")
    gp.close()


def test_append_after_an_unchecked_scoring_call_keeps_that_calls_latched_status():
    g = rand_problem(5, 1, 60, 4, 200)
    k = 8
    gp = b.r3_gp_fit(dev(g["X"][:, :-k]), dev(g["y"][:, :-k]), g["ell"], g["sf2"], g["sn2"])
    bad = g["Xcand"].copy()
    bad[0, 17, 2] = np.nan
    b.r3_gp_score(gp, dev(bad))                              # latches "non-finite candidate"; not checked yet
    b.r3_gp_append(gp, dev(g["X"][:, -k:]), dev(g["y"][:, -k:]))   # valid data: must succeed
    assert b.r3_gp_size(gp) == 60
    with pytest.raises(b.R3Error) as e:                      # the scoring call's problem is still reported
        b.r3_gp_check(gp)
    assert e.value.status == 2
    compare_everything(g, gp, 8, "after append")
    gp.close()


def test_freed_blocks_of_every_size_are_kept_and_given_back_on_request():
    """The device-memory cache keeps a closed handle's blocks, the small ones included (a small history's fit is
    two dozen of them), hands them to the next fit of the same shape, and returns everything on r3_trim_cache."""
    b.r3_trim_cache()
    assert b.r3_cached_bytes() == 0
    g = rand_problem(21, 1, 48, 5, 64)
    fit_gpu(g).close()
    kept = b.r3_cached_bytes()
    assert kept > 0
    gp = fit_gpu(g)                       # the same shape again: served from the cache
    assert b.r3_cached_bytes() < kept
    compare_everything(g, gp, 8, "fit from cached blocks")
    gp.close()
    assert b.r3_cached_bytes() >= kept
    big = rand_problem(22, 1, 700, 9, 64)  # blocks above 1 MiB go through the same cache
    fit_gpu(big).close()
    assert b.r3_cached_bytes() > kept + (1 << 20)
    b.r3_trim_cache()
    assert b.r3_cached_bytes() == 0
    gp = fit_gpu(g)
    compare_everything(g, gp, 8, "fit after the cache was emptied")
    gp.close()


def test_two_live_handles_that_share_a_kernel_instantiation():
    """Handles with different feature counts need different amounts of shared memory from the same kernel;
    fitting one must not take away what the other needs."""
    ga = rand_problem(11, 1, 256, 16, 700)
    gb = rand_problem(12, 1, 512, 64, 700)
    a = fit_gpu(ga, b.ENGINE_TENSOR)
    bb = fit_gpu(gb, b.ENGINE_TENSOR)
    for g, gp, what in ((ga, a, "A"), (gb, bb, "B"), (ga, a, "A again")):
        _scores_match(g, gp, what)
    c = fit_gpu(rand_problem(13, 1, 300, 128, 10), b.ENGINE_TENSOR)   # a third shape in between
    _scores_match(ga, a, "A after C")
    _scores_match(gb, bb, "B after C")
    for h in (a, bb, c):
        h.close()
