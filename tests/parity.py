"""Tolerance rules used by the GPU parity tests and the smoke check.

mu, sigma: relative 1e-4, with an absolute floor for values that cross zero:
    |d mu|    <= 1e-4 |mu_ref|    + 1e-6 max|y|
    |d sigma| <= 1e-4 sigma_ref   + 1e-6 sqrt(signal_var)
EI: absolute 1e-5 * max(EI_ref) over the compared set -- but never below the smallest normal FP32 number:
    the library returns EI in FP32, and a pool whose largest EI is 1e-160 (every candidate hopeless) cannot be
    resolved to 1e-165 in that type; such values come back as 0.
top-k: with tol = 1e-5 * max(EI_ref): if the oracle's gap between rank k and k+1 exceeds tol the index
sets must be equal; otherwise every chosen index must have EI_ref >= EI_ref[rank k] - tol.  A position
may differ from the oracle's only if the two oracle values differ by <= tol.
"""
import numpy as np

MU_REL, MU_ABS = 1e-4, 1e-6
SIGMA_REL, SIGMA_ABS = 1e-4, 1e-6
EI_REL_OF_MAX = 1e-5
EI_ABS_FLOOR = float(np.finfo(np.float32).tiny)   # 1.18e-38: EI is an FP32 output


def check_scores(mu, sigma, ei, mu_ref, sigma_ref, ei_ref, y_absmax, sf2, ei_max=None, what=""):
    mu, sigma, ei = (np.asarray(a, dtype=np.float64) for a in (mu, sigma, ei))
    emax = float(np.max(ei_ref)) if ei_max is None else float(ei_max)
    tol_mu = MU_REL * np.abs(mu_ref) + MU_ABS * y_absmax
    tol_sd = SIGMA_REL * sigma_ref + SIGMA_ABS * np.sqrt(sf2)
    tol_ei = max(EI_REL_OF_MAX * emax, EI_ABS_FLOOR)
    bad_mu = np.abs(mu - mu_ref) > tol_mu
    bad_sd = np.abs(sigma - sigma_ref) > tol_sd
    bad_ei = np.abs(ei - ei_ref) > tol_ei
    msg = []
    for name, bad, got, ref, tol in (("mu", bad_mu, mu, mu_ref, tol_mu), ("sigma", bad_sd, sigma, sigma_ref, tol_sd),
                                     ("ei", bad_ei, ei, ei_ref, np.broadcast_to(tol_ei, ei.shape))):
        if bad.any():
            j = int(np.argmax(np.abs(got - ref) / np.maximum(tol, 1e-300)))
            msg.append(f"{what} {name}: {int(bad.sum())}/{bad.size} outside tolerance; worst at {j}: "
                       f"got {got.flat[j]!r} ref {ref.flat[j]!r} tol {tol.flat[j]!r}")
    assert not msg, "\n".join(msg)
    return {
        "mu_err_over_tol": float(np.max(np.abs(mu - mu_ref) / tol_mu)),
        "sigma_err_over_tol": float(np.max(np.abs(sigma - sigma_ref) / tol_sd)),
        "ei_err_over_tol": float(np.max(np.abs(ei - ei_ref)) / tol_ei) if tol_ei > 0 else 0.0,
    }


def check_topk(idx, ei_ref_of, ref_idx, ref_val, ref_next_val, ei_max, what=""):
    """idx: the k indices chosen by the GPU; ei_ref_of(i) -> oracle EI of candidate i;
    ref_idx/ref_val: the oracle's top-k; ref_next_val: the oracle's value at rank k+1 (or -inf)."""
    idx = np.asarray(idx, dtype=np.int64)
    k = idx.size
    tol = max(EI_REL_OF_MAX * float(ei_max), EI_ABS_FLOOR)
    assert len(set(idx.tolist())) == k, f"{what}: repeated index in top-k"
    kth = float(ref_val[k - 1])
    if kth - float(ref_next_val) > tol:
        assert set(idx.tolist()) == set(np.asarray(ref_idx).tolist()), f"{what}: top-k set differs from the oracle's"
    vals = np.array([ei_ref_of(int(i)) for i in idx])
    assert np.all(vals >= kth - tol), f"{what}: a chosen candidate is more than tol below the oracle's rank-k value"
    for p in range(k):
        if idx[p] != ref_idx[p]:
            assert abs(vals[p] - float(ref_val[p])) <= tol, f"{what}: position {p} differs beyond tolerance"
