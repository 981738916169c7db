"""Thin Python binding of ``libr3gp.so`` (the C ABI declared in ``include/r3.h``).

Argument marshalling only: every step of the scoring path runs in the library's
CUDA kernels.  PyTorch supplies device memory (``torch.Tensor.data_ptr``) and the
current stream; there is no CPU fallback -- if the library or a CUDA device is
missing, the calls raise.

The functions carry the names of the C entry points.  Tensors passed in must be
contiguous float32 on the current CUDA device (host arrays where the C ABI says
"host").
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# R3_LIB_VARIANT=check loads the bounds-checking build of the same library (build.py --check)
LIB_PATH = os.path.join(_HERE, "libr3gp_check.so" if os.environ.get("R3_LIB_VARIANT") == "check" else "libr3gp.so")

R3_OK = 0
STATUS_NAMES = {
    0: "R3_OK", 1: "R3_ERR_INVALID_ARG", 2: "R3_ERR_NONFINITE", 3: "R3_ERR_NOT_PD", 4: "R3_ERR_ALLOC",
    5: "R3_ERR_CUDA", 6: "R3_ERR_DEVICE_TIMEOUT", 7: "R3_ERR_UNSUPPORTED",
}
ENGINE_AUTO, ENGINE_SIMT, ENGINE_TENSOR = 0, 1, 2

_lib = None

_vp, _i, _ll, _ull = ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong, ctypes.c_ulonglong
_fp = ctypes.POINTER(ctypes.c_float)

# name -> (restype, argtypes); every symbol include/r3.h declares
class BoOptions(ctypes.Structure):
    _fields_ = [("q", ctypes.c_int), ("max_rounds", ctypes.c_int), ("max_seconds", ctypes.c_double),
                ("patience", ctypes.c_int), ("optimize_every", ctypes.c_int), ("lie", ctypes.c_int),
                ("surrogate", ctypes.c_int), ("levels", ctypes.POINTER(ctypes.c_int)), ("gamma", ctypes.c_float)]


EVALUATE_FN = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.POINTER(ctypes.c_float), ctypes.c_int, ctypes.c_int,
                               ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int), ctypes.c_void_p)

SIGNATURES = {
    "r3_gp_fit": (_i, [_vp, _vp, _fp, _fp, _fp, _i, _i, _i, _vp, ctypes.POINTER(_vp)]),
    "r3_gp_score": (_i, [_vp, _vp, _ll, _vp, _vp, _vp, _vp]),
    "r3_topk": (_i, [_vp, _i, _ll, _i, _vp, _vp, _vp, _ull, _vp]),
    "r3_topk_scratch_bytes": (_ull, [_i, _ll, _i]),
    "r3_trim_cache": (None, []),
    "r3_cached_bytes": (_ull, []),
    "r3_gp_lml": (_i, [_vp, _vp, _vp, _vp]),
    "r3_bo_run": (_i, [_vp, _vp, _i, _i, _fp, ctypes.c_float, ctypes.c_float, _vp, _ll, ctypes.POINTER(BoOptions),
                       EVALUATE_FN, _vp, _fp, _fp, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int),
                       ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int), ctypes.POINTER(_vp), _vp]),
    "r3_gp_refit": (_i, [_vp, _fp, _fp, _fp, _vp]),
    "r3_gp_optimize": (_i, [_vp, _i, ctypes.c_double, _vp, _vp, _vp, _vp, ctypes.POINTER(ctypes.c_int), _vp]),
    "r3_gp_propose": (_i, [_vp, _vp, _ll, _i, _i, _i, _vp, _vp, ctypes.POINTER(ctypes.c_int), _vp]),
    "r3_gp_append": (_i, [_vp, _vp, _vp, _i, _vp]),
    "r3_gp_size": (_i, [_vp]),
    "r3_tpe_fit": (_i, [_vp, _vp, ctypes.POINTER(ctypes.c_int), _i, _i, ctypes.c_float, ctypes.c_float, _vp,
                        ctypes.POINTER(_vp)]),
    "r3_tpe_score": (_i, [_vp, _vp, _ll, _vp, _vp]),
    "r3_tpe_check": (_i, [_vp, _vp]),
    "r3_tpe_get_model": (_i, [_vp, ctypes.POINTER(ctypes.c_int), _vp, _vp, _vp, _vp]),
    "r3_tpe_free": (None, [_vp]),
    "r3_topk_noalloc": (_i, [_vp, _i, _ll, _i, _vp, _vp, _vp]),
    "r3_gp_score_topk": (_i, [_vp, _vp, _ll, _i, _vp, _vp, _vp, _vp, _vp, _vp]),
    "r3_gp_score_topk_host": (_i, [_vp, _vp, _ll, _i, _vp, _vp, _vp, _vp, _vp, _vp]),
    "r3_gp_check": (_i, [_vp, _vp]),
    "r3_gp_set_wait_limit": (_i, [_vp, _ll]),
    "r3_gp_test_withhold": (_i, [_vp, _ll]),
    "r3_test_fail_allocation": (_ll, [_ll]),
    "r3_gp_get_best": (_i, [_vp, _fp]),
    "r3_gp_set_best": (_i, [_vp, _fp]),
    "r3_gp_set_engine": (_i, [_vp, _i]),
    "r3_gp_engine": (_i, [_vp]),
    "r3_gp_get_factor": (_i, [_vp, _vp, _vp]),
    "r3_gp_last_rescued": (_i, [_vp, _vp, ctypes.POINTER(_ll)]),
    "r3_gp_tensor_info": (_i, [_vp, ctypes.POINTER(ctypes.c_int)]),
    "r3_gp_profile": (_i, [_vp, _i]),
    "r3_gp_profile_read": (_i, [_vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(_ll)]),
    "r3_launch_count": (_ull, []),
    "r3_launch_count_reset": (None, []),
    "r3_gp_free": (None, [_vp]),
    "r3_status_string": (ctypes.c_char_p, [_i]),
    "r3_last_error": (ctypes.c_char_p, []),
    "r3_version": (_i, []),
}


class R3Error(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


def load():
    """Load ``libr3gp.so``; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2604_11109_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def _check(status: int):
    if status != R3_OK:
        raise R3Error(status, load().r3_last_error().decode())


def _stream():
    import torch
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev_f32(t, name):
    import torch
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous float32 CUDA tensor")
    return ctypes.c_void_p(t.data_ptr())


def _host_f32(a, shape, name):
    a = np.ascontiguousarray(np.broadcast_to(np.asarray(a, dtype=np.float32), shape))
    return a, a.ctypes.data_as(_fp)


class GP:
    """Owner of one ``r3_gp_t*``; freed on ``close()`` or garbage collection."""

    def __init__(self, handle: int, batch: int, n: int, d: int):
        self._h = ctypes.c_void_p(handle)
        self.batch, self.n, self.d = batch, n, d

    @property
    def handle(self):
        if not self._h:
            raise ValueError("GP handle already freed")
        return self._h

    def close(self):
        if self._h:
            load().r3_gp_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def r3_gp_fit(X, y, lengthscales, signal_var, noise_var) -> GP:
    """X [batch][n][d] (or [n][d]) and y [batch][n] CUDA float32; hyper-parameters host arrays."""
    if X.dim() == 2:
        X, y = X.unsqueeze(0), y.unsqueeze(0)
    batch, n, d = X.shape
    if tuple(y.shape) != (batch, n):
        raise ValueError("y must be [batch][n]")
    ell, ell_p = _host_f32(lengthscales, (batch, d), "lengthscales")
    sf2, sf2_p = _host_f32(signal_var, (batch,), "signal_var")
    sn2, sn2_p = _host_f32(noise_var, (batch,), "noise_var")
    out = ctypes.c_void_p()
    _check(load().r3_gp_fit(_dev_f32(X, "X"), _dev_f32(y, "y"), ell_p, sf2_p, sn2_p, batch, n, d, _stream(),
                            ctypes.byref(out)))
    return GP(out.value, batch, n, d)


def _pool(gp: GP, Xcand):
    if Xcand.dim() == 2:
        Xcand = Xcand.unsqueeze(0)
    if Xcand.shape[0] != gp.batch or Xcand.shape[2] != gp.d:
        raise ValueError("Xcand must be [batch][m][d]")
    return Xcand, int(Xcand.shape[1])


def r3_gp_score(gp: GP, Xcand, out=None):
    """Returns (mu, sigma, ei), each CUDA float32 [batch][m]; asynchronous on the current stream."""
    import torch
    Xcand, m = _pool(gp, Xcand)
    mu, sigma, ei = out if out is not None else (
        torch.empty((gp.batch, m), dtype=torch.float32, device=Xcand.device) for _ in range(3))
    _check(load().r3_gp_score(gp.handle, _dev_f32(Xcand, "Xcand"), m, _dev_f32(mu, "mu"), _dev_f32(sigma, "sigma"),
                              _dev_f32(ei, "ei"), _stream()))
    return mu, sigma, ei


def r3_topk(ei, k: int, scratch=None):
    """ei CUDA float32 [batch][m] (or [m]) -> (idx int32 [batch][k], val float32 [batch][k])."""
    import torch
    squeeze = ei.dim() == 1
    if squeeze:
        ei = ei.unsqueeze(0)
    batch, m = ei.shape
    lib = load()
    idx = torch.empty((batch, k), dtype=torch.int32, device=ei.device)
    val = torch.empty((batch, k), dtype=torch.float32, device=ei.device)
    if scratch is None:
        nbytes = int(lib.r3_topk_scratch_bytes(batch, m, k))
        scratch = torch.empty(max(nbytes, 1), dtype=torch.uint8, device=ei.device)
    _check(lib.r3_topk(_dev_f32(ei, "ei"), batch, m, k, ctypes.c_void_p(idx.data_ptr()),
                       ctypes.c_void_p(val.data_ptr()), ctypes.c_void_p(scratch.data_ptr()), scratch.numel(),
                       _stream()))
    return (idx[0], val[0]) if squeeze else (idx, val)


def r3_topk_noalloc(ei, k: int, out):
    """r3_topk without any allocation: the library's fixed key array is the workspace and the caller
    supplies the outputs, out = (idx int32 [batch][k], val float32 [batch][k] or None).  For callers that
    cannot allocate device memory at call time; limited to batch * ceil(m / 4096) * k <= 65536."""
    if ei.dim() == 1:
        ei = ei.unsqueeze(0)
    batch, m = ei.shape
    idx, val = out
    _check(load().r3_topk_noalloc(_dev_f32(ei, "ei"), batch, m, k, ctypes.c_void_p(idx.data_ptr()),
                                  ctypes.c_void_p(val.data_ptr()) if val is not None else ctypes.c_void_p(), _stream()))
    return out


def r3_topk_scratch_bytes(batch: int, m: int, k: int) -> int:
    return int(load().r3_topk_scratch_bytes(int(batch), int(m), int(k)))


def r3_gp_score_topk(gp: GP, Xcand, k: int, out=None):
    """One proposal round on device buffers: returns (mu, sigma, ei, idx, val)."""
    import torch
    Xcand, m = _pool(gp, Xcand)
    if out is None:
        mu, sigma, ei = (torch.empty((gp.batch, m), dtype=torch.float32, device=Xcand.device) for _ in range(3))
        idx = torch.empty((gp.batch, k), dtype=torch.int32, device=Xcand.device)
        val = torch.empty((gp.batch, k), dtype=torch.float32, device=Xcand.device)
    else:
        mu, sigma, ei, idx, val = out
    _check(load().r3_gp_score_topk(gp.handle, _dev_f32(Xcand, "Xcand"), m, k, _dev_f32(mu, "mu"),
                                   _dev_f32(sigma, "sigma"), _dev_f32(ei, "ei"), ctypes.c_void_p(idx.data_ptr()),
                                   _dev_f32(val, "val"), _stream()))
    return mu, sigma, ei, idx, val


def r3_gp_score_topk_host(gp: GP, Xcand_host, k: int, out):
    """Host-buffer form: Xcand_host and the tensors of ``out`` = (mu, sigma, ei, idx, val) live in
    (ideally pinned) host memory; any of mu/sigma/ei/val may be None.  Synchronises."""
    m = int(Xcand_host.shape[-2])
    mu, sigma, ei, idx, val = out

    def hp(t):
        return ctypes.c_void_p(t.data_ptr()) if t is not None else ctypes.c_void_p()

    _check(load().r3_gp_score_topk_host(gp.handle, hp(Xcand_host), m, k, hp(mu), hp(sigma), hp(ei), hp(idx), hp(val),
                                        _stream()))
    return out


def r3_gp_lml(gp: GP):
    """(lml [batch], gradient [batch][d + 2] in (log lengthscales, log signal_var, log noise_var)), FP64."""
    lml = np.empty((gp.batch,), dtype=np.float64)
    grad = np.empty((gp.batch, gp.d + 2), dtype=np.float64)
    _check(load().r3_gp_lml(gp.handle, ctypes.c_void_p(lml.ctypes.data), ctypes.c_void_p(grad.ctypes.data), _stream()))
    return lml, grad


STOP_REASONS = ("max_rounds", "max_seconds", "no_improvement", "pool_exhausted", "history_full", "stopped_by_caller")


def r3_bo_run(X0, y0, lengthscales, signal_var, noise_var, pool, evaluate, q=8, max_rounds=10, max_seconds=0.0,
              patience=0, optimize_every=0, lie="believer", keep_handle=False, surrogate="gp", levels=None, gamma=0.25):
    """The whole inner search on one GP.  ``evaluate(x)`` gets a float32 array [q][d] of configurations and
    returns (y [q], valid [q]) or (y, valid, stop).  Returns a dict with best_x, best_y, rounds, evaluated,
    discarded, stop_reason (and ``gp`` when keep_handle)."""
    n0, d = X0.shape
    m = int(pool.shape[0])
    ell, ell_p = _host_f32(lengthscales, (d,), "lengthscales")
    lv = None if levels is None else np.ascontiguousarray(np.asarray(levels, dtype=np.int32))
    opts = BoOptions(int(q), int(max_rounds), float(max_seconds), int(patience), int(optimize_every),
                     {"believer": 0, "liar": 1}[lie], {"gp": 0, "tpe": 1}[surrogate],
                     None if lv is None else lv.ctypes.data_as(ctypes.POINTER(ctypes.c_int)), float(gamma))
    failure = []

    def trampoline(xp, qq, dd, yp, vp, _user):
        try:
            x = np.ctypeslib.as_array(xp, shape=(qq, dd)).copy()
            out = evaluate(x)
            y, valid = np.asarray(out[0], dtype=np.float32), np.asarray(out[1])
            for i in range(qq):
                yp[i] = float(y[i])
                vp[i] = int(bool(valid[i]))
            return int(bool(out[2])) if len(out) > 2 else 0
        except Exception as exc:  # an exception must not cross the C boundary
            failure.append(exc)
            for i in range(qq):
                vp[i] = 0      # nothing of this round enters the history
            return 1

    cb = EVALUATE_FN(trampoline)
    best_x = np.empty((d,), dtype=np.float32)
    best_y = ctypes.c_float()
    rounds, evaluated, discarded, reason = ctypes.c_int(), ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    handle = ctypes.c_void_p()
    _check(load().r3_bo_run(_dev_f32(X0, "X0"), _dev_f32(y0, "y0"), n0, d, ell_p, float(signal_var), float(noise_var),
                            _dev_f32(pool, "pool"), m, ctypes.byref(opts), cb, None, best_x.ctypes.data_as(_fp),
                            ctypes.byref(best_y), ctypes.byref(rounds), ctypes.byref(evaluated), ctypes.byref(discarded),
                            ctypes.byref(reason), ctypes.byref(handle) if keep_handle else None, _stream()))
    if failure:
        if keep_handle and handle.value:
            load().r3_gp_free(handle)
        raise failure[0]
    out = {"best_x": best_x, "best_y": float(best_y.value), "rounds": rounds.value, "evaluated": evaluated.value,
           "discarded": discarded.value, "stop_reason": STOP_REASONS[reason.value]}
    if keep_handle and handle.value:
        n = int(load().r3_gp_size(handle))
        out["gp"] = GP(handle.value, 1, n, d)
    return out


def r3_gp_refit(gp: GP, lengthscales, signal_var, noise_var):
    """Condition the handle's histories on other hyper-parameters (host arrays as for r3_gp_fit)."""
    ell, ell_p = _host_f32(lengthscales, (gp.batch, gp.d), "lengthscales")
    sf2, sf2_p = _host_f32(signal_var, (gp.batch,), "signal_var")
    sn2, sn2_p = _host_f32(noise_var, (gp.batch,), "noise_var")
    _check(load().r3_gp_refit(gp.handle, ell_p, sf2_p, sn2_p, _stream()))


def r3_gp_optimize(gp: GP, max_evals: int = 60, gtol: float = 1e-3):
    """Maximise the log marginal likelihood over the hyper-parameters: returns (lengthscales [batch][d],
    signal_var [batch], noise_var [batch], lml [batch], evaluations used)."""
    ell = np.empty((gp.batch, gp.d), dtype=np.float32)
    sf2 = np.empty((gp.batch,), dtype=np.float32)
    sn2 = np.empty((gp.batch,), dtype=np.float32)
    lml = np.empty((gp.batch,), dtype=np.float64)
    used = ctypes.c_int()
    _check(load().r3_gp_optimize(gp.handle, int(max_evals), float(gtol), ctypes.c_void_p(ell.ctypes.data),
                                 ctypes.c_void_p(sf2.ctypes.data), ctypes.c_void_p(sn2.ctypes.data),
                                 ctypes.c_void_p(lml.ctypes.data), ctypes.byref(used), _stream()))
    return ell, sf2, sn2, lml, used.value


def r3_gp_propose(gp: GP, Xcand, q: int, shortlist: int = 0, lie: str = "believer"):
    """q pool members per GP chosen greedily by fantasies: returns (idx int32 [batch][q], EI at pick time
    float32 [batch][q], certified bool [batch])."""
    import torch
    Xcand, m = _pool(gp, Xcand)
    idx = torch.empty((gp.batch, q), dtype=torch.int32, device=Xcand.device)
    val = torch.empty((gp.batch, q), dtype=torch.float32, device=Xcand.device)
    cert = (ctypes.c_int * gp.batch)()
    _check(load().r3_gp_propose(gp.handle, _dev_f32(Xcand, "Xcand"), m, int(q), int(shortlist),
                                {"believer": 0, "liar": 1}[lie], ctypes.c_void_p(idx.data_ptr()),
                                ctypes.c_void_p(val.data_ptr()), cert, _stream()))
    return idx, val, np.array([bool(c) for c in cert])


def r3_gp_append(gp: GP, Xnew, ynew):
    """Add k observations per GP: Xnew [batch][k][d] (or [k][d]) and ynew [batch][k] CUDA float32."""
    if Xnew.dim() == 2:
        Xnew, ynew = Xnew.unsqueeze(0), ynew.unsqueeze(0)
    batch, k, d = Xnew.shape
    if batch != gp.batch or d != gp.d or tuple(ynew.shape) != (batch, k):
        raise ValueError("Xnew must be [batch][k][d] and ynew [batch][k]")
    _check(load().r3_gp_append(gp.handle, _dev_f32(Xnew, "Xnew"), _dev_f32(ynew, "ynew"), k, _stream()))
    gp.n = r3_gp_size(gp)


def r3_gp_size(gp: GP) -> int:
    return int(load().r3_gp_size(gp.handle))


def r3_gp_check(gp: GP):
    _check(load().r3_gp_check(gp.handle, _stream()))


def r3_gp_set_wait_limit(gp: GP, cycles: int):
    _check(load().r3_gp_set_wait_limit(gp.handle, int(cycles)))


def r3_gp_test_withhold(gp: GP, chunk: int):
    _check(load().r3_gp_test_withhold(gp.handle, int(chunk)))


def r3_test_fail_allocation(after: int) -> int:
    return int(load().r3_test_fail_allocation(int(after)))


def r3_gp_tensor_info(gp: GP) -> dict:
    """Shape of the tensor-core engine for this handle (zeros when it does not serve it)."""
    info = (ctypes.c_int * 8)()
    _check(load().r3_gp_tensor_info(gp.handle, info))
    names = ("NV", "P", "DP", "NP", "G", "w_stages", "kstar_in_tmem", "f8_cross_terms")
    return dict(zip(names, (int(v) for v in info)))


def r3_gp_get_best(gp: GP) -> np.ndarray:
    best = np.empty(gp.batch, dtype=np.float32)
    _check(load().r3_gp_get_best(gp.handle, best.ctypes.data_as(_fp)))
    return best


def r3_gp_set_best(gp: GP, best):
    b, p = _host_f32(best, (gp.batch,), "best")
    _check(load().r3_gp_set_best(gp.handle, p))


def r3_gp_set_engine(gp: GP, engine: int):
    _check(load().r3_gp_set_engine(gp.handle, int(engine)))


def r3_gp_engine(gp: GP) -> int:
    return int(load().r3_gp_engine(gp.handle))


def r3_gp_get_factor(gp: GP):
    """(alpha [batch][n], L [batch][n][n]) as FP64 numpy arrays."""
    alpha = np.empty((gp.batch, gp.n), dtype=np.float64)
    L = np.empty((gp.batch, gp.n, gp.n), dtype=np.float64)
    _check(load().r3_gp_get_factor(gp.handle, alpha.ctypes.data_as(_vp), L.ctypes.data_as(_vp)))
    return alpha, L


def r3_gp_last_rescued(gp: GP) -> int:
    """Candidates the last scoring call recomputed in FP64 (synchronises the current stream)."""
    total = _ll()
    _check(load().r3_gp_last_rescued(gp.handle, _stream(), ctypes.byref(total)))
    return int(total.value)


def r3_gp_profile(gp: GP, enable: bool):
    _check(load().r3_gp_profile(gp.handle, 1 if enable else 0))


def r3_gp_profile_read(gp: GP):
    """(summed milliseconds of the dominant kernel, number of launches) since the last read."""
    ms, cnt = ctypes.c_double(), _ll()
    _check(load().r3_gp_profile_read(gp.handle, ctypes.byref(ms), ctypes.byref(cnt)))
    return float(ms.value), int(cnt.value)


def r3_launch_count() -> int:
    return int(load().r3_launch_count())


def r3_launch_count_reset():
    load().r3_launch_count_reset()


def r3_gp_free(gp: GP):
    gp.close()


class TPE:
    """Owner of one ``r3_tpe_t*``; freed on ``close()`` or garbage collection."""

    def __init__(self, handle: int, n: int, d: int):
        self._h = ctypes.c_void_p(handle)
        self.n, self.d = n, d

    @property
    def handle(self):
        if not self._h:
            raise ValueError("TPE handle already freed")
        return self._h

    def close(self):
        if self._h:
            load().r3_tpe_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def r3_tpe_fit(X, y, levels, gamma: float = 0.25, prior_weight: float = 1.0) -> TPE:
    """X [n][d] and y [n] CUDA float32; levels host int array [d] (0 = ordinal, C >= 2 = categorical)."""
    n, d = X.shape
    if tuple(y.shape) != (n,):
        raise ValueError("y must be [n]")
    lv = np.ascontiguousarray(np.asarray(levels, dtype=np.int32))
    if lv.shape != (d,):
        raise ValueError("levels must be [d]")
    out = ctypes.c_void_p()
    _check(load().r3_tpe_fit(_dev_f32(X, "X"), _dev_f32(y, "y"), lv.ctypes.data_as(ctypes.POINTER(ctypes.c_int)), n, d,
                             float(gamma), float(prior_weight), _stream(), ctypes.byref(out)))
    return TPE(out.value, n, d)


def r3_tpe_score(tpe: TPE, Xcand, out=None):
    """Log-density ratio of every candidate: Xcand [m][d] CUDA float32 -> score [m]."""
    import torch
    m, d = Xcand.shape
    if d != tpe.d:
        raise ValueError("Xcand must be [m][d]")
    if out is None:
        out = torch.empty((m,), dtype=torch.float32, device=Xcand.device)
    _check(load().r3_tpe_score(tpe.handle, _dev_f32(Xcand, "Xcand"), m, _dev_f32(out, "score"), _stream()))
    return out


def r3_tpe_check(tpe: TPE):
    _check(load().r3_tpe_check(tpe.handle, _stream()))


def r3_tpe_get_model(tpe: TPE):
    """Host copies of the fitted model: (n_good, order [n], comps [d][n+2][4], counts [d][2], table [d][64])."""
    n_good = ctypes.c_int()
    order = np.empty((tpe.n,), dtype=np.int32)
    comps = np.empty((tpe.d, tpe.n + 2, 4), dtype=np.float32)
    counts = np.empty((tpe.d, 2), dtype=np.int32)
    table = np.empty((tpe.d, 64), dtype=np.float32)
    _check(load().r3_tpe_get_model(tpe.handle, ctypes.byref(n_good), ctypes.c_void_p(order.ctypes.data),
                                   ctypes.c_void_p(comps.ctypes.data), ctypes.c_void_p(counts.ctypes.data),
                                   ctypes.c_void_p(table.ctypes.data)))
    return n_good.value, order, comps, counts, table


def r3_tpe_free(tpe: TPE):
    tpe.close()


def r3_trim_cache():
    """Return the device memory the library keeps for reuse to the driver."""
    load().r3_trim_cache()


def r3_cached_bytes() -> int:
    return int(load().r3_cached_bytes())


def r3_version() -> int:
    return int(load().r3_version())


def r3_status_string(status: int) -> str:
    return load().r3_status_string(int(status)).decode()


def r3_last_error() -> str:
    return load().r3_last_error().decode()
