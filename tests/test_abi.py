"""The C-ABI library loads on a machine without a GPU and exports every symbol the header declares;
host-side argument validation works without touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2604_11109_b200 import binding as b

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "r3.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(r3_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound():
    lib = b.load()
    names = _declared_symbols()
    assert "r3_gp_fit" in names and "r3_gp_score" in names and "r3_topk" in names
    for name in names:
        assert hasattr(lib, name), f"{name} declared in r3.h but not exported"
        assert name in b.SIGNATURES, f"{name} has no ctypes signature"
        assert hasattr(b, name), f"{name} has no Python wrapper of the same name"
    assert set(b.SIGNATURES) == set(names)


def test_version_and_status_strings():
    assert b.r3_version() >= 100
    seen = {b.r3_status_string(s) for s in range(8)}
    assert len(seen) == 8 and "ok" in seen


def test_fit_rejects_bad_arguments_on_the_host():
    lib = b.load()
    out = ctypes.c_void_p(1)
    one = np.ones(4, dtype=np.float32).ctypes.data_as(ctypes.POINTER(ctypes.c_float))
    assert lib.r3_gp_fit(None, None, None, None, None, 1, 1, 1, None, ctypes.byref(out)) == 1
    assert out.value is None
    assert "NULL" in b.r3_last_error()
    fake = ctypes.c_void_p(16)  # never dereferenced: validation fails first
    assert lib.r3_gp_fit(fake, fake, one, one, one, 1, 0, 1, None, ctypes.byref(out)) == 1
    assert lib.r3_gp_fit(fake, fake, one, one, one, 1, 1, 100000, None, ctypes.byref(out)) == 1
    neg = np.array([-1.0], dtype=np.float32).ctypes.data_as(ctypes.POINTER(ctypes.c_float))
    assert lib.r3_gp_fit(fake, fake, neg, one, one, 1, 4, 1, None, ctypes.byref(out)) == 1
    assert "lengthscale" in b.r3_last_error()
    assert lib.r3_gp_fit(fake, fake, one, neg, one, 1, 4, 1, None, ctypes.byref(out)) == 1
    assert lib.r3_gp_fit(fake, fake, one, one, neg, 1, 4, 1, None, ctypes.byref(out)) == 1


def test_topk_and_score_reject_bad_arguments_on_the_host():
    lib = b.load()
    fake = ctypes.c_void_p(16)
    assert lib.r3_topk(None, 1, 10, 1, fake, None, None, 0, None) == 1
    assert lib.r3_topk(fake, 1, 10, 11, fake, None, None, 0, None) == 1       # k > m
    assert lib.r3_topk(fake, 1, 10000, 1025, fake, None, None, 0, None) == 1  # k > 1024
    assert lib.r3_topk(fake, 0, 10, 1, fake, None, None, 0, None) == 1
    assert lib.r3_gp_score(None, fake, 1, fake, fake, fake, None) == 1
    assert lib.r3_gp_check(None, None) == 1
    assert lib.r3_topk_scratch_bytes(1, 1 << 20, 128) >= 2 * 256 * 128 * 8
    lib.r3_gp_free(None)  # no-op


def test_no_device_means_an_error_not_a_fallback():
    torch = pytest.importorskip("torch")
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    lib = b.load()
    out = ctypes.c_void_p()
    x = np.zeros(4, dtype=np.float32)
    ones = np.ones(4, dtype=np.float32)
    fp = ctypes.POINTER(ctypes.c_float)
    st = lib.r3_gp_fit(ctypes.c_void_p(x.ctypes.data), ctypes.c_void_p(x.ctypes.data), ones.ctypes.data_as(fp),
                       ones.ctypes.data_as(fp), ones.ctypes.data_as(fp), 1, 4, 1, None, ctypes.byref(out))
    assert st in (4, 5) and out.value is None


def test_launch_counter():
    b.r3_launch_count_reset()
    assert b.r3_launch_count() == 0
