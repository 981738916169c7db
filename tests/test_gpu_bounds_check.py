"""The bounds-checking build of the library (``build.py --check``, ``-DR3_BOUNDS_CHECK``): the scoring, guard
and top-k kernels verify their shared-memory, tensor-memory and global indices and report a violation through
the handle's status instead of faulting.  It stands in for compute-sanitizer, which is not available where the
library is developed.  The small element-by-element cases (several tiles, ragged tails in every dimension, both
engines, multi-pass histories) run against that build in a child process: every result must still match the
oracle and no index check may fire (a fired check makes ``r3_gp_check`` fail with the line of the check).
"""
import os
import subprocess
import sys

import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_cases_pass_under_the_bounds_checking_build():
    from paper_2604_11109_b200 import build
    lib = build.build(check=True)
    assert os.path.exists(lib)
    env = dict(os.environ, R3_LIB_VARIANT="check")
    which = subprocess.run([sys.executable, "-c", "from paper_2604_11109_b200 import binding as b; b.load(); print(b.LIB_PATH)"],
                           cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert which.stdout.strip().endswith("libr3gp_check.so"), which.stdout + which.stderr
    sel = "small_cases or near_observations or random_shapes or paired or wait_that_runs_out or two_live"
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"),
                        os.path.join(ROOT, "tests", "test_gpu_failure_paths.py"), "-m", "gpu", "-x", "-q", "-k", sel,
                        "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = (r.stdout + r.stderr)[-3000:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and "failed" not in r.stdout, tail
