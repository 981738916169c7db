"""Builds ``libr3gp.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2604_11109_b200.build [--force] [--verbose] [--check]

The shared object is written beside this file so that it travels with the source
tree; nothing is installed and no JIT cache is used.  ``--check`` builds
``libr3gp_check.so`` instead: the same sources with ``-DR3_BOUNDS_CHECK``, in which the
scoring, guard and top-k kernels verify their shared-memory, tensor-memory and global
indices and report a violation through the handle's status instead of faulting (the
stand-in for compute-sanitizer; ``R3_LIB_VARIANT=check`` makes the binding load it).
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libr3gp.so")
LIB_CHECK = os.path.join(HERE, "libr3gp_check.so")
SOURCES = ["r3_api.cu", "r3_fit.cu", "r3_score_simt.cu", "r3_rescue.cu", "r3_score_tc.cu", "r3_score_tc2.cu", "r3_topk.cu",
           "r3_tpe.cu", "r3_alloc.cu", "r3_propose.cu", "r3_lml.cu", "r3_optimize.cu",
           "r3_driver.cu"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "r3.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False, check: bool = False) -> str:
    """Compile every .cu of the library for sm_100a and link ``libr3gp.so`` (``check``: the bounds-checking
    build ``libr3gp_check.so``); returns its path."""
    lib = LIB_CHECK if check else LIB
    if not force and not _stale(lib):
        return lib
    objdir = os.path.join(HERE, "build", "check" if check else "")
    os.makedirs(objdir, exist_ok=True)
    common = ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"),
              "-I", CSRC] + ARCH
    if check:
        common += ["-DR3_BOUNDS_CHECK"]
    if verbose:
        common += ["-Xptxas", "-v"]
    procs = []
    for src in SOURCES:
        obj = os.path.join(objdir, src.replace(".cu", ".o"))
        cmd = [_nvcc(), "-c", os.path.join(CSRC, src), "-o", obj] + common
        procs.append((src, obj, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    objs = []
    for src, obj, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode:
            sys.stderr.write(f"== {src}\n{out}\n")
        if p.returncode:
            raise RuntimeError(f"nvcc failed on {src}")
        objs.append(obj)
    tmp = lib + f".tmp{os.getpid()}"
    link = [_nvcc(), "-shared", "-o", tmp] + objs + ARCH
    r = subprocess.run(link, capture_output=True, text=True)
    if r.returncode:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError("link failed")
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, check="--check" in sys.argv))
