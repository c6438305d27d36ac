"""Compile the CUDA sources into libsagekv.so (in-tree, next to this file) for sm_100a."""

from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsagekv.so")
LIB_CHECKED = os.path.join(HERE, "libsagekv_checked.so")   # the same interface built with -DSAGEKV_CHECKS
LIB_TRACE = os.path.join(HERE, "libsagekv_trace.so")       # built with -DSAGEKV_TRACE: timeline stamps in the decode kernel
SOURCES = ["api.cu", "score.cu", "score_static.cu", "select_compact.cu", "decode_attn.cu", "variants.cu"]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "sagekv.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checks: bool = False, trace: bool = False) -> str:
    """checks=True builds libsagekv_checked.so: every global-memory index of the kernels is range-checked and a
    violation is reported through sagekv_status instead of being executed (load it with SAGEKV_LIB=<path>)."""
    lib = LIB_TRACE if trace else (LIB_CHECKED if checks else LIB)
    if not force and not needs_build(lib):
        return lib
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", lib] + (["-DSAGEKV_TRACE"] if trace else (["-DSAGEKV_CHECKS"] if checks else [])) + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, checks="--checks" in sys.argv, trace="--trace" in sys.argv))
