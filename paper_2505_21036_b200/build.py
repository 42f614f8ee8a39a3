"""Builds librainfusion.so (sm_100a) in-tree with nvcc.  `python -m paper_2505_21036_b200.build`.

`--checked` builds librainfusion_checked.so as well: the same sources with -DRF_BOUNDS_CHECK, whose kernels check
the indices of their global-memory writes and of the schedule they read (see rf_bounds_checked in the header).
Select it with the environment variable RAINFUSION_LIBRARY=<path> (read by api.load)."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "librainfusion.so")
LIB_CHECKED = os.path.join(PKG, "librainfusion_checked.so")
SOURCES = ["rf_api.cu", "rf_mask.cu", "rf_arm.cu", "rf_attn.cu", "rf_host.cu"]
HEADERS = ["rf_common.cuh", "rf_sm100.cuh", "rf_attn_common.cuh", os.path.join("..", "..", "include", "rainfusion.h")]


def nvcc_path() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found; the CUDA path cannot be built")
    return cand


def stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    lib = LIB_CHECKED if checked else LIB
    if not force and not stale(lib):
        return lib
    cmd = [nvcc_path(), "-shared", "-Xcompiler", "-fPIC", "-O3", "-std=c++17", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib]
    if checked:
        cmd += ["-DRF_BOUNDS_CHECK"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    if "--checked" in sys.argv:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked=True))
