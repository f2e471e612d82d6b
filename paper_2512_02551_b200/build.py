"""Builds ``libhgemm.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2512_02551_b200.build [--force] [--verbose] [--checked]

``--checked`` builds ``libhgemm_checked.so`` instead: the same sources with ``-DHGEMM_CHECKED=1`` (invariants tested on the
device, violations reported through the status word); the binding loads it when the environment variable ``HGEMM_LIB`` names it.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libhgemm.so")
LIB_CHECKED = os.path.join(HERE, "libhgemm_checked.so")      # the same sources with -DHGEMM_CHECKED=1 (see include/hgemm.h)
SOURCES = ["hgemm_api.cu", "hgemm_static_scratch.cu", "hgemm_planner.cpp", "hgemm_table.cpp"]
DEPS = SOURCES + ["hgemm_kernel.cuh", "hgemm_light_kernel.cuh", "hgemm_small_kernel.cuh", "ptx_sm100.cuh", "hgemm_planner.h", "hgemm_table.inc",
                  os.path.join("..", "..", "include", "hgemm.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(os.path.join(CSRC, d)) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    lib = LIB_CHECKED if checked else LIB
    if not force and not is_stale(lib):
        return lib
    tmp = lib + f".tmp{os.getpid()}"
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-o", tmp]
    if checked:
        cmd += ["-DHGEMM_CHECKED=1"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True, cwd=CSRC)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, checked="--checked" in sys.argv))
