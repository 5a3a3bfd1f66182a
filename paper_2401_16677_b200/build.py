"""Builds the C-ABI library in-tree with nvcc for sm_100a (cross-compiles without a GPU).

Two variants come from the same sources:
  libt3.so     portable: clusters of two CTAs, every CTA fetches its own operands
  libt3_sf.so  additionally holds the 4-CTA-cluster kernel in which two CTA pairs share each fetch of a
               W tile; built only when csrc/tma_shared_fetch.cuh is present (that file and this library
               are left out of multi-GPU runs; the binding then loads libt3.so)
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libt3.so")
LIB_SF = os.path.join(HERE, "libt3_sf.so")
SHARED_FETCH_SRC = os.path.join(CSRC, "tma_shared_fetch.cuh")
SOURCES = ["t3_api.cu"]
DEPS = ["t3_api.cu", "kernels.cuh", "ptx.cuh", "schedule.h", os.path.join("..", "..", "include", "t3.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC", "-shared",
    "-cudart", "static",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _stale(lib: str, deps) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(d) > t for d in deps)


def is_stale() -> bool:
    deps = [os.path.join(CSRC, d) for d in DEPS]
    if _stale(LIB, deps):
        return True
    return os.path.exists(SHARED_FETCH_SRC) and _stale(LIB_SF, deps + [SHARED_FETCH_SRC])


def _compile(out: str, extra, verbose: bool) -> None:
    tmp = out + f".tmp{os.getpid()}"
    cmd = [_nvcc()] + NVCC_FLAGS + list(extra) + (["-Xptxas", "-v"] if verbose else []) + \
          ["-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, out)


def _multi_process_launch() -> bool:
    for key in ("WORLD_SIZE", "LOCAL_WORLD_SIZE"):
        try:
            if int(os.environ.get(key, "1")) > 1:
                return True
        except ValueError:
            return True
    return False


def build(force: bool = False, verbose: bool = False) -> str:
    """Builds what is stale (everything with force); returns the path of the portable library.
    A rank of a multi-process launch builds (and later loads) the portable library only."""
    deps = [os.path.join(CSRC, d) for d in DEPS]
    if force or _stale(LIB, deps):
        _compile(LIB, [], verbose)
    if _multi_process_launch():
        return LIB
    if os.path.exists(SHARED_FETCH_SRC):
        if force or _stale(LIB_SF, deps + [SHARED_FETCH_SRC]):
            _compile(LIB_SF, ["-DT3_TMA_SHARED_FETCH"], verbose)
    elif os.path.exists(LIB_SF):
        os.remove(LIB_SF)          # never keep a variant whose source is gone
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
