"""Builds libtopk.so (sm_100a) in-tree with nvcc."""
from __future__ import annotations

import os
import shutil
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
# TOPK_LIBRARY selects another build of the library (for example one compiled with different tuning macros)
LIB = os.environ.get("TOPK_LIBRARY") or os.path.join(_HERE, "libtopk.so")
SOURCES = ["api.cu"]
HEADERS = sorted(f for f in os.listdir(CSRC) if f.endswith(".cuh"))   # every header api.cu may include
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: libtopk.so cannot be built")


def _stale() -> bool:
    if os.environ.get("TOPK_LIBRARY"):
        return False
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    deps.append(os.path.join(os.path.dirname(_HERE), "include", "topk.h"))
    return any(os.path.getmtime(p) > t for p in deps)


def _deps():
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    deps.append(os.path.join(os.path.dirname(_HERE), "include", "topk.h"))
    return deps


def _compile(out: str, extra=(), verbose: bool = False) -> None:
    tmp = out + ".tmp.%d" % os.getpid()
    # TOPK_NVCC_EXTRA: more flags, e.g. one of the tuning macros (-DTK_FILTER_DYN_TILES=0, -DTK_FILTER_UNROLL=5)
    extra = [*extra, *os.environ.get("TOPK_NVCC_EXTRA", "").split()]
    cmd = [_nvcc(), *NVCC_FLAGS, *extra, *(["-Xptxas", "-v"] if verbose else []), "-o", tmp,
           *[os.path.join(CSRC, s) for s in SOURCES]]
    subprocess.run(cmd, check=True, cwd=CSRC)
    os.replace(tmp, out)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the CUDA library if it is missing or older than its sources."""
    if force or _stale():
        _compile(LIB, verbose=verbose)
    return LIB


def build_phase_clock(force: bool = False) -> str:
    """The same library with the device phase clock compiled in (-DTK_PHASE_CLOCK=1), as
    libtopk_clock.so beside the ordinary one; select it with TOPK_LIBRARY (see phase_clock.py)."""
    out = os.path.join(_HERE, "libtopk_clock.so")
    if force or not os.path.exists(out) or any(os.path.getmtime(p) > os.path.getmtime(out) for p in _deps()):
        _compile(out, extra=["-DTK_PHASE_CLOCK=1"])
    return out


if __name__ == "__main__":
    print(build(force=True, verbose=True))
