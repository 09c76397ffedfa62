"""Builds libpp.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Every .cu under csrc/ is compiled to an object of its own (in parallel, only when it or a header
is newer than the object) and the objects are linked into libpp.so next to this file."""
from __future__ import annotations

import glob
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libpp.so")
LIB_DEBUG = os.path.join(HERE, "libpp_dbg.so")  # the same sources with -DPP_DEBUG_BOUNDS

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC", "--fmad=false", "-I", os.path.join(ROOT, "include"),
]


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def headers() -> list[str]:
    return glob.glob(os.path.join(CSRC, "*.cuh")) + [os.path.join(ROOT, "include", "pp.h")]


def _newer(deps, target) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def stale() -> bool:
    return _newer(sources() + headers(), LIB)


def _build(lib: str, suffix: str, extra: list[str], force: bool, verbose: bool) -> str:
    if not (force or _newer(sources() + headers(), lib)):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    if not os.path.exists(nvcc):
        nvcc = "nvcc"
    os.makedirs(OBJ, exist_ok=True)
    jobs, objs = [], []
    for src in sources():
        obj = os.path.join(OBJ, os.path.basename(src)[:-3] + suffix + ".o")
        objs.append(obj)
        if force or _newer([src] + headers(), obj):
            cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", "-o", obj, src]
            jobs.append((cmd, subprocess.Popen(cmd)))
    for cmd, proc in jobs:
        if proc.wait() != 0:
            raise subprocess.CalledProcessError(proc.returncode, cmd)
    subprocess.run([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib] + objs, check=True)
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libpp.so.  nvcc cross-compiles without a GPU."""
    return _build(LIB, "", [], force, verbose)


def build_debug(force: bool = False) -> str:
    """The bounds-checking build of the same sources, libpp_dbg.so: every index into the state table
    and the rank table is checked, a violation sets the device error word instead of trapping."""
    return _build(LIB_DEBUG, "_dbg", ["-DPP_DEBUG_BOUNDS"], force, False)


if __name__ == "__main__":
    import sys
    print(build(force="-f" in sys.argv or "-v" in sys.argv, verbose="-v" in sys.argv))
