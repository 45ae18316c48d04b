"""Build the CUDA library in-tree with nvcc for sm_100a.

``python -m paper_2008_01425_b200.build`` (or ``build()``) compiles
``csrc/*.cu`` / ``csrc/*.cpp`` into ``paper_2008_01425_b200/libpowergossip.so``.
nvcc cross-compiles, so no GPU is needed to build.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libpowergossip.so")
LIB_CHECKED = os.path.join(HERE, "libpowergossip_checked.so")     # the same sources with -DPG_BOUNDS_CHECK

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--shared",
    "-DPG_BUILDING_LIBRARY",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")) + glob.glob(os.path.join(CSRC, "*.cpp")))


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(INCLUDE, "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile the library if it is missing or older than its sources.

    checked=True builds the bounds-checked variant beside it (libpowergossip_checked.so): every
    kernel verifies the address ranges it is about to touch against the workspace section they
    belong to and raises PG_ERR_BOUNDS instead of touching anything outside.  Load it by pointing
    the PG_LIBRARY environment variable at it before the binding is imported.
    """
    lib = LIB_CHECKED if checked else LIB
    if not force and not _stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = lib + ".%d.tmp" % os.getpid()
    extra = ["-DPG_BOUNDS_CHECK"] if checked else []
    cmd = [nvcc] + NVCC_FLAGS + extra + ["-I", INCLUDE, "-I", CSRC, "-o", tmp] + sources()
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
        print(" ".join(cmd))
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
