"""In-tree build of the C-ABI CUDA library (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libstrata_moe.so")
SOURCES = ["api.cu", "layout.cu", "dispatch.cu", "combine.cu", "partition.cu", "collective.cu", "rowmap.cu", "expert.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-Wall", "-cudart", "static"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _deps():
    out = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    inc = os.path.join(ROOT, "include")
    out.extend(os.path.join(inc, f) for f in os.listdir(inc))
    return out


# The same sources with the test hooks compiled in and a short limit on every bounded device wait: used
# only by the test of the time-out path (tests/test_gpu_timeout.py), never by the product path.
TEST_HOOKS_LIB = os.path.join(HERE, "libstrata_moe_testhooks.so")
TEST_HOOKS_DEFINES = ["-DSTRATA_TEST_HOOKS", "-DSTRATA_WAIT_LIMIT=2000"]


def stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(d) > t for d in _deps())


def _compile(lib: str, defines, verbose: bool) -> str:
    cmd = [_nvcc(), *NVCC_FLAGS, *defines, "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-shared",
           *[os.path.join(CSRC, s) for s in SOURCES], "-o", lib + ".tmp"]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
        print(" ".join(cmd), file=sys.stderr)
    subprocess.run(cmd, check=True)
    os.replace(lib + ".tmp", lib)
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libstrata_moe.so next to this file; returns its path."""
    if not force and not stale():
        return LIB
    return _compile(LIB, [], verbose)


def build_test_hooks(force: bool = False) -> str:
    """Compile the test-hooks variant (see TEST_HOOKS_LIB); returns its path."""
    if not force and not stale(TEST_HOOKS_LIB):
        return TEST_HOOKS_LIB
    return _compile(TEST_HOOKS_LIB, TEST_HOOKS_DEFINES, False)


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
    if "--test-hooks" in sys.argv:
        print(build_test_hooks(force=True))
