"""Build the CUDA library in-tree: ``python -m paper_2602_02071_b200.build``.

Compiles ``csrc/baps_lib.cu`` (one translation unit that includes every kernel) for sm_100a into
``paper_2602_02071_b200/libbaps.so``.  nvcc cross-compiles, so no GPU is needed to build.
"""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libbaps.so")
# Second build of the same sources for the wait test only: every bounded device-side wait gives up
# after 1 ms instead of 2 s, and the TMA producer can be told to leave one tile load out.  Nothing
# but tests/test_gpu_wait_timeout.py loads it.
WAIT_TEST_LIB = os.path.join(_HERE, "libbaps_waittest.so")
WAIT_TEST_FLAGS = ["-DBAPS_WAIT_LIMIT_NS=1000000ull", "-DBAPS_TEST_SKIP_LOAD=1"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v",
]


def _sources():
    out = [os.path.join(_HERE, "..", "include", "baps.h")]
    for name in sorted(os.listdir(CSRC)):
        if name.endswith((".cu", ".cuh", ".h")):
            out.append(os.path.join(CSRC, name))
    return out


def _compile(lib: str, extra_flags, log_name: str, force: bool, verbose: bool) -> str:
    newest = max(os.path.getmtime(p) for p in _sources())
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= newest:
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc, *NVCC_FLAGS, *extra_flags, "-o", lib, os.path.join(CSRC, "baps_lib.cu")]
    res = subprocess.run(cmd, capture_output=True, text=True)
    log = res.stdout + res.stderr
    with open(os.path.join(_HERE, log_name), "w") as f:
        f.write(" ".join(cmd) + "\n" + log)
    if verbose or res.returncode != 0:
        sys.stderr.write(log)
    if res.returncode != 0:
        raise RuntimeError(f"nvcc failed building {os.path.basename(lib)} (see {log_name})")
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the library if it is missing or older than any source; return its path."""
    extra = os.environ.get("BAPS_NVCC_EXTRA", "").split()       # developer switch, e.g. -DNAME=1
    return _compile(LIB, extra, "build.log", force, verbose)


def build_wait_test(force: bool = False, verbose: bool = False) -> str:
    """Compile the wait-test build of the library (see WAIT_TEST_LIB)."""
    return _compile(WAIT_TEST_LIB, WAIT_TEST_FLAGS, "build_waittest.log", force, verbose)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
    print(build_wait_test(force="--force" in sys.argv, verbose=False))
