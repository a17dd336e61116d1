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


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile if the library is missing or older than any source; return its path."""
    newest = max(os.path.getmtime(p) for p in _sources())
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= newest:
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    extra = os.environ.get("BAPS_NVCC_EXTRA", "").split()       # developer switch, e.g. -DNAME=1
    cmd = [nvcc, *NVCC_FLAGS, *extra, "-o", LIB, os.path.join(CSRC, "baps_lib.cu")]
    res = subprocess.run(cmd, capture_output=True, text=True)
    log = res.stdout + res.stderr
    with open(os.path.join(_HERE, "build.log"), "w") as f:
        f.write(" ".join(cmd) + "\n" + log)
    if verbose or res.returncode != 0:
        sys.stderr.write(log)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libbaps.so (see build.log)")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
