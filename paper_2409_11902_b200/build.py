"""Builds libac.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Every .cu file is compiled to an object of its own (in parallel, and only when it or a header is
newer than the object), then the objects are linked into the shared library.
"""
from __future__ import annotations

import glob
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "_build")
LIB = os.path.join(PKG, "libac.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return (glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh"))
            + [os.path.join(ROOT, "include", "ac.h"), os.path.abspath(__file__)])


def _newer(deps, target) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(f) > t for f in deps)


def _obj(src: str) -> str:
    return os.path.join(OBJ, os.path.basename(src)[:-3] + ".o")


def build_library(force: bool = False, verbose: bool = False) -> str:
    srcs, hdrs = sources(), _headers()
    todo = [s for s in srcs if force or _newer([s] + hdrs, _obj(s))]
    if not todo and not _newer([_obj(s) for s in srcs], LIB):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ, exist_ok=True)
    base = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else [])
    base += ["-I", os.path.join(ROOT, "include"), "-I", CSRC]

    def compile_one(src):
        subprocess.run(base + ["-c", src, "-o", _obj(src)], check=True)

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        list(pool.map(compile_one, todo))
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", LIB]
                   + [_obj(s) for s in srcs] + ["-lcuda"], check=True)
    return LIB


if __name__ == "__main__":
    import sys
    print(build_library(force=True, verbose="-v" in sys.argv))
