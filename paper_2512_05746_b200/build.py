"""Compile csrc/*.cu for sm_100a into libhq.so next to this file (nvcc cross-compiles without a GPU)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_DIR = os.path.dirname(os.path.abspath(__file__))
LIB = os.path.join(_DIR, "libhq.so")
SOURCES = sorted(glob.glob(os.path.join(_DIR, "csrc", "*.cu")))
HEADERS = sorted(glob.glob(os.path.join(_DIR, "csrc", "*.cuh"))) + [os.path.join(os.path.dirname(_DIR), "include", "hq.h")]


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles every csrc/*.cu to an object file (in parallel) and links them into libhq.so."""
    if not force and not stale():
        return LIB
    from concurrent.futures import ThreadPoolExecutor
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cflags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]
    if verbose:
        cflags += ["-Xptxas", "-v"]
    objdir = os.path.join(_DIR, "_build")
    os.makedirs(objdir, exist_ok=True)

    def compile_one(src: str) -> str:
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + f".{os.getpid()}.o")
        subprocess.check_call([nvcc] + cflags + ["-c", "-o", obj, src])
        return obj

    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 4)) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    tmp = LIB + f".tmp{os.getpid()}"
    try:
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "static",
                               "-o", tmp] + objs)
        os.replace(tmp, LIB)
    finally:
        for o in objs:
            if os.path.exists(o):
                os.remove(o)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
