"""Builds ``libcott.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU).

Every ``csrc/*.cu`` is compiled to an object of its own (in parallel; an object is rebuilt only
when its source, a header or the flags changed) and the objects are linked into one shared
library."""
from __future__ import annotations

import concurrent.futures
import glob
import hashlib
import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
OBJ = os.path.join(_PKG, "build")
LIB = os.path.join(_PKG, "libcott.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xptxas", "-v",
]


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers() -> list[str]:
    return (glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) +
            glob.glob(os.path.join(_ROOT, "include", "*.h")))


def _stale(target: str, deps: list[str]) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False, lib: str | None = None) -> str:
    """Compile every ``csrc/*.cu`` and link them into one shared library; returns its path."""
    lib = lib or LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    extra = os.environ.get("COTT_EXTRA_NVCC_FLAGS", "").split()
    tag = hashlib.sha1(" ".join(NVCC_FLAGS + extra).encode()).hexdigest()[:10]
    os.makedirs(OBJ, exist_ok=True)
    hdrs = _headers()
    jobs = []
    objs = []
    for src in sources():
        obj = os.path.join(OBJ, f"{os.path.splitext(os.path.basename(src))[0]}.{tag}.o")
        objs.append(obj)
        if force or _stale(obj, [src] + hdrs):
            jobs.append([nvcc, *NVCC_FLAGS, *extra, "-I", os.path.join(_ROOT, "include"), "-I", CSRC,
                         "-c", src, "-o", obj])

    def run(cmd):
        return cmd, subprocess.run(cmd, capture_output=True, text=True)

    if jobs:
        with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, len(jobs))) as pool:
            for cmd, res in pool.map(run, jobs):
                if verbose or res.returncode != 0:
                    print(res.stdout)
                    print(res.stderr)
                if res.returncode != 0:
                    raise RuntimeError("nvcc failed compiling " + cmd[-3])
    if jobs or force or _stale(lib, objs):
        res = subprocess.run([nvcc, "-shared", "-Xcompiler", "-fPIC", "-o", lib, *objs], capture_output=True, text=True)
        if verbose or res.returncode != 0:
            print(res.stdout)
            print(res.stderr)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed linking libcott.so")
    return lib


if __name__ == "__main__":
    build(force=True, verbose=True)
