"""Builds libssgd.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_1903_04488_b200.build [--force] [--verbose]

Every .cu under csrc/ is one translation unit; they are compiled in parallel and linked into one library.
"""
from __future__ import annotations

import concurrent.futures
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libssgd.so")
OBJ = os.path.join(HERE, "build")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-diag-suppress", "128,177",
]


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps() -> list[str]:
    return sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    return os.path.getmtime(LIB) < max(os.path.getmtime(p) for p in _deps())


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu under csrc/ and link libssgd.so (nvcc cross-compiles; no GPU needed)."""
    if force or stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        os.makedirs(OBJ, exist_ok=True)
        newest_header = max(os.path.getmtime(p) for p in _deps() if not p.endswith(".cu"))
        jobs = []
        for src in sources():
            obj = os.path.join(OBJ, os.path.basename(src)[:-3] + ".o")
            if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), newest_header):
                jobs.append([nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) +
                            ["-I", INCLUDE, "-c", "-o", obj, src])
        with concurrent.futures.ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 1))) as pool:
            for rc in pool.map(subprocess.call, jobs):
                if rc:
                    raise subprocess.CalledProcessError(rc, "nvcc")
        objs = [os.path.join(OBJ, os.path.basename(s)[:-3] + ".o") for s in sources()]
        tmp = LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp] + objs)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
