"""In-tree build of the CUDA shared library (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libgorio.so")
SOURCES = ["gorio_api.cu", "search_kernels.cu", "noalloc_entry.cu"]
HEADERS = ["gorio_internal.h", os.path.join("..", "..", "include", "gorio.h")] + [
    os.path.join("device", f) for f in ("mem.cuh", "queue.cuh", "page_cache.cuh", "scoring.cuh", "arrival.cuh", "batch.cuh",
                                        "list.cuh", "pq.cuh", "scheduler.cuh")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-pthread"]


def _stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libgorio.so next to this file (nvcc cross-compiles without a GPU)."""
    if not force and not _stale():
        return LIB_PATH
    # one builder at a time: ranks of a multi-process launch may all find the library stale
    import fcntl
    with open(os.path.join(_HERE, ".build.lock"), "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        try:
            if not force and not _stale():      # another process built it while this one waited
                return LIB_PATH
            nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
            objs = []
            for src in SOURCES:
                obj = os.path.join(CSRC, src.replace(".cu", ".o"))
                cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", os.path.join(CSRC, src), "-o", obj]
                subprocess.check_call(cmd)
                objs.append(obj)
            tmp = LIB_PATH + ".tmp"
            subprocess.check_call([nvcc, "-shared", "-o", tmp] + objs + ["-lcudart"])
            os.replace(tmp, LIB_PATH)           # readers never see a half-written library
        finally:
            fcntl.flock(lock, fcntl.LOCK_UN)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
