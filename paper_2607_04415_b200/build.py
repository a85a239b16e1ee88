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
                                        "list.cuh", "pq.cuh", "scheduler.cuh", "resident.cuh")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-pthread"]


STAMP_PATH = LIB_PATH + ".stamp"      # hash of the sources and flags the library was built from


def _source_hash() -> str:
    import hashlib
    h = hashlib.sha256(" ".join(NVCC_FLAGS).encode())
    for f in SOURCES + HEADERS:
        with open(os.path.join(CSRC, f), "rb") as fh:
            h.update(f.encode() + b"\0" + fh.read())
    return h.hexdigest()


def kernel_source_hash() -> str:
    """Hash of the device code alone (kernels and the structures they share with the host):
    what a profiler capture of a kernel's memory traffic is tied to.  Host-side edits do not
    change it."""
    import hashlib
    h = hashlib.sha256()
    for f in ["search_kernels.cu", "gorio_internal.h"] + [x for x in HEADERS if x.startswith("device")]:
        with open(os.path.join(CSRC, f), "rb") as fh:
            h.update(f.encode() + b"\0" + fh.read())
    return h.hexdigest()[:16]


def _stale() -> bool:
    """True unless the library was built from exactly these sources (file times do not survive a
    copy of the tree to another machine, contents do)."""
    if not (os.path.exists(LIB_PATH) and os.path.exists(STAMP_PATH)):
        return True
    with open(STAMP_PATH) as fh:
        return fh.read().strip() != _source_hash()


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
            with open(STAMP_PATH, "w") as fh:
                fh.write(_source_hash())
        finally:
            fcntl.flock(lock, fcntl.LOCK_UN)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
