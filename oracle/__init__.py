"""ctypes front end of the CPU oracle (beam_oracle.c) -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this.
It shares no code with the CUDA path and never imports it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "beam_oracle.c")
_LIB = os.path.join(_HERE, "libbeam_oracle.so")
_lib = None


class _OrcIndex(ctypes.Structure):
    _fields_ = [
        ("n_nodes", ctypes.c_uint64),
        ("dim", ctypes.c_uint32),
        ("dtype", ctypes.c_uint32),
        ("max_degree", ctypes.c_uint32),
        ("npp", ctypes.c_uint32),
        ("page_bytes", ctypes.c_uint32),
        ("entry", ctypes.c_uint32),
        ("pages", ctypes.c_void_p),
        ("pq_m", ctypes.c_uint32),
        ("pq_ksub", ctypes.c_uint32),
        ("pq_cent", ctypes.c_void_p),
        ("pq_codes", ctypes.c_void_p),
    ]


def build(force: bool = False) -> str:
    """Compile beam_oracle.c with gcc into a shared library next to it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = f"{_LIB}.{os.getpid()}.tmp"      # several processes may find it stale at once: never a half-written file
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.orc_search.restype = ctypes.c_int
        lib.orc_search.argtypes = [
            ctypes.POINTER(_OrcIndex), ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32,
            ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_uint64,
            ctypes.POINTER(ctypes.c_uint64)]
        lib.orc_exact_dist.restype = ctypes.c_double
        lib.orc_exact_dist.argtypes = [ctypes.POINTER(_OrcIndex), ctypes.c_void_p, ctypes.c_uint32]
        lib.orc_adc_dist.restype = ctypes.c_uint32
        lib.orc_adc_dist.argtypes = [ctypes.POINTER(_OrcIndex), ctypes.c_void_p, ctypes.c_uint32]
        _lib = lib
    return _lib


class OracleIndex:
    """A paged node store (numpy, host) plus the entry node; optional PQ arrays."""

    def __init__(self, pages, n_nodes, dim, dtype, max_degree, npp, entry,
                 pq_centroids=None, pq_codes=None):
        self.pages = np.ascontiguousarray(pages, dtype=np.uint8)
        self.dtype = "u8" if str(dtype) in ("u8", "uint8") else "f32"
        self.n_nodes, self.dim, self.R, self.npp, self.entry = n_nodes, dim, max_degree, npp, entry
        self.pq_centroids = None if pq_centroids is None else np.ascontiguousarray(pq_centroids, dtype=np.uint8)
        self.pq_codes = None if pq_codes is None else np.ascontiguousarray(pq_codes, dtype=np.uint8)
        self.n_pages = (n_nodes + npp - 1) // npp
        d = _OrcIndex()
        d.n_nodes, d.dim, d.dtype = n_nodes, dim, 0 if self.dtype == "u8" else 1
        d.max_degree, d.npp, d.page_bytes, d.entry = max_degree, npp, 4096, entry
        d.pages = self.pages.ctypes.data
        if self.pq_centroids is not None:
            d.pq_m, d.pq_ksub = self.pq_centroids.shape[0], self.pq_centroids.shape[1]
            d.pq_cent, d.pq_codes = self.pq_centroids.ctypes.data, self.pq_codes.ctypes.data
        self._desc = d

    @classmethod
    def from_workload(cls, w, use_pq=False):
        return cls(w.pages, w.N, w.d, w.dtype, w.R, w.npp, w.entry,
                   w.pq_centroids if use_pq else None, w.pq_codes if use_pq else None)

    def _queries(self, queries):
        return np.ascontiguousarray(queries, dtype=np.uint8 if self.dtype == "u8" else np.float32)

    def search(self, queries, K, L, W, q_range=None, order_mode=0, threads=1, want_union=False):
        """Returns dict(ids [nq,K] u32, dists [nq,K] u32|f32, counters [nq,5] u32, page_union|None).

        counters columns: pages_distinct, n_iter, n_expand, n_eval, sum_deg.
        Rows outside q_range are left as 0xFFFFFFFF / 0.
        """
        lib = _load()
        q = self._queries(queries)
        nq = q.shape[0]
        b, e = q_range if q_range is not None else (0, nq)
        ids = np.full((nq, K), 0xFFFFFFFF, dtype=np.uint32)
        dists = np.zeros((nq, K), dtype=np.uint32 if self.dtype == "u8" else np.float32)
        counters = np.zeros((nq, 5), dtype=np.uint32)
        threads = max(1, min(threads, e - b))
        unions = [np.zeros(self.n_pages, dtype=np.uint8) if want_union else None for _ in range(threads)]
        bounds = np.linspace(b, e, threads + 1).astype(int)

        def run(t):
            u = unions[t]
            return lib.orc_search(ctypes.byref(self._desc), q.ctypes.data, int(bounds[t]), int(bounds[t + 1]),
                                  K, L, W, ids.ctypes.data, dists.ctypes.data, counters.ctypes.data,
                                  u.ctypes.data if u is not None else None, order_mode, None, 0, None)

        if threads == 1:
            rcs = [run(0)]
        else:
            with ThreadPoolExecutor(threads) as ex:
                rcs = list(ex.map(run, range(threads)))
        if any(rcs):
            raise RuntimeError(f"oracle search failed with status {max(rcs)}")
        union = None
        if want_union:
            union = np.zeros(self.n_pages, dtype=np.uint8)
            for u in unions:
                union |= u
        return dict(ids=ids, dists=dists, counters=counters, page_union=union)

    def search_trace(self, query, K, L, W, order_mode=0, cap=1 << 20):
        """One query with a per-iteration trace: list of (frontier ids, [(dist, id, expanded)...])."""
        lib = _load()
        q = self._queries(query).reshape(1, -1)
        ids = np.zeros((1, K), dtype=np.uint32)
        dists = np.zeros((1, K), dtype=np.uint32 if self.dtype == "u8" else np.float32)
        counters = np.zeros((1, 5), dtype=np.uint32)
        trace = np.zeros(cap, dtype=np.uint32)
        tlen = ctypes.c_uint64(0)
        rc = lib.orc_search(ctypes.byref(self._desc), q.ctypes.data, 0, 1, K, L, W, ids.ctypes.data,
                            dists.ctypes.data, counters.ctypes.data, None, order_mode,
                            trace.ctypes.data, cap, ctypes.byref(tlen))
        if rc:
            raise RuntimeError(f"oracle search failed with status {rc}")
        assert tlen.value <= cap, "trace buffer too small"
        its, p = [], 0
        while p < tlen.value:
            nf = int(trace[p]); p += 1
            front = trace[p:p + nf].tolist(); p += nf
            nl = int(trace[p]); p += 1
            lst = [tuple(int(x) for x in trace[p + 3 * i:p + 3 * i + 3]) for i in range(nl)]
            p += 3 * nl
            its.append((front, lst))
        return dict(ids=ids[0], dists=dists[0], counters=counters[0], iterations=its)

    def exact_dist(self, query, v):
        q = self._queries(query)
        return _load().orc_exact_dist(ctypes.byref(self._desc), q.ctypes.data, int(v))

    def adc_dist(self, query, v):
        q = self._queries(query)
        return _load().orc_adc_dist(ctypes.byref(self._desc), q.ctypes.data, int(v))
