"""ctypes binding of include/gorio.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

EXPORTED_SYMBOLS = [
    "gorio_index_open", "gorio_cache_config", "gorio_set_tuning", "gorio_search", "gorio_search_host",
    "gorio_stats", "gorio_stats_reset", "gorio_index_close", "gorio_status_str", "gorio_last_error",
    "gorio_search_resident_noalloc", "gorio_link_probe",
]

STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "CUDA", 3: "NOMEM", 4: "STATE", 5: "TIMEOUT",
                6: "CAPACITY", 7: "INDEX_CORRUPT", 8: "INTERNAL"}


class GorioError(RuntimeError):
    def __init__(self, status, detail=""):
        self.status = status
        super().__init__(f"gorio status {status} ({STATUS_NAMES.get(status, '?')}): {detail}")


class _IndexDesc(ctypes.Structure):
    _fields_ = [("n_nodes", ctypes.c_uint64), ("dim", ctypes.c_uint32), ("dtype", ctypes.c_uint32),
                ("max_degree", ctypes.c_uint32), ("nodes_per_page", ctypes.c_uint32),
                ("page_bytes", ctypes.c_uint32), ("entry_id", ctypes.c_uint32),
                ("host_pages", ctypes.c_void_p), ("pq_m", ctypes.c_uint32), ("flags", ctypes.c_uint32),
                ("pq_centroids_dev", ctypes.c_void_p), ("pq_codes_dev", ctypes.c_void_p)]


class _CacheCfg(ctypes.Structure):
    _fields_ = [("capacity_pages", ctypes.c_uint64), ("remote_latency_ns", ctypes.c_uint32),
                ("max_outstanding", ctypes.c_uint32), ("preload", ctypes.c_uint32),
                ("timeout_ms", ctypes.c_uint32), ("granularity", ctypes.c_uint32),
                ("copy_mode", ctypes.c_uint32)]


class _Tuning(ctypes.Structure):
    _fields_ = [("max_inflight", ctypes.c_uint32), ("visited_capacity", ctypes.c_uint32),
                ("warps_per_block", ctypes.c_uint32), ("blocks_per_sm", ctypes.c_uint32),
                ("stash_entries", ctypes.c_uint32), ("blocking", ctypes.c_uint32),
                ("request_backlog", ctypes.c_uint32), ("no_fast_path", ctypes.c_uint32),
                ("shared_pull", ctypes.c_uint32)]


_STAT_FIELDS = ["pages_hit", "pages_missed", "pages_fetched", "dedupe_joins", "evictions", "retries",
                "max_outstanding_seen", "queries_done", "n_eval", "n_expand", "sum_degree", "n_iter",
                "resumes", "search_ns", "proxy_batches", "posted", "proxy_service_ns", "proxy_iters",
                "proxy_ack_wait_iters", "proxy_window_full_iters", "proxy_ring_empty_iters",
                "proxy_outstanding_sum", "warp_ns_arrivals", "warp_ns_queries", "warp_ns_idle",
                "arrivals_consumed", "warp_ns_copies", "stash_hits", "fetched_bytes"]


class Stats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint64) for n in _STAT_FIELDS]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n in _STAT_FIELDS}


def lib_path() -> str:
    """libgorio.so next to this file, or the build named by $GORIO_LIB (to compare two builds)."""
    return os.environ.get("GORIO_LIB") or os.path.join(_HERE, "libgorio.so")


def load_library():
    """Load libgorio.so; raises if it has not been built (no fallback exists)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = lib_path()
    if not os.path.exists(path):
        raise GorioError(2, f"{path} is missing: build it with `python -m paper_2607_04415_b200.build`")
    lib = ctypes.CDLL(path)
    vp, u32 = ctypes.c_void_p, ctypes.c_uint32
    lib.gorio_index_open.argtypes = [ctypes.POINTER(_IndexDesc), ctypes.c_int, ctypes.POINTER(vp)]
    lib.gorio_cache_config.argtypes = [vp, ctypes.POINTER(_CacheCfg)]
    lib.gorio_set_tuning.argtypes = [vp, ctypes.POINTER(_Tuning)]
    lib.gorio_search.argtypes = [vp, vp, u32, u32, u32, u32, vp, vp, vp, vp, vp]
    lib.gorio_search_host.argtypes = [vp, vp, u32, u32, u32, u32, vp, vp, vp, vp]
    lib.gorio_search_resident_noalloc.argtypes = [ctypes.POINTER(_IndexDesc), vp, vp, u32, u32, u32, u32, vp, vp, vp, vp]
    lib.gorio_stats.argtypes = [vp, ctypes.POINTER(Stats)]
    lib.gorio_stats_reset.argtypes = [vp]
    lib.gorio_link_probe.argtypes = [vp, u32, u32, ctypes.c_int, vp, ctypes.POINTER(ctypes.c_double)]
    lib.gorio_index_close.argtypes = [vp]
    lib.gorio_status_str.argtypes = [ctypes.c_int]
    lib.gorio_status_str.restype = ctypes.c_char_p
    lib.gorio_last_error.argtypes = [vp]
    lib.gorio_last_error.restype = ctypes.c_char_p
    for name in EXPORTED_SYMBOLS:
        if name not in ("gorio_status_str", "gorio_last_error"):
            getattr(lib, name).restype = ctypes.c_int
    _LIB = lib
    return lib


def _invalid(msg):
    return GorioError(1, msg)


def check_queries(queries, dim: int, dtype: str, device_index: Optional[int] = None):
    """Shape, element type, layout and placement of a query tensor, checked before its raw
    pointer goes to the library (which cannot see any of them): [nq, dim], uint8 or float32 as
    the index, contiguous, on the index's CUDA device."""
    want = torch.uint8 if dtype == "u8" else torch.float32
    if not isinstance(queries, torch.Tensor) or queries.dim() != 2:
        raise _invalid("queries must be a 2-D torch tensor [nq, dim]")
    if queries.shape[1] != dim:
        raise _invalid(f"queries have {queries.shape[1]} columns, the index has dim {dim}")
    if queries.dtype != want:
        raise _invalid(f"queries are {queries.dtype}, the index holds {want}")
    if not queries.is_contiguous():
        raise _invalid("queries must be contiguous (row major)")
    if not queries.is_cuda:
        raise _invalid("queries must be a CUDA tensor")
    if device_index is not None and queries.device.index != device_index:
        raise _invalid(f"queries live on cuda:{queries.device.index}, the index on cuda:{device_index}")
    if queries.data_ptr() % 4 != 0:
        raise _invalid("queries must be at least 4-byte aligned")


def check_resident_pages(pages_dev, n_nodes: int, nodes_per_page: int, device):
    """The device page store handed to the allocation-free entry: uint8, contiguous, on the
    queries' device, at least 4-byte aligned and large enough for every page the index
    description implies (the kernels read the page of any neighbour id below n_nodes)."""
    if nodes_per_page < 1 or n_nodes < 1:
        raise _invalid("n_nodes and nodes_per_page must be positive")
    n_pages = (n_nodes + nodes_per_page - 1) // nodes_per_page
    if not isinstance(pages_dev, torch.Tensor) or pages_dev.dtype != torch.uint8 or not pages_dev.is_contiguous():
        raise _invalid("pages_dev must be a contiguous uint8 torch tensor")
    if not pages_dev.is_cuda or pages_dev.device != device:
        raise _invalid("pages_dev must live on the same CUDA device as the queries")
    if pages_dev.numel() < n_pages * 4096:
        raise _invalid(f"pages_dev holds {pages_dev.numel()} bytes, the index description needs {n_pages * 4096}")
    if pages_dev.data_ptr() % 4 != 0:
        raise _invalid("pages_dev must be at least 4-byte aligned")


class Index:
    """gorio_index_open / cache_config / search / stats / close with torch tensors for memory."""

    def __init__(self, pages: np.ndarray, n_nodes: int, dim: int, dtype: str, max_degree: int,
                 nodes_per_page: int, entry_id: int, device: int = 0,
                 pq_centroids: Optional[torch.Tensor] = None, pq_codes: Optional[torch.Tensor] = None,
                 already_pinned: bool = False):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        assert pages.dtype == np.uint8 and pages.flags["C_CONTIGUOUS"]
        self._pages = pages                      # borrowed by the library until close
        self._pq = (pq_centroids, pq_codes)      # keep the device tensors alive
        self.dtype = "u8" if str(dtype) in ("u8", "uint8") else "f32"
        self.dim, self.device = dim, device
        d = _IndexDesc()
        d.n_nodes, d.dim, d.dtype = n_nodes, dim, 0 if self.dtype == "u8" else 1
        d.max_degree, d.nodes_per_page, d.page_bytes, d.entry_id = max_degree, nodes_per_page, 4096, entry_id
        d.host_pages = pages.ctypes.data
        d.flags = 1 if already_pinned else 0
        if pq_centroids is not None:
            assert pq_centroids.is_cuda and pq_codes.is_cuda and pq_centroids.dtype == torch.uint8
            d.pq_m = pq_centroids.shape[0]
            d.pq_centroids_dev, d.pq_codes_dev = pq_centroids.data_ptr(), pq_codes.data_ptr()
        self._check(self._lib.gorio_index_open(ctypes.byref(d), device, ctypes.byref(self._h)), opened=False)

    @classmethod
    def from_workload(cls, w, device=0, use_pq=False, pin=False):
        """pin=True copies the page store into CUDA-allocated pinned memory first (instead of
        page-locking the numpy buffer in place)."""
        cent = codes = None
        if use_pq:
            cent = torch.as_tensor(w.pq_centroids).contiguous().cuda(device)
            codes = torch.as_tensor(w.pq_codes).contiguous().cuda(device)
        pages, keep = w.pages, None
        if pin:
            keep = torch.from_numpy(w.pages).pin_memory()
            pages = keep.numpy()
        ix = cls(pages, w.N, w.d, w.dtype, w.R, w.npp, w.entry, device, cent, codes, already_pinned=pin)
        ix._pinned_store = keep
        return ix

    def _check(self, status, opened=True):
        if status != 0:
            detail = self._lib.gorio_last_error(self._h).decode() if opened and self._h else ""
            raise GorioError(status, detail or self._lib.gorio_status_str(status).decode())

    def cache_config(self, capacity_pages, remote_latency_ns=0, max_outstanding=256, preload=False,
                     timeout_ms=0, granularity="page", copy_engine=False):
        """granularity: "page" (a miss fetches the 4 KB page) or "record" (only the wanted node's record).
        copy_engine: the proxy thread copies each page itself (one cudaMemcpyAsync per request)
        instead of commanding warps of the search kernel to pull it."""
        gran = {"page": 0, "record": 1}[granularity]
        cfg = _CacheCfg(int(capacity_pages), int(remote_latency_ns), int(max_outstanding), int(bool(preload)),
                        int(timeout_ms), gran, 1 if copy_engine else 0)
        self._check(self._lib.gorio_cache_config(self._h, ctypes.byref(cfg)))

    def set_tuning(self, max_inflight=0, visited_capacity=0, warps_per_block=0, blocks_per_sm=0, stash_entries=0,
                   blocking=0, request_backlog=0, no_fast_path=0, shared_pull=0):
        t = _Tuning(max_inflight, visited_capacity, warps_per_block, blocks_per_sm, stash_entries, int(blocking),
                    request_backlog, int(no_fast_path), int(shared_pull))
        self._check(self._lib.gorio_set_tuning(self._h, ctypes.byref(t)))

    def search(self, queries: torch.Tensor, K: int, L: int, W: int, want_counters=True, stream=None):
        """queries: CUDA tensor [nq, dim] of the index dtype.  Returns dict of CUDA tensors."""
        check_queries(queries, self.dim, self.dtype, self.device)
        nq = queries.shape[0]
        dev = queries.device
        ids = torch.empty((nq, K), dtype=torch.int32, device=dev)
        dists = torch.empty((nq, K), dtype=torch.int32 if self.dtype == "u8" else torch.float32, device=dev)
        pages = torch.empty(nq, dtype=torch.int32, device=dev)
        counters = torch.empty((nq, 5), dtype=torch.int32, device=dev) if want_counters else None
        s = stream if stream is not None else torch.cuda.current_stream(dev)
        self._check(self._lib.gorio_search(self._h, queries.data_ptr(), nq, K, L, W, ids.data_ptr(),
                                           dists.data_ptr(), pages.data_ptr(),
                                           counters.data_ptr() if want_counters else None, s.cuda_stream))
        return dict(ids=ids, dists=dists, pages_distinct=pages, counters=counters)

    def search_host(self, queries: np.ndarray, K: int, L: int, W: int, out: Optional[dict] = None):
        """Host buffers in, host buffers out (the copies happen inside the C call).  `out` may
        supply preallocated (e.g. pinned) arrays: ids, dists, pages, counters."""
        q = np.ascontiguousarray(queries)
        if q.ndim != 2 or q.shape[1] != self.dim or q.dtype != (np.uint8 if self.dtype == "u8" else np.float32):
            raise _invalid(f"queries must be [nq, {self.dim}] of the index's element type")
        nq = q.shape[0]
        out = out or {}
        ids = out.get("ids", np.empty((nq, K), dtype=np.uint32))
        dists = out.get("dists", np.empty((nq, K), dtype=np.uint32 if self.dtype == "u8" else np.float32))
        pages = out.get("pages", np.empty(nq, dtype=np.uint32))
        counters = out.get("counters", np.empty((nq, 5), dtype=np.uint32))
        self._check(self._lib.gorio_search_host(self._h, q.ctypes.data, nq, K, L, W, ids.ctypes.data,
                                                dists.ctypes.data, pages.ctypes.data, counters.ctypes.data))
        return dict(ids=ids.view(np.uint32), dists=dists if self.dtype == "f32" else dists.view(np.uint32),
                    pages_distinct=pages.view(np.uint32), counters=counters.view(np.uint32))

    def stats(self) -> dict:
        s = Stats()
        self._check(self._lib.gorio_stats(self._h, ctypes.byref(s)))
        return s.as_dict()

    def stats_reset(self):
        self._check(self._lib.gorio_stats_reset(self._h))

    def link_probe(self, n_pulls: int, pages_in_flight: int, sequential: bool = False, stream=None) -> float:
        """GB/s the host link delivers to `pages_in_flight` warps pulling 4 KB pages of the store (no search)."""
        gbs = ctypes.c_double(0.0)
        sp = ctypes.c_void_p(stream.cuda_stream) if stream is not None else None
        self._check(self._lib.gorio_link_probe(self._h, n_pulls, pages_in_flight, int(sequential), sp, ctypes.byref(gbs)))
        return gbs.value

    def close(self):
        if self._h:
            self._lib.gorio_index_close(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def search_resident_noalloc(pages_dev: torch.Tensor, n_nodes: int, dim: int, dtype: str, max_degree: int,
                            nodes_per_page: int, entry_id: int, queries: torch.Tensor, K: int, L: int, W: int,
                            stream=None):
    """gorio_search_resident_noalloc: search an index that is fully resident in device memory
    without any allocation inside the library (the result tensors are allocated here, by the
    caller's allocator, before the call).  For callers that cannot call cudaMalloc; limits
    and sharing rules are in include/gorio.h."""
    lib = load_library()
    u8 = str(dtype) in ("u8", "uint8")
    check_queries(queries, dim, "u8" if u8 else "f32")
    check_resident_pages(pages_dev, n_nodes, nodes_per_page, queries.device)
    d = _IndexDesc()
    d.n_nodes, d.dim, d.dtype = n_nodes, dim, 0 if u8 else 1
    d.max_degree, d.nodes_per_page, d.page_bytes, d.entry_id = max_degree, nodes_per_page, 4096, entry_id
    nq, dev = queries.shape[0], queries.device
    ids = torch.empty((nq, K), dtype=torch.int32, device=dev)
    dists = torch.empty((nq, K), dtype=torch.int32 if u8 else torch.float32, device=dev)
    pages = torch.empty(nq, dtype=torch.int32, device=dev)
    s = stream if stream is not None else torch.cuda.current_stream(dev)
    with torch.cuda.device(dev):
        st = lib.gorio_search_resident_noalloc(ctypes.byref(d), pages_dev.data_ptr(), queries.data_ptr(), nq, K, L, W,
                                               ids.data_ptr(), dists.data_ptr(), pages.data_ptr(), s.cuda_stream)
    if st != 0:
        raise GorioError(st, lib.gorio_last_error(None).decode())
    return dict(ids=ids, dists=dists, pages_distinct=pages)
