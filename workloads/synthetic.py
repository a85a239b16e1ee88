"""Seeded synthetic workloads shaped like the paper's evaluation inputs.

The paper evaluates on a SIFT1M DiskANN-style on-disk graph index with 10,000
queries and recall@10 (Section 5.1, "Environment" and "Benchmark").  That dataset
is not available here, so every input is a seeded synthetic stand-in that takes
the workload's shape only: N, d, element type, out-degree, query count, K.

Everything here is input construction.  Heavy steps (kNN graph, PQ training,
ground truth) run through torch on whichever device is given; for uint8 data all
distances are integers below 2**24, so fp32 matmuls are exact and the results
are identical on CPU and GPU.

Recipes (numpy ``default_rng`` = PCG64; seeds: data 0, queries 1, random edges 2,
PQ 3):

* u8 vectors: ``centers = uniform(32, 224, (C, d))``; ``assign = integers(0, C, N)``;
  rows in chunks of 65,536: ``clip(rint(centers[assign] + 20 * standard_normal), 0, 255)``.
* f32 vectors: ``centers = 2 * standard_normal((C, d))`` stored fp32 (variance 4);
  rows in chunks of 2**20: ``centers[assign] + standard_normal(fp32)``.
* graph: exact k nearest other nodes by (distance, id), over all nodes or inside
  the node's generator cluster, followed by ``n_rand`` uniform random targets
  (self, duplicates and kNN members rejected; optionally same-cluster targets too).
* page store: node i lives in page ``i // npp`` at byte ``(i % npp) * node_bytes``;
  a node is ``vector[d]``, ``degree`` (u32 LE), ``R`` neighbour ids (u32 LE, unused
  entries 0xFFFFFFFF); page tails are zero.
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np
import torch

PAGE_BYTES = 4096
INVALID_ID = 0xFFFFFFFF


# --------------------------------------------------------------------------- vectors
def _u8_rows(rng, centers, assign, sigma=20.0, chunk=65536):
    n, d = assign.shape[0], centers.shape[1]
    out = np.empty((n, d), dtype=np.uint8)
    for s in range(0, n, chunk):
        a = assign[s:s + chunk]
        x = centers[a] + sigma * rng.standard_normal((a.shape[0], d))
        out[s:s + chunk] = np.clip(np.rint(x), 0, 255).astype(np.uint8)
    return out


def gen_u8(N, C, nq, d=128, seed_data=0, seed_q=1):
    """uint8 Gaussian-cluster vectors and queries. Returns (data, assign, queries)."""
    rng = np.random.default_rng(seed_data)
    centers = rng.uniform(32.0, 224.0, (C, d))
    assign = rng.integers(0, C, N)
    data = _u8_rows(rng, centers, assign)
    rq = np.random.default_rng(seed_q)
    aq = rq.integers(0, C, nq)
    queries = _u8_rows(rq, centers, aq)
    return data, assign.astype(np.int64), queries


def _f32_rows(rng, centers, assign, chunk=1 << 20):
    n, d = assign.shape[0], centers.shape[1]
    out = np.empty((n, d), dtype=np.float32)
    for s in range(0, n, chunk):
        a = assign[s:s + chunk]
        out[s:s + chunk] = centers[a] + rng.standard_normal((a.shape[0], d), dtype=np.float32)
    return out


def gen_f32(N, C, nq, d=96, seed_data=0, seed_q=1):
    """float32 Gaussian-cluster vectors and queries. Returns (data, assign, queries)."""
    rng = np.random.default_rng(seed_data)
    centers = (2.0 * rng.standard_normal((C, d))).astype(np.float32)
    assign = rng.integers(0, C, N)
    data = _f32_rows(rng, centers, assign)
    rq = np.random.default_rng(seed_q)
    aq = rq.integers(0, C, nq)
    queries = _f32_rows(rq, centers, aq)
    return data, assign.astype(np.int64), queries


# --------------------------------------------------------------------------- graph
def _pairwise_sq(xb: torch.Tensor, y: torch.Tensor, yn: torch.Tensor) -> torch.Tensor:
    """Squared L2 between the rows of xb and y (fp32). Exact for uint8-valued inputs."""
    xn = (xb * xb).sum(1, keepdim=True)
    return xn + yn[None, :] - 2.0 * (xb @ y.T)


def _group_knn(x: torch.Tensor, k: int, integer: bool, max_elems=1 << 24) -> torch.Tensor:
    """k nearest *other* rows of x for every row, ordered by (distance, row index).

    Returns int64 [M, kk] with kk = min(k, M-1).
    """
    M = x.shape[0]
    kk = min(k, M - 1)
    if kk <= 0:
        return torch.empty((M, 0), dtype=torch.int64, device=x.device)
    yn = (x * x).sum(1)
    rows_per = max(1, max_elems // M)
    out = torch.empty((M, kk), dtype=torch.int64, device=x.device)
    ar = torch.arange(M, device=x.device)
    for s in range(0, M, rows_per):
        e = min(M, s + rows_per)
        D = _pairwise_sq(x[s:e], x, yn)
        if integer:
            key = D.round().to(torch.int64) * M + ar[None, :]
            key[ar[: e - s], ar[s:e]] = torch.iinfo(torch.int64).max  # no self edge
            sel = torch.topk(key, kk, dim=1, largest=False, sorted=True).values
            out[s:e] = sel % M
        else:
            D[ar[: e - s], ar[s:e]] = float("inf")
            order = torch.sort(D, dim=1, stable=True).indices  # ties keep index order
            out[s:e] = order[:, :kk]
    return out


def _random_edges(N, knn, deg_knn, n_rand, seed, assign, cross_only, device, chunk=1 << 16):
    """n_rand uniform random targets per node, rejecting self, duplicates, kNN members
    (and same-cluster targets when cross_only). Draw order: rows in chunks of 65,536,
    n_rand + 8 draws per row, first n_rand valid draws kept."""
    rng = np.random.default_rng(seed)
    extra = n_rand + 8
    out = np.full((N, n_rand), INVALID_ID, dtype=np.uint32)
    cnt = np.zeros(N, dtype=np.int64)
    if n_rand == 0:
        return out, cnt
    assign_t = torch.as_tensor(assign, device=device) if assign is not None else None
    short_rows = []
    for s in range(0, N, chunk):
        e = min(N, s + chunk)
        cand = torch.as_tensor(rng.integers(0, N, (e - s, extra)), device=device)
        rows = torch.arange(s, e, device=device)
        bad = cand == rows[:, None]
        if cross_only:
            bad |= assign_t[cand] == assign_t[rows][:, None]
        kn = torch.as_tensor(knn[s:e].astype(np.int64), device=device)
        bad |= (cand[:, :, None] == kn[:, None, :]).any(2)
        # duplicate of an earlier draw in the same row
        eq = cand[:, :, None] == cand[:, None, :]
        earlier = torch.tril(torch.ones(extra, extra, dtype=torch.bool, device=device), -1)
        bad |= (eq & earlier[None]).any(2)
        order = torch.sort(bad.to(torch.int8), dim=1, stable=True).indices[:, :n_rand]
        picked = torch.gather(cand, 1, order)
        ok = ~torch.gather(bad, 1, order)
        c = ok.sum(1)
        picked = torch.where(ok, picked, torch.full_like(picked, INVALID_ID))
        out[s:e] = picked.cpu().numpy().astype(np.uint32)
        cnt[s:e] = c.cpu().numpy()
        short_rows.extend((s + np.nonzero(cnt[s:e] < n_rand)[0]).tolist())
    # rare rows (or tiny inputs) that ran out of valid draws: sample the allowed set
    for r in short_rows:
        have = set(out[r, : cnt[r]].tolist())
        banned = set(knn[r, : deg_knn[r]].tolist()) | have | {r}
        allowed = [t for t in range(N) if t not in banned
                   and not (cross_only and assign[t] == assign[r])]
        rr = np.random.default_rng([seed, r])
        need = min(n_rand - cnt[r], len(allowed))
        if need > 0:
            pick = rr.choice(len(allowed), size=need, replace=False)
            out[r, cnt[r]: cnt[r] + need] = np.asarray(allowed, dtype=np.uint32)[pick]
            cnt[r] += need
    return out, cnt


def knn_graph(data, k, n_rand, groups=None, seed=2, cross_only=False, device=None):
    """Navigation graph: exact k-NN by (distance, id) + n_rand random edges.

    groups=None searches all nodes; otherwise an int array assigning every node to a
    group and neighbours are searched inside the node's own group.
    Returns (deg uint32 [N], nbrs uint32 [N, k + n_rand], unused = 0xFFFFFFFF).
    """
    device = device or ("cuda" if torch.cuda.is_available() else "cpu")
    N = data.shape[0]
    R = k + n_rand
    integer = data.dtype == np.uint8
    knn = np.full((N, k), INVALID_ID, dtype=np.uint32)
    deg_knn = np.zeros(N, dtype=np.int64)
    if groups is None:
        member_lists = [np.arange(N)]
    else:
        order = np.argsort(groups, kind="stable")
        bounds = np.searchsorted(groups[order], np.arange(int(groups.max()) + 2))
        member_lists = [order[bounds[g]:bounds[g + 1]] for g in range(len(bounds) - 1)]
    for idx in member_lists:
        if idx.shape[0] == 0:
            continue
        x = torch.as_tensor(data[idx], device=device).to(torch.float32)
        loc = _group_knn(x, k, integer).cpu().numpy()
        kk = loc.shape[1]
        knn[idx, :kk] = idx[loc].astype(np.uint32)
        deg_knn[idx] = kk
    rnd, cnt = _random_edges(N, knn, deg_knn, n_rand, seed, groups, cross_only, device)
    nbrs = np.full((N, R), INVALID_ID, dtype=np.uint32)
    deg = (deg_knn + cnt).astype(np.uint32)
    full = (deg_knn == k)
    # common case: kNN part is full -> random edges follow at column k
    nbrs[:, :k] = knn
    nbrs[full, k:] = rnd[full]
    for r in np.nonzero(~full)[0]:
        d0 = deg_knn[r]
        nbrs[r, d0:d0 + cnt[r]] = rnd[r, : cnt[r]]
    return deg, nbrs


def medoid(data, chunk=1 << 20) -> int:
    """Node closest (squared L2, float64) to the coordinate-wise mean; ties -> lowest id."""
    N = data.shape[0]
    mean = np.zeros(data.shape[1], dtype=np.float64)
    for s in range(0, N, chunk):
        mean += data[s:s + chunk].astype(np.float64).sum(0)
    mean /= N
    best, best_id = np.inf, 0
    for s in range(0, N, chunk):
        d = ((data[s:s + chunk].astype(np.float64) - mean) ** 2).sum(1)
        j = int(np.argmin(d))
        if d[j] < best:
            best, best_id = float(d[j]), s + j
    return best_id


# --------------------------------------------------------------------------- page store
def node_bytes(d, dtype, R):
    esz = 1 if np.dtype(dtype) == np.uint8 else 4
    return d * esz + 4 + 4 * R


def write_page_store(data, deg, nbrs, npp):
    """Pack nodes into 4 KB pages. Returns uint8 [n_pages, 4096]."""
    N, d = data.shape
    R = nbrs.shape[1]
    nb = node_bytes(d, data.dtype, R)
    assert npp * nb <= PAGE_BYTES, "nodes do not fit the page"
    vb = d * data.dtype.itemsize
    n_pages = (N + npp - 1) // npp
    pages = np.zeros((n_pages, PAGE_BYTES), dtype=np.uint8)
    full = N // npp
    raw_v = np.ascontiguousarray(data).view(np.uint8).reshape(N, vb)
    raw_d = np.ascontiguousarray(deg.astype("<u4")).view(np.uint8).reshape(N, 4)
    raw_n = np.ascontiguousarray(nbrs.astype("<u4")).view(np.uint8).reshape(N, 4 * R)
    if full:
        view = pages[:full, : npp * nb].reshape(full, npp, nb)
        m = full * npp
        view[:, :, :vb] = raw_v[:m].reshape(full, npp, vb)
        view[:, :, vb:vb + 4] = raw_d[:m].reshape(full, npp, 4)
        view[:, :, vb + 4:] = raw_n[:m].reshape(full, npp, 4 * R)
    for i in range(full * npp, N):
        off = (i % npp) * nb
        pages[i // npp, off:off + vb] = raw_v[i]
        pages[i // npp, off + vb:off + vb + 4] = raw_d[i]
        pages[i // npp, off + vb + 4:off + nb] = raw_n[i]
    return pages


def parse_page_store(pages, N, d, dtype, R, npp):
    """Inverse of write_page_store: returns (data, deg, nbrs)."""
    dtype = np.dtype(dtype)
    nb = node_bytes(d, dtype, R)
    vb = d * dtype.itemsize
    data = np.empty((N, d), dtype=dtype)
    deg = np.empty(N, dtype=np.uint32)
    nbrs = np.empty((N, R), dtype=np.uint32)
    for i in range(N):
        rec = pages[i // npp, (i % npp) * nb:(i % npp + 1) * nb]
        data[i] = rec[:vb].view(dtype)
        deg[i] = rec[vb:vb + 4].view("<u4")[0]
        nbrs[i] = rec[vb + 4:].view("<u4")
    return data, deg, nbrs


# --------------------------------------------------------------------------- PQ
def train_pq(data, m=32, ksub=256, seed=3, sample=65536, iters=10, device=None, chunk=1 << 16):
    """Product quantiser with centroids rounded to uint8 (so every table entry of the
    asymmetric distance is an exact integer). Returns (centroids u8 [m, ksub, dsub],
    codes u8 [N, m]); code = nearest rounded centroid, ties -> lowest index."""
    device = device or ("cuda" if torch.cuda.is_available() else "cpu")
    N, d = data.shape
    assert d % m == 0
    dsub = d // m
    rng = np.random.default_rng(seed)
    s_idx = rng.choice(N, size=min(sample, N), replace=False)
    init_idx = rng.choice(s_idx.shape[0], size=ksub, replace=s_idx.shape[0] < ksub)
    X = torch.as_tensor(data[s_idx], device=device).to(torch.float32).reshape(-1, m, dsub)
    X = X.permute(1, 0, 2).contiguous()                    # [m, S, dsub]
    cent = X[:, torch.as_tensor(init_idx, device=device), :].clone()   # [m, ksub, dsub]
    for _ in range(iters):
        D = torch.cdist(X, cent) ** 2                      # [m, S, ksub]
        a = D.argmin(2)                                    # first minimum
        onehot_sum = torch.zeros_like(cent, dtype=torch.float64)
        counts = torch.zeros((m, ksub), dtype=torch.float64, device=device)
        onehot_sum.scatter_add_(1, a[:, :, None].expand(-1, -1, dsub), X.to(torch.float64))
        counts.scatter_add_(1, a, torch.ones_like(a, dtype=torch.float64))
        new = (onehot_sum / counts.clamp(min=1)[:, :, None]).to(torch.float32)
        cent = torch.where(counts[:, :, None] > 0, new, cent)
    cent_u8 = torch.clamp(torch.round(cent), 0, 255)        # round half to even
    cn = (cent_u8 * cent_u8).sum(2)                        # [m, ksub]
    codes = np.empty((N, m), dtype=np.uint8)
    for s in range(0, N, chunk):
        xb = torch.as_tensor(data[s:s + chunk], device=device).to(torch.float32)
        xb = xb.reshape(-1, m, dsub).permute(1, 0, 2)       # [m, B, dsub]
        D = (xb * xb).sum(2, keepdim=True) + cn[:, None, :] - 2.0 * torch.bmm(xb, cent_u8.transpose(1, 2))
        codes[s:s + chunk] = D.argmin(2).T.to(torch.uint8).cpu().numpy()
    return cent_u8.to(torch.uint8).cpu().numpy(), codes


# --------------------------------------------------------------------------- ground truth
def ground_truth(data, queries, k=10, device=None, block=1 << 18):
    """Exact top-k over all nodes by (squared L2, id). Returns uint32 [nq, k]."""
    device = device or ("cuda" if torch.cuda.is_available() else "cpu")
    N = data.shape[0]
    nq = queries.shape[0]
    integer = data.dtype == np.uint8
    q = torch.as_tensor(queries, device=device).to(torch.float32)
    qn = (q * q).sum(1, keepdim=True)
    if integer:
        best = torch.full((nq, k), torch.iinfo(torch.int64).max, dtype=torch.int64, device=device)
        shift = 1 << 32
        for s in range(0, N, block):
            x = torch.as_tensor(data[s:s + block], device=device).to(torch.float32)
            D = qn + (x * x).sum(1)[None, :] - 2.0 * (q @ x.T)
            key = D.round().to(torch.int64) * shift + torch.arange(s, s + x.shape[0], device=device)[None, :]
            best = torch.topk(torch.cat([best, key], 1), k, dim=1, largest=False, sorted=True).values
        return (best % shift).cpu().numpy().astype(np.uint32)
    # fp32: shortlist by fp32 matmul, then re-rank the shortlist in float64
    short = max(64, 4 * k)
    bd = torch.full((nq, short), float("inf"), device=device)
    bi = torch.zeros((nq, short), dtype=torch.int64, device=device)
    for s in range(0, N, block):
        x = torch.as_tensor(data[s:s + block], device=device)
        D = qn + (x * x).sum(1)[None, :] - 2.0 * (q @ x.T)
        ids = torch.arange(s, s + x.shape[0], device=device)[None, :].expand(nq, -1)
        cd = torch.cat([bd, D], 1)
        ci = torch.cat([bi, ids], 1)
        sel = torch.topk(cd, min(short, cd.shape[1]), dim=1, largest=False).indices
        bd, bi = torch.gather(cd, 1, sel), torch.gather(ci, 1, sel)
    bi_np = bi.cpu().numpy()
    out = np.empty((nq, k), dtype=np.uint32)
    q64 = queries.astype(np.float64)
    for i in range(nq):
        cand = np.unique(bi_np[i])
        dd = ((data[cand].astype(np.float64) - q64[i]) ** 2).sum(1)
        order = np.lexsort((cand, dd))[:k]
        out[i] = cand[order]
    return out


def recall_at_k(ids, gt, k=10):
    """mean over queries of |ids[:k] ∩ gt[:k]| / k."""
    hit = 0
    for a, b in zip(ids[:, :k], gt[:, :k]):
        hit += len(set(a.tolist()) & set(b.tolist()))
    return hit / (k * ids.shape[0])


# --------------------------------------------------------------------------- workloads
@dataclasses.dataclass
class Workload:
    name: str
    N: int
    d: int
    dtype: str            # "u8" | "f32"
    R: int
    npp: int
    entry: int
    pages: np.ndarray     # uint8 [n_pages, 4096]
    queries: np.ndarray   # [nq, d]
    data: np.ndarray      # [N, d]  (kept for ground truth / checks)
    deg: np.ndarray
    nbrs: np.ndarray
    K: int = 10
    L: int = 64
    W: int = 4
    cache_frac: float = 1.0
    latency_us: float = 0.0
    max_outstanding: int = 256
    preload: bool = False
    pq_centroids: Optional[np.ndarray] = None   # u8 [m, 256, dsub]
    pq_codes: Optional[np.ndarray] = None       # u8 [N, m]
    gt: Optional[np.ndarray] = None

    @property
    def n_pages(self):
        return self.pages.shape[0]

    @property
    def nq(self):
        return self.queries.shape[0]

    @property
    def node_bytes(self):
        return node_bytes(self.d, np.uint8 if self.dtype == "u8" else np.float32, self.R)

    @property
    def cache_pages(self):
        return int(np.floor(self.cache_frac * self.n_pages))


def workload_key(cfg: int, N: int, npp: int, nq: int, L: int, W: int, slots: int) -> str:
    """Name of a (workload, search parameters, cache size) combination in stored result files."""
    return f"cfg{cfg}:N={N}:npp={npp}:nq={nq}:L={L}:W={W}:slots={slots}"


def make_workload(name, kind, N, C, nq, d, k, n_rand, npp, clustered_knn, cross_only,
                  with_pq=False, with_gt=True, device=None, seed_q=1, **search):
    """Generate vectors, graph, page store (and optionally PQ and ground truth)."""
    if kind == "u8":
        data, assign, queries = gen_u8(N, C, nq, d, seed_q=seed_q)
    else:
        data, assign, queries = gen_f32(N, C, nq, d, seed_q=seed_q)
    deg, nbrs = knn_graph(data, k, n_rand, groups=assign if clustered_knn else None,
                          seed=2, cross_only=cross_only, device=device)
    entry = medoid(data)
    pages = write_page_store(data, deg, nbrs, npp)
    w = Workload(name=name, N=N, d=d, dtype=kind, R=k + n_rand, npp=npp, entry=entry,
                 pages=pages, queries=queries, data=data, deg=deg, nbrs=nbrs, **search)
    if with_pq:
        w.pq_centroids, w.pq_codes = train_pq(data, m=32, device=device)
    if with_gt:
        w.gt = ground_truth(data, queries, k=w.K, device=device)
    return w


def make_config(index, scale=1.0, nq=None, device=None, with_gt=True, seed_q=1):
    """The five evaluation configurations (1-based index). ``scale`` < 1 shrinks N and the
    cluster count together so cluster sizes, degrees and page packing keep their shape."""
    def sc(x, lo=1):
        return max(lo, int(round(x * scale)))
    if index in (1, 2):
        w = make_workload(f"cfg{index}", "u8", sc(10_000, 64), 16, nq or 1000, 128, 24, 8, 1,
                          clustered_knn=False, cross_only=False, device=device, with_gt=with_gt, seed_q=seed_q,
                          K=10, L=64, W=4)
        if index == 1:
            w.cache_frac, w.preload, w.latency_us = 1.0, True, 0.0
        else:
            w.cache_frac, w.preload, w.latency_us = 0.10, False, 0.0
        return w
    if index in (3, 4):
        w = make_workload(f"cfg{index}", "u8", sc(1_000_000, 4096), sc(256, 2), nq or 10_000, 128,
                          48, 16, 10, clustered_knn=True, cross_only=True, with_pq=(index == 4),
                          device=device, with_gt=with_gt, seed_q=seed_q, K=10, L=100, W=4)
        w.cache_frac, w.preload, w.latency_us, w.max_outstanding = 0.20, False, 20.0, 256
        return w
    if index == 5:
        w = make_workload("cfg5", "f32", sc(10_000_000, 4096), sc(4096, 2), nq or 10_000, 96,
                          48, 16, 6, clustered_knn=True, cross_only=False, device=device,
                          with_gt=with_gt, seed_q=seed_q, K=10, L=128, W=4)
        w.cache_frac, w.preload, w.latency_us, w.max_outstanding = 0.10, False, 20.0, 256
        return w
    raise ValueError("config index must be 1..5")
