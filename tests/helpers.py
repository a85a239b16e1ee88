"""Test-only helpers: an independent set-form restatement of the search, brute force,
reachability, and tiny hand-made indexes.  Nothing here is used by the oracle or by the
CUDA path."""
from __future__ import annotations

import heapq

import numpy as np

from workloads import write_page_store

INVALID = 0xFFFFFFFF


def sqdist(q, x):
    """Squared L2 in Python ints (uint8) or float64 (fp32), straight from the definition."""
    if x.dtype == np.uint8:
        return int(((q.astype(np.int64) - x.astype(np.int64)) ** 2).sum())
    s = 0.0
    for a, b in zip(q.astype(np.float64).tolist(), x.astype(np.float64).tolist()):
        s += (a - b) * (a - b)
    return s


def adjacency(deg, nbrs):
    return [set(int(v) for v in nbrs[i, :deg[i]]) for i in range(deg.shape[0])]


def reachable(adj, entry):
    seen, stack = {entry}, [entry]
    while stack:
        u = stack.pop()
        for v in adj[u]:
            if v not in seen:
                seen.add(v)
                stack.append(v)
    return seen


def brute_topk(data, q, ids, k):
    """Exact top-k over the node set `ids` by (distance, id)."""
    keys = sorted((sqdist(q, data[i]), i) for i in ids)
    return keys[:k]


def setform_search(data, adj, entry, q, K, L, W, npp, keyfn=None):
    """Sort-everything-each-iteration restatement with Python sets.

    keyfn(v) -> navigation distance (defaults to the exact distance).  Returns
    (list of (dist, id) of length <= L, seen set, expanded list, n_iter)."""
    keyfn = keyfn or (lambda v: sqdist(q, data[v]))
    seen = {entry}
    members = {entry: keyfn(entry)}       # id -> distance, for ids currently in the list
    expanded = set()
    order_expanded = []
    n_iter = 0
    while True:
        ranked = sorted((d, v) for v, d in members.items())
        frontier = [v for d, v in ranked if v not in expanded][:W]
        if not frontier:
            break
        n_iter += 1
        expanded.update(frontier)
        order_expanded.extend(frontier)
        new = set()
        for u in frontier:
            new |= adj[u]
        new -= seen
        seen |= new
        for v in new:
            members[v] = keyfn(v)
        ranked = sorted((d, v) for v, d in members.items())[:L]
        members = {v: d for d, v in ranked}
    ranked = sorted((d, v) for v, d in members.items())
    return ranked, seen, order_expanded, n_iter


def greedy_w1(data, adj, entry, q, L):
    """Textbook greedy best-first search with a bounded result list (W = 1), heap based."""
    d0 = sqdist(q, data[entry])
    visited = {entry}
    cand = [(d0, entry)]                  # min-heap of unexpanded
    best = [(-d0, -entry)]                # max-heap (by key) of the bounded list
    in_list = {entry}
    while cand:
        d, u = heapq.heappop(cand)
        if u not in in_list:              # dropped from the bounded list meanwhile
            continue
        for v in sorted(adj[u]):
            if v in visited:
                continue
            visited.add(v)
            dv = sqdist(q, data[v])
            if len(best) < L or (dv, v) < (-best[0][0], -best[0][1]):
                heapq.heappush(best, (-dv, -v))
                in_list.add(v)
                heapq.heappush(cand, (dv, v))
                if len(best) > L:
                    _, nw = heapq.heappop(best)
                    in_list.discard(-nw)
    return sorted((-a, -b) for a, b in best)


def ring_index(coords, d=4, npp=1, R=2, dtype=np.uint8):
    """Nodes on a line (first coordinate = coords[i], others 0) with ring adjacency."""
    n = len(coords)
    data = np.zeros((n, d), dtype=dtype)
    data[:, 0] = coords
    deg = np.full(n, 2, dtype=np.uint32)
    nbrs = np.full((n, R), INVALID, dtype=np.uint32)
    for i in range(n):
        nbrs[i, 0] = (i - 1) % n
        nbrs[i, 1] = (i + 1) % n
    return data, deg, nbrs, write_page_store(data, deg, nbrs, npp)


def random_graph(rng, N, R, min_deg=1):
    deg = rng.integers(min_deg, R + 1, N).astype(np.uint32)
    nbrs = np.full((N, R), INVALID, dtype=np.uint32)
    for i in range(N):
        nbrs[i, :deg[i]] = rng.integers(0, N, deg[i])      # duplicates and self loops allowed
    return deg, nbrs


def fp32_parity(w, got, ref, rows=None):
    """The fp32 tolerance: >= 99.9 % of queries have identical ids; every other query must
    differ only by swaps or substitutions among near ties (true double distances within 1e-5
    relative, rank by rank; no duplicates; sorted within the tolerance); reported distances
    within fp32 rounding of the oracle's; counters (where the entry point reports them)
    identical wherever the ids are; recall@10 within 0.001 (when ground truth is at hand)."""
    from workloads import recall_at_k
    rows = np.arange(w.nq) if rows is None else rows
    gi, ri = got["ids"][rows], ref["ids"]
    same = (gi == ri).all(1)
    assert same.mean() >= 0.999, f"id match rate {same.mean():.5f}"
    q64 = w.queries[rows].astype(np.float64)
    for r in np.nonzero(~same)[0]:
        assert len(set(gi[r].tolist())) == gi.shape[1]
        dg = ((w.data[gi[r]].astype(np.float64) - q64[r]) ** 2).sum(1)
        do = ((w.data[ri[r]].astype(np.float64) - q64[r]) ** 2).sum(1)
        assert (np.abs(dg - do) <= 1e-5 * do).all(), f"query {rows[r]}: unexplained mismatch"
        assert (dg[1:] >= dg[:-1] * (1 - 1e-5)).all()
    np.testing.assert_allclose(got["dists"][rows][same], ref["dists"][same], rtol=2e-6)
    if got.get("counters") is not None:
        assert (got["counters"][rows][same] == ref["counters"][same]).mean() >= 0.999
    if w.gt is not None:
        assert abs(recall_at_k(gi, w.gt[rows]) - recall_at_k(ri, w.gt[rows])) <= 0.001
