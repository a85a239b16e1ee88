"""Pins for the CPU oracle: everything here checks oracle/beam_oracle.c against something
other than itself -- closed forms, a hand-worked example, brute force, textbook special
cases and an independent set-form restatement."""
import os

import numpy as np
import pytest

from oracle import OracleIndex
from workloads import (make_config, node_bytes, parse_page_store, train_pq, write_page_store)
from helpers import (INVALID, adjacency, brute_topk, greedy_w1, random_graph, reachable,
                     ring_index, setform_search, sqdist)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "ring8.txt")


def _index(data, deg, nbrs, npp, entry, **kw):
    pages = write_page_store(data, deg, nbrs, npp)
    dt = "u8" if data.dtype == np.uint8 else "f32"
    return OracleIndex(pages, data.shape[0], data.shape[1], dt, nbrs.shape[1], npp, entry, **kw)


# ------------------------------------------------------------------ distances (closed forms)
def test_u8_distance_extremes_and_zero():
    d = 128
    data = np.zeros((3, d), dtype=np.uint8)
    data[1] = 255
    data[2] = np.arange(d) % 256
    deg = np.zeros(3, dtype=np.uint32)
    nbrs = np.full((3, 2), INVALID, dtype=np.uint32)
    ix = _index(data, deg, nbrs, 3, 0)
    assert ix.exact_dist(np.zeros(d, np.uint8), 1) == 128 * 255 * 255 == 8323200
    assert ix.exact_dist(np.full(d, 255, np.uint8), 0) == 8323200
    assert ix.exact_dist(data[2], 2) == 0
    assert ix.exact_dist(np.zeros(d, np.uint8), 2) == sum(i * i for i in range(d))


def test_distances_match_numpy_on_random_vectors():
    rng = np.random.default_rng(7)
    for dt, d, npp in ((np.uint8, 128, 10), (np.float32, 96, 6)):
        N = 50
        data = (rng.integers(0, 256, (N, d)).astype(np.uint8) if dt == np.uint8
                else rng.standard_normal((N, d)).astype(np.float32) * 3)
        q = data[::-1][:5].copy() if dt == np.uint8 else rng.standard_normal((5, d)).astype(np.float32)
        deg = np.zeros(N, dtype=np.uint32)
        nbrs = np.full((N, 64), INVALID, dtype=np.uint32)
        ix = _index(data, deg, nbrs, npp, 0)
        for qi in range(5):
            for v in (0, 9, 10, 11, 49):
                ref = ((q[qi].astype(np.float64) - data[v].astype(np.float64)) ** 2).sum()
                got = ix.exact_dist(q[qi], v)
                if dt == np.uint8:
                    assert got == ref
                else:
                    assert abs(got - ref) <= 1e-12 * ref


# ------------------------------------------------------------------ hand-worked example
def _golden_cases():
    cases, cur = [], None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tag, rest = line.split(None, 1)
        if tag == "case":
            name, K, L, W, npp = rest.split()
            cur = dict(name=name, K=int(K), L=int(L), W=int(W), npp=int(npp), iters=[])
            cases.append(cur)
        elif tag == "iter":
            f, l = rest.split("|")
            cur["iters"].append(([int(x) for x in f.split()],
                                 [tuple(int(y) for y in e.split(":")) for e in l.split()]))
        elif tag == "result":
            cur["result"] = [tuple(int(y) for y in e.split(":")) for e in rest.split()]
        elif tag == "counters":
            cur["counters"] = [int(x) for x in rest.split()]
    return cases


@pytest.mark.parametrize("case", _golden_cases(), ids=lambda c: c["name"])
def test_ring8_worked_example(case):
    coords = [10 * i for i in range(8)]
    if case["name"] == "tie":
        coords[7] = 60
    data, deg, nbrs, pages = ring_index(coords, d=4, npp=case["npp"])
    ix = OracleIndex(pages, 8, 4, "u8", 2, case["npp"], 3)
    q = np.zeros(4, dtype=np.uint8)
    q[0] = 62
    out = ix.search_trace(q, case["K"], case["L"], case["W"])
    assert [(int(i), int(d)) for i, d in zip(out["ids"], out["dists"])] == case["result"]
    assert out["counters"].tolist() == case["counters"]
    if case["iters"]:
        assert out["iterations"] == case["iters"]


# ------------------------------------------------------------------ brute force / exhaustive limit
@pytest.mark.parametrize("W", [1, 2, 4, 7])
def test_exhaustive_list_returns_exact_topk_over_reachable_set(W):
    rng = np.random.default_rng(100 + W)
    N, d, R, npp, K = 600, 16, 6, 10, 10
    data = rng.integers(0, 256, (N, d)).astype(np.uint8)
    deg, nbrs = random_graph(rng, N, R)
    entry = 17
    ix = _index(data, deg, nbrs, npp, entry)
    adj = adjacency(deg, nbrs)
    reach = reachable(adj, entry)
    assert 1 < len(reach) <= N
    queries = rng.integers(0, 256, (8, d)).astype(np.uint8)
    out = ix.search(queries, K, N, W)
    for qi in range(8):
        ref = brute_topk(data, queries[qi], reach, K)
        assert [(int(dd), int(i)) for i, dd in zip(out["ids"][qi], out["dists"][qi])] == ref
        assert out["counters"][qi, 3] == len(reach)                       # every reachable node scored
        assert out["counters"][qi, 2] == len(reach)                       # ... and expanded
        assert out["counters"][qi, 0] == len({v // npp for v in reach})   # distinct pages


def test_fp32_exhaustive_matches_brute_force():
    rng = np.random.default_rng(5)
    N, d, R, npp, K = 300, 96, 64, 6, 10
    data = rng.standard_normal((N, d)).astype(np.float32)
    deg, nbrs = random_graph(rng, N, R, min_deg=3)
    ix = _index(data, deg, nbrs, npp, 0)
    reach = reachable(adjacency(deg, nbrs), 0)
    queries = rng.standard_normal((4, d)).astype(np.float32)
    out = ix.search(queries, K, N, 4)
    for qi in range(4):
        ref = brute_topk(data, queries[qi], reach, K)
        assert out["ids"][qi].tolist() == [i for _, i in ref]
        np.testing.assert_allclose(out["dists"][qi], [dd for dd, _ in ref], rtol=1e-6)


@pytest.mark.parametrize("L,W", [(5, 1), (12, 3), (40, 4)])
def test_complete_graph_scores_every_node(L, W):
    rng = np.random.default_rng(9)
    N, d, K = 40, 8, 5
    data = rng.integers(0, 256, (N, d)).astype(np.uint8)
    deg = np.full(N, N - 1, dtype=np.uint32)
    nbrs = np.array([[j for j in range(N) if j != i] for i in range(N)], dtype=np.uint32)
    entry = 11
    ix = _index(data, deg, nbrs, 1, entry)
    queries = rng.integers(0, 256, (6, d)).astype(np.uint8)
    out = ix.search(queries, K, L, W)
    for qi in range(6):
        ref = brute_topk(data, queries[qi], range(N), N)
        assert [(int(dd), int(i)) for i, dd in zip(out["ids"][qi], out["dists"][qi])] == ref[:K]
        assert out["counters"][qi, 3] == N
        entry_in_top = (sqdist(queries[qi], data[entry]), entry) in ref[:L]
        assert out["counters"][qi, 2] == (L if entry_in_top or L >= N else L + 1)


def test_short_results_are_padded():
    data, deg, nbrs, pages = ring_index([0, 10, 20], d=4, npp=1)
    deg[:] = 0                                   # isolate every node: only the entry is reachable
    pages = write_page_store(data, deg, nbrs, 1)
    ix = OracleIndex(pages, 3, 4, "u8", 2, 1, 1)
    out = ix.search(np.zeros((1, 4), np.uint8), 3, 3, 2)
    assert out["ids"][0].tolist() == [1, INVALID, INVALID]
    assert out["dists"][0].tolist() == [100, INVALID, INVALID]


def test_corrupt_store_is_an_error():
    data, deg, nbrs, pages = ring_index([0, 10, 20, 30], d=4, npp=1)
    nbrs[2, 0] = 99                              # neighbour id >= N
    pages = write_page_store(data, deg, nbrs, 1)
    with pytest.raises(RuntimeError):
        OracleIndex(pages, 4, 4, "u8", 2, 1, 0).search(np.zeros((1, 4), np.uint8), 1, 4, 1)
    nbrs[2, 0] = 1
    deg[1] = 3                                   # degree > R
    pages = write_page_store(data, deg, nbrs, 1)
    with pytest.raises(RuntimeError):
        OracleIndex(pages, 4, 4, "u8", 2, 1, 0).search(np.zeros((1, 4), np.uint8), 1, 4, 1)


# ------------------------------------------------------------------ W = 1 is textbook greedy search
def test_w1_equals_heap_based_greedy_search():
    rng = np.random.default_rng(21)
    N, d, R, L = 800, 12, 8, 25
    data = rng.integers(0, 64, (N, d)).astype(np.uint8)      # small range -> many distance ties
    deg, nbrs = random_graph(rng, N, R, min_deg=2)
    ix = _index(data, deg, nbrs, 7, 3)
    adj = adjacency(deg, nbrs)
    queries = rng.integers(0, 64, (10, d)).astype(np.uint8)
    out = ix.search(queries, L, L, 1)
    for qi in range(10):
        ref = greedy_w1(data, adj, 3, queries[qi], L)
        got = [(int(dd), int(i)) for i, dd in zip(out["ids"][qi], out["dists"][qi]) if i != INVALID]
        assert got == ref


# ------------------------------------------------------------------ independent restatement + invariants
@pytest.fixture(scope="module")
def small_cfgs():
    return {
        "cfg1": make_config(1, scale=0.3, nq=40),
        "cfg3": make_config(3, scale=0.01, nq=40),
        "cfg5": make_config(5, scale=0.001, nq=30),
    }


@pytest.mark.parametrize("name", ["cfg1", "cfg3", "cfg5"])
def test_matches_setform_restatement_and_invariants(small_cfgs, name):
    w = small_cfgs[name]
    ix = OracleIndex.from_workload(w)
    out = ix.search(w.queries, w.K, w.L, w.W, want_union=True)
    adj = adjacency(w.deg, w.nbrs)
    union = set()
    for qi in range(w.nq):
        ranked, seen, expanded, n_iter = setform_search(w.data, adj, w.entry, w.queries[qi],
                                                        w.K, w.L, w.W, w.npp)
        ids = out["ids"][qi].tolist()
        assert ids == [v for _, v in ranked[:w.K]]
        c = out["counters"][qi]
        pages = {v // w.npp for v in seen}
        union |= pages
        assert c[0] == len(pages)
        assert c[1] == n_iter and c[2] == len(expanded) and c[3] == len(seen)
        assert c[4] == sum(int(w.deg[u]) for u in expanded)
        if w.npp == 1:
            assert c[0] == c[3]
        # reported distances equal recomputed ones; output strictly increasing in key
        dd = out["dists"][qi]
        for k, v in enumerate(ids):
            ref = sqdist(w.queries[qi], w.data[v])
            if w.dtype == "u8":
                assert int(dd[k]) == ref
            else:
                assert dd[k] == np.float32(ref)
        keys = [(sqdist(w.queries[qi], w.data[v]), v) for v in ids]
        assert keys == sorted(keys) and len(set(ids)) == len(ids)
        assert set(ids) <= set(expanded)          # every returned entry was expanded
    assert int(out["page_union"].sum()) == len(union)


@pytest.mark.parametrize("mode", [1, 2])
def test_processing_order_does_not_change_results(small_cfgs, mode):
    for name in ("cfg1", "cfg3", "cfg5"):
        w = small_cfgs[name]
        ix = OracleIndex.from_workload(w)
        a = ix.search(w.queries, w.K, w.L, w.W)
        b = ix.search(w.queries, w.K, w.L, w.W, order_mode=mode)
        assert (a["ids"] == b["ids"]).all() and (a["dists"] == b["dists"]).all()
        assert (a["counters"] == b["counters"]).all()


def test_threads_do_not_change_results(small_cfgs):
    w = small_cfgs["cfg3"]
    ix = OracleIndex.from_workload(w)
    a = ix.search(w.queries, w.K, w.L, w.W)
    b = ix.search(w.queries, w.K, w.L, w.W, threads=4)
    assert (a["ids"] == b["ids"]).all() and (a["counters"] == b["counters"]).all()


# ------------------------------------------------------------------ PQ navigation
@pytest.fixture(scope="module")
def pq_small():
    w = make_config(3, scale=0.01, nq=30)
    w.pq_centroids, w.pq_codes = train_pq(w.data, m=32, sample=4096, iters=4)
    return w


def test_adc_equals_distance_to_reconstruction(pq_small):
    w = pq_small
    ix = OracleIndex.from_workload(w, use_pq=True)
    m, dsub = 32, w.d // 32
    rng = np.random.default_rng(3)
    for qi in range(5):
        for v in rng.integers(0, w.N, 20):
            recon = np.concatenate([w.pq_centroids[j, w.pq_codes[v, j]] for j in range(m)])
            assert recon.shape[0] == m * dsub
            assert ix.adc_dist(w.queries[qi], int(v)) == sqdist(w.queries[qi], recon.astype(np.uint8))


def test_pq_search_matches_setform_restatement(pq_small):
    w = pq_small
    ix = OracleIndex.from_workload(w, use_pq=True)
    adj = adjacency(w.deg, w.nbrs)
    recon = np.stack([w.pq_centroids[j, w.pq_codes[:, j]] for j in range(32)], 1).reshape(w.N, w.d)
    for L, W in ((50, 1), (100, 4), (60, 8)):
        out = ix.search(w.queries, w.K, L, W)
        for qi in range(w.nq):
            q = w.queries[qi]
            _, seen, expanded, n_iter = setform_search(w.data, adj, w.entry, q, w.K, L, W, w.npp,
                                                       keyfn=lambda v: sqdist(q, recon[v]))
            pool = sorted((sqdist(q, w.data[u]), u) for u in expanded)[:w.K]
            got = [(int(dd), int(i)) for i, dd in zip(out["dists"][qi], out["ids"][qi])]
            assert [(dd, i) for dd, i in zip(out["dists"][qi].tolist(), out["ids"][qi].tolist())] == \
                   [(dd, i) for dd, i in pool] + [(INVALID, INVALID)] * (w.K - len(pool))
            c = out["counters"][qi]
            assert c[0] == len({u // w.npp for u in expanded})
            assert c[1] == n_iter and c[2] == len(expanded) and c[3] == len(seen)
            del got


def test_pq_on_codebook_points_equals_exact_search():
    """If every node equals its own reconstruction, PQ navigation must return exactly the
    exact-navigation result."""
    rng = np.random.default_rng(11)
    m, ksub, dsub, N, R = 32, 256, 4, 1500, 12
    cent = rng.integers(0, 256, (m, ksub, dsub)).astype(np.uint8)
    codes = rng.integers(0, ksub, (N, m)).astype(np.uint8)
    data = np.stack([cent[j, codes[:, j]] for j in range(m)], 1).reshape(N, m * dsub)
    deg, nbrs = random_graph(rng, N, R, min_deg=4)
    pages = write_page_store(data, deg, nbrs, 9)
    exact = OracleIndex(pages, N, m * dsub, "u8", R, 9, 5)
    pq = OracleIndex(pages, N, m * dsub, "u8", R, 9, 5, pq_centroids=cent, pq_codes=codes)
    q = rng.integers(0, 256, (12, m * dsub)).astype(np.uint8)
    a = exact.search(q, 10, 40, 4)
    b = pq.search(q, 10, 40, 4)
    assert (a["ids"] == b["ids"]).all() and (a["dists"] == b["dists"]).all()
    assert (a["counters"][:, 1:] == b["counters"][:, 1:]).all()     # same walk; pages differ by design


# ------------------------------------------------------------------ page store
@pytest.mark.parametrize("npp,dt,d,R", [(1, np.uint8, 128, 32), (10, np.uint8, 128, 64), (6, np.float32, 96, 64)])
def test_page_store_round_trip(npp, dt, d, R):
    rng = np.random.default_rng(1)
    N = 10 * npp + 3                                  # last page is partial
    data = (rng.integers(0, 256, (N, d)).astype(np.uint8) if dt == np.uint8
            else rng.standard_normal((N, d)).astype(np.float32))
    deg, nbrs = random_graph(rng, N, R)
    pages = write_page_store(data, deg, nbrs, npp)
    nb = node_bytes(d, dt, R)
    assert pages.shape == ((N + npp - 1) // npp, 4096)
    assert not pages[:, npp * nb:].any()              # page tails are zero
    d2, g2, n2 = parse_page_store(pages, N, d, dt, R, npp)
    assert (d2 == data).all() and (g2 == deg).all() and (n2 == nbrs).all()
    # the oracle reads vector, degree and ids from the same offsets
    ix = OracleIndex(pages, N, d, "u8" if dt == np.uint8 else "f32", R, npp, 0)
    v = N - 1
    assert ix.exact_dist(data[v], v) == 0
