"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, element by
element on the same seeded inputs.  uint8 data must match bit-exactly (ids, integer
distances, per-query counters); fp32 within the tolerance procedure below."""
import os

import numpy as np
import pytest
import torch

from oracle import OracleIndex
from helpers import fp32_parity as _fp32_parity
from workloads import make_config, make_workload, recall_at_k, train_pq, write_page_store

pytestmark = pytest.mark.gpu

THREADS = os.cpu_count() or 8      # oracle threads: every query of the full-size runs is compared


@pytest.fixture(scope="module")
def gorio():
    from paper_2607_04415_b200 import build
    build.build()
    import paper_2607_04415_b200 as g
    return g


def _u32(t):
    return t.cpu().numpy().view(np.uint32)


def _gpu_search(g, w, capacity, L=None, W=None, K=None, use_pq=False, queries=None, tuning=None, **cfg):
    ix = g.Index.from_workload(w, use_pq=use_pq)
    try:
        cfg.setdefault("timeout_ms", 60000)
        ix.cache_config(capacity, **cfg)
        if tuning:
            ix.set_tuning(**tuning)
        q = torch.as_tensor(w.queries if queries is None else queries).cuda()
        out = ix.search(q, K or w.K, L or w.L, W or w.W)
        torch.cuda.synchronize()
        res = dict(ids=_u32(out["ids"]), counters=_u32(out["counters"]), pages=_u32(out["pages_distinct"]),
                   dists=_u32(out["dists"]) if w.dtype == "u8" else out["dists"].cpu().numpy(),
                   stats=ix.stats())
        return res
    finally:
        ix.close()


def _assert_exact(got, ref, rows=None):
    sl = slice(None) if rows is None else rows
    assert (got["ids"][sl] == ref["ids"][sl]).all()
    assert (got["dists"][sl] == ref["dists"][sl]).all()
    assert (got["counters"][sl] == ref["counters"][sl]).all()
    assert (got["pages"][sl] == ref["counters"][sl][:, 0]).all()


def _check_stats_invariants(st, ref_counters, max_outstanding, union_pages=None, preloaded=0):
    assert st["pages_fetched"] <= st["pages_missed"]
    assert int(ref_counters[:, 0].sum()) <= st["pages_hit"] + st["pages_missed"]
    assert st["max_outstanding_seen"] <= max_outstanding
    assert st["queries_done"] == ref_counters.shape[0]
    assert st["n_eval"] == int(ref_counters[:, 3].sum())
    assert st["n_expand"] == int(ref_counters[:, 2].sum())
    assert st["sum_degree"] == int(ref_counters[:, 4].sum())
    if union_pages is not None:
        assert st["pages_fetched"] >= union_pages - preloaded


# ------------------------------------------------------------------ configs 1 and 2 (10k nodes)
@pytest.fixture(scope="module")
def cfg1():
    w = make_config(1)
    ref = OracleIndex.from_workload(w).search(w.queries, w.K, w.L, w.W, threads=8, want_union=True)
    return w, ref


def test_config1_fully_cached_bit_exact(gorio, cfg1):
    w, ref = cfg1
    got = _gpu_search(gorio, w, w.n_pages, preload=True)
    _assert_exact(got, ref)
    st = got["stats"]
    assert st["pages_missed"] == 0 and st["pages_fetched"] == 0       # whole index resident
    _check_stats_invariants(st, ref["counters"], 256)
    assert recall_at_k(got["ids"], w.gt) == recall_at_k(ref["ids"], w.gt)


def test_config2_ten_percent_cache_bit_exact(gorio, cfg1):
    w, ref = cfg1
    cap = int(0.10 * w.n_pages)
    got = _gpu_search(gorio, w, cap, remote_latency_ns=0, max_outstanding=256)
    _assert_exact(got, ref)
    st = got["stats"]
    assert st["pages_missed"] > 0 and st["dedupe_joins"] > 0 and st["evictions"] > 0 and st["resumes"] > 0
    _check_stats_invariants(st, ref["counters"], 256, union_pages=int(ref["page_union"].sum()))


def test_cold_cache_with_room_for_every_page_fetches_each_page_once(gorio, cfg1):
    """Dedupe proof: with capacity for every page nothing is evicted, so the number of
    descriptors serviced must equal the number of distinct pages all queries touched."""
    w, ref = cfg1
    got = _gpu_search(gorio, w, w.n_pages, preload=False, max_outstanding=256)
    _assert_exact(got, ref)
    assert got["stats"]["pages_fetched"] == int(ref["page_union"].sum())
    assert got["stats"]["evictions"] == 0


@pytest.mark.parametrize("cfg", [
    dict(capacity=16), dict(capacity=64, max_outstanding=1), dict(capacity=1000, remote_latency_ns=20000),
    dict(capacity=1000, remote_latency_ns=200000, max_outstanding=32),
    dict(capacity=1000, max_outstanding=4), dict(capacity=1000, max_outstanding=1024),
    dict(capacity=2500, tuning=dict(warps_per_block=4)), dict(capacity=2500, tuning=dict(max_inflight=48)),
    dict(capacity=2500, tuning=dict(warps_per_block=8, blocks_per_sm=2)),
    dict(capacity=1000, remote_latency_ns=20000, tuning=dict(blocking=1)),
    dict(capacity=1000, tuning=dict(request_backlog=100000)), dict(capacity=1000, max_outstanding=8, tuning=dict(request_backlog=8)),
    dict(capacity=1000, tuning=dict(stash_entries=1)), dict(capacity=1000, tuning=dict(stash_entries=64)),
], ids=lambda c: "-".join(f"{k}={v}" for k, v in c.items() if k != "tuning") + ("-tuned" if "tuning" in c else ""))
def test_results_do_not_depend_on_cache_proxy_or_geometry(gorio, cfg1, cfg):
    """The proxy never touches search state, so outputs must be identical under any cache
    size, latency, outstanding depth and launch geometry."""
    w, ref = cfg1
    cfg = dict(cfg)
    cap = cfg.pop("capacity")
    nq = 200 if cap < 100 else 1000
    got = _gpu_search(gorio, w, cap, queries=w.queries[:nq], **cfg)
    _assert_exact(got, ref, rows=slice(0, nq))
    assert got["stats"]["max_outstanding_seen"] <= cfg.get("max_outstanding", 256)


def test_host_buffer_entry_point_matches(gorio, cfg1):
    w, ref = cfg1
    ix = gorio.Index.from_workload(w)
    try:
        ix.cache_config(2000, remote_latency_ns=5000)
        out = ix.search_host(w.queries, w.K, w.L, w.W)
    finally:
        ix.close()
    assert (out["ids"] == ref["ids"]).all() and (out["dists"] == ref["dists"]).all()
    assert (out["counters"] == ref["counters"]).all() and (out["pages_distinct"] == ref["counters"][:, 0]).all()


@pytest.mark.parametrize("cfg", [
    dict(capacity=1000, remote_latency_ns=0), dict(capacity=1000, remote_latency_ns=20000, max_outstanding=64),
    dict(capacity=64, max_outstanding=4), dict(capacity=1000, granularity="record"),
    dict(capacity=2000, remote_latency_ns=5000, tuning=dict(blocking=1)),
], ids=lambda c: "-".join(f"{k}={v}" for k, v in c.items() if k != "tuning") + ("-tuned" if "tuning" in c else ""))
def test_copy_engine_proxy_fills_slots_itself_bit_exact(gorio, cfg1, cfg):
    """copy_mode = copy engine: the proxy thread moves every page with a cudaMemcpyAsync of its own
    and publishes the completion once an event says the copy has landed; no warp copies pages.
    Results are the oracle's, as in the default mode; every wait is bounded by timeout_ms."""
    w, ref = cfg1
    cfg = dict(cfg)
    cap = cfg.pop("capacity")
    nq = 200
    got = _gpu_search(gorio, w, cap, queries=w.queries[:nq], copy_engine=True, timeout_ms=30000, **cfg)
    _assert_exact(got, ref, rows=slice(0, nq))
    st = got["stats"]
    assert st["pages_fetched"] > 0 and st["pages_fetched"] <= st["pages_missed"]
    assert st["max_outstanding_seen"] <= cfg.get("max_outstanding", 256)
    assert st["warp_ns_copies"] == 0                       # no SM time went into fills


def test_copy_engine_dedupe_proof_and_config3_shape(gorio, cfg1):
    w, ref = cfg1
    got = _gpu_search(gorio, w, w.n_pages, queries=w.queries[:300], copy_engine=True, timeout_ms=30000)
    _assert_exact(got, ref, rows=slice(0, 300))
    union = OracleIndex.from_workload(w).search(w.queries[:300], w.K, w.L, w.W, threads=4, want_union=True)["page_union"]
    assert got["stats"]["pages_fetched"] == int(union.sum()) and got["stats"]["evictions"] == 0
    w3 = make_config(3, scale=0.02, nq=200, with_gt=False)            # 10 nodes per page, R = 64
    ref3 = OracleIndex.from_workload(w3).search(w3.queries, w3.K, w3.L, w3.W, threads=4)
    got3 = _gpu_search(gorio, w3, w3.cache_pages, remote_latency_ns=20000, copy_engine=True, timeout_ms=60000)
    _assert_exact(got3, ref3)


@pytest.mark.parametrize("shared,warps,pq,bps", [(0, 0, False, 0), (1, 0, False, 0), (0, 2, False, 0), (0, 3, False, 0),
                                                 (0, 0, True, 0), (1, 0, True, 0), (0, 4, False, 2)])
def test_puller_warps_and_shared_pull_both_match_oracle(gorio, shared, warps, pq, bps):
    """Who pulls admitted pages: by default the last warp of every block does nothing else and
    pulls in ring order; tuning.shared_pull hands the pulls back to the worker warps.  Same
    results either way, also with the fewest warps per block (2: block 0 is poller and poster only,
    every other block one worker and one puller), with two blocks per SM (still one puller per SM's
    worth of blocks) and with PQ navigation."""
    w = make_config(3, scale=0.02, nq=300, with_gt=False)              # 10 nodes per page, R = 64
    if pq:
        w.pq_centroids, w.pq_codes = train_pq(w.data, m=32, sample=4096, iters=3)
    ref = OracleIndex.from_workload(w, use_pq=pq).search(w.queries, w.K, w.L, w.W, threads=4)
    got = _gpu_search(gorio, w, w.cache_pages, use_pq=pq, remote_latency_ns=5000, max_outstanding=64,
                      tuning=dict(shared_pull=shared, warps_per_block=warps, blocks_per_sm=bps))
    _assert_exact(got, ref)
    st = got["stats"]
    assert st["pages_fetched"] > 0 and st["max_outstanding_seen"] <= 64 and st["warp_ns_copies"] > 0


def test_link_probe_reports_a_plausible_rate(gorio, cfg1):
    """gorio_link_probe pulls pages of the pinned store with the loads of a page fill and nothing
    else; it must return a positive rate below the link's nominal 64 GB/s and reject bad arguments."""
    w, _ = cfg1
    ix = gorio.Index.from_workload(w)
    try:
        ix.cache_config(64)
        for seq in (False, True):
            gbs = ix.link_probe(20000, 64, sequential=seq)
            assert 1.0 < gbs < 64.0
        for bad in ((0, 64), (100, 0), (100, 20000)):
            with pytest.raises(gorio.GorioError) as e:
                ix.link_probe(*bad)
            assert e.value.status == 1
    finally:
        ix.close()


@pytest.mark.parametrize("K,L,W", [(1, 1, 1), (10, 10, 1), (64, 64, 4), (10, 200, 8), (100, 256, 16), (5, 33, 3)])
def test_parameter_edges(gorio, cfg1, K, L, W):
    w, _ = cfg1
    q = w.queries[:64]
    ref = OracleIndex.from_workload(w).search(q, K, L, W)
    got = _gpu_search(gorio, w, 1500, K=K, L=L, W=W, queries=q)
    _assert_exact(got, ref)


def test_single_query_and_unreachable_results_are_padded(gorio):
    from helpers import ring_index
    data, deg, nbrs, pages = ring_index([0, 10, 20, 30, 40], d=4, npp=2)
    deg[:] = 0
    pages = write_page_store(data, deg, nbrs, 2)
    ix = gorio.Index(pages, 5, 4, "u8", 2, 2, 1)
    try:
        ix.cache_config(16)
        out = ix.search(torch.zeros((1, 4), dtype=torch.uint8).cuda(), 3, 4, 2)
        assert _u32(out["ids"]).tolist() == [[1, 0xFFFFFFFF, 0xFFFFFFFF]]
        assert _u32(out["dists"]).tolist() == [[100, 0xFFFFFFFF, 0xFFFFFFFF]]
        assert _u32(out["counters"]).tolist() == [[1, 1, 1, 1, 0]]
    finally:
        ix.close()


def test_empty_batch_is_rejected_and_one_node_index_works(gorio):
    """Degenerate inputs: no queries (an argument error, nothing launched), an index of a single
    node without edges, and a two-node index whose lists hold self loops and duplicates."""
    pages1 = write_page_store(np.array([[7, 7, 7, 7]], dtype=np.uint8), np.zeros(1, np.uint32),
                              np.full((1, 3), 0xFFFFFFFF, np.uint32), 1)
    ix = gorio.Index(pages1, 1, 4, "u8", 3, 1, 0)
    try:
        ix.cache_config(16)
        with pytest.raises(gorio.GorioError) as e:
            ix.search(torch.zeros((0, 4), dtype=torch.uint8).cuda(), 1, 1, 1)
        assert e.value.status == 1
        q = torch.tensor([[7, 7, 7, 9], [0, 0, 0, 0]], dtype=torch.uint8).cuda()
        out = ix.search(q, 2, 4, 2)
        assert _u32(out["ids"]).tolist() == [[0, 0xFFFFFFFF], [0, 0xFFFFFFFF]]
        assert _u32(out["dists"]).tolist() == [[4, 0xFFFFFFFF], [196, 0xFFFFFFFF]]
        assert _u32(out["counters"]).tolist() == [[1, 1, 1, 1, 0]] * 2
    finally:
        ix.close()
    data = np.array([[0, 0, 0, 0], [3, 0, 0, 0]], dtype=np.uint8)
    deg = np.array([3, 3], dtype=np.uint32)
    nbrs = np.array([[0, 1, 1], [1, 1, 0]], dtype=np.uint32)           # self loops and duplicates
    pages2 = write_page_store(data, deg, nbrs, 2)
    ref = OracleIndex(pages2, 2, 4, "u8", 3, 2, 0).search(np.array([[2, 0, 0, 0]], dtype=np.uint8), 2, 2, 1)
    ix = gorio.Index(pages2, 2, 4, "u8", 3, 2, 0)
    try:
        ix.cache_config(16)
        out = ix.search(torch.tensor([[2, 0, 0, 0]], dtype=torch.uint8).cuda(), 2, 2, 1)
        assert (_u32(out["ids"]) == ref["ids"]).all() and (_u32(out["dists"]) == ref["dists"]).all()
        assert (_u32(out["counters"]) == ref["counters"]).all()
        assert _u32(out["ids"]).tolist() == [[1, 0]] and _u32(out["dists"]).tolist() == [[1, 4]]
    finally:
        ix.close()


def test_ring_worked_example_on_gpu(gorio):
    from helpers import ring_index
    data, deg, nbrs, pages = ring_index([10 * i for i in range(8)], d=4, npp=2)
    ix = gorio.Index(pages, 8, 4, "u8", 2, 2, 3)
    try:
        ix.cache_config(16)
        q = torch.tensor([[62, 0, 0, 0]], dtype=torch.uint8).cuda()
        out = ix.search(q, 2, 3, 2)
        assert _u32(out["ids"]).tolist() == [[6, 7]] and _u32(out["dists"]).tolist() == [[4, 64]]
        assert _u32(out["counters"]).tolist() == [[4, 5, 6, 8, 12]]
    finally:
        ix.close()


# ------------------------------------------------------------------ whole index resident: the fast path
@pytest.mark.parametrize("K,L,W", [(1, 1, 1), (10, 64, 4), (10, 10, 1), (64, 64, 4), (10, 200, 8), (100, 256, 16), (5, 33, 3)])
@pytest.mark.parametrize("fast", [True, False])
def test_resident_fast_path_and_general_path_both_match_oracle(gorio, cfg1, K, L, W, fast):
    """With the whole index preloaded a warp runs each query start to end (list in registers,
    candidates in shared memory); tuning.no_fast_path sends the same search through the general
    park-and-resume path.  Both must give the oracle's ids, distances and counters."""
    w, _ = cfg1
    q = w.queries[:300]
    ref = OracleIndex.from_workload(w).search(q, K, L, W, threads=4)
    got = _gpu_search(gorio, w, w.n_pages, K=K, L=L, W=W, queries=q, preload=True, tuning=dict(no_fast_path=0 if fast else 1))
    _assert_exact(got, ref)
    st = got["stats"]
    assert st["pages_missed"] == 0 and st["pages_fetched"] == 0 and st["queries_done"] == 300
    assert st["pages_hit"] == int(ref["counters"][:, 3].sum() + ref["counters"][:, 2].sum())      # one lookup per item


@pytest.mark.parametrize("tuning", [dict(warps_per_block=2), dict(warps_per_block=5, blocks_per_sm=2), dict(warps_per_block=24),
                                    dict(max_inflight=7)],
                         ids=lambda t: "-".join(f"{k}={v}" for k, v in t.items()))
def test_resident_fast_path_geometry_and_slot_recycling(gorio, cfg1, tuning):
    """Far more queries than worker warps or query slots (slots are recycled) and odd launch
    geometries on the fast path.  (Its hash-set form of the visited / page sets is what the
    allocation-free entry point runs; see test_zz_no_alloc.py.)"""
    w, ref = cfg1
    reps = 6
    q = np.tile(w.queries, (reps, 1))
    rows = np.arange(q.shape[0]) % w.nq
    got = _gpu_search(gorio, w, w.n_pages, queries=q, preload=True, tuning=tuning)
    assert (got["ids"] == ref["ids"][rows]).all() and (got["dists"] == ref["dists"][rows]).all()
    assert (got["counters"] == ref["counters"][rows]).all() and (got["pages"] == ref["counters"][rows, 0]).all()
    assert got["stats"]["queries_done"] == q.shape[0]


def test_resident_fast_path_other_shapes(gorio):
    """fp32 vectors (3 blocks of chunks), a PQ index (rerank pool in registers), vectors that are
    not whole 16-byte chunks (strided path) and 10-per-page records, all fully resident."""
    from workloads import node_bytes as nbytes
    w5 = make_config(5, scale=0.005, nq=300)
    ref5 = OracleIndex.from_workload(w5).search(w5.queries, w5.K, w5.L, w5.W, threads=4)
    _fp32_parity(w5, _gpu_search(gorio, w5, w5.n_pages, preload=True), ref5)
    w3 = make_config(3, scale=0.03, nq=400)
    ref3 = OracleIndex.from_workload(w3).search(w3.queries, w3.K, w3.L, w3.W, threads=4)
    _assert_exact(_gpu_search(gorio, w3, w3.n_pages, preload=True), ref3)
    w3.pq_centroids, w3.pq_codes = train_pq(w3.data, m=32, sample=16384, iters=4)
    for L, W, K in ((50, 1, 10), (100, 8, 10), (64, 4, 28), (64, 4, 40)):      # K + W = 44: the general path takes it
        refp = OracleIndex.from_workload(w3, use_pq=True).search(w3.queries, K, L, W, threads=4)
        _assert_exact(_gpu_search(gorio, w3, w3.n_pages, K=K, L=L, W=W, use_pq=True, preload=True), refp)
    d, R = 20, 12
    npp = 4096 // nbytes(d, np.uint8, R)
    wo = make_workload("odd", "u8", 6000, 6, 300, d, R - 4, 4, npp, clustered_knn=True, cross_only=False, K=10, L=48, W=3)
    refo = OracleIndex.from_workload(wo).search(wo.queries, wo.K, wo.L, wo.W, threads=4)
    _assert_exact(_gpu_search(gorio, wo, wo.n_pages, preload=True), refo)


def test_resident_fast_path_reports_a_corrupt_page(gorio):
    from helpers import ring_index
    data, deg, nbrs, pages = ring_index([0, 10, 20, 30], d=4, npp=1)
    nbrs[1, 1] = 99                                      # neighbour id >= N
    pages = write_page_store(data, deg, nbrs, 1)
    ix = gorio.Index(pages, 4, 4, "u8", 2, 1, 0)
    try:
        ix.cache_config(16, preload=True)
        with pytest.raises(gorio.GorioError) as e:
            ix.search(torch.zeros((3, 4), dtype=torch.uint8).cuda(), 1, 4, 1)
        assert e.value.status == 7
    finally:
        ix.close()


# ------------------------------------------------------------------ failure handling without faults
def test_corrupt_page_is_reported_not_trapped(gorio):
    from helpers import ring_index
    data, deg, nbrs, pages = ring_index([0, 10, 20, 30], d=4, npp=1)
    nbrs[0, 0] = 1234                                    # neighbour id >= N
    pages = write_page_store(data, deg, nbrs, 1)
    ix = gorio.Index(pages, 4, 4, "u8", 2, 1, 0)
    try:
        ix.cache_config(16)
        with pytest.raises(gorio.GorioError) as e:
            ix.search(torch.zeros((2, 4), dtype=torch.uint8).cuda(), 1, 4, 1)
        assert e.value.status == 7
    finally:
        ix.close()


def test_visited_set_overflow_is_a_capacity_error_and_index_stays_usable(gorio, cfg1):
    w, ref = cfg1
    ix = gorio.Index.from_workload(w)
    try:
        ix.cache_config(w.n_pages, preload=True)
        ix.set_tuning(visited_capacity=256)               # far fewer than the ~1000 nodes a query scores
        q = torch.as_tensor(w.queries[:32]).cuda()
        with pytest.raises(gorio.GorioError) as e:
            ix.search(q, w.K, w.L, w.W)
        assert e.value.status == 6
        ix.set_tuning()                                   # defaults again: same index, same context
        out = ix.search(q, w.K, w.L, w.W)
        assert (_u32(out["ids"]) == ref["ids"][:32]).all()
    finally:
        ix.close()


def test_remote_tier_that_never_answers_times_out_cleanly(gorio, cfg1):
    """The wait runs out (completions are held back by a 4 s latency against a 300 ms
    budget): the search returns TIMEOUT, every kernel has exited, and the same index then
    searches correctly again."""
    w, ref = cfg1
    ix = gorio.Index.from_workload(w)
    try:
        ix.cache_config(1000, remote_latency_ns=4_000_000_000, timeout_ms=300)
        q = torch.as_tensor(w.queries[:100]).cuda()
        with pytest.raises(gorio.GorioError) as e:
            ix.search(q, w.K, w.L, w.W)
        assert e.value.status == 5
        ix.cache_config(1000, remote_latency_ns=0, timeout_ms=60000)
        out = ix.search(q, w.K, w.L, w.W)
        assert (_u32(out["ids"]) == ref["ids"][:100]).all()
    finally:
        ix.close()


def test_call_order_and_argument_checks(gorio, cfg1):
    w, _ = cfg1
    ix = gorio.Index.from_workload(w)
    try:
        q = torch.as_tensor(w.queries[:4]).cuda()
        with pytest.raises(gorio.GorioError) as e:
            ix.search(q, 10, 64, 4)                        # before cache_config
        assert e.value.status == 4
        ix.cache_config(64)
        for K, L, W in ((0, 8, 1), (9, 8, 1), (1, 257, 1), (1, 8, 0), (1, 8, 17)):
            with pytest.raises(gorio.GorioError) as e:
                ix.search(q, K, L, W)
            assert e.value.status == 1
        with pytest.raises(gorio.GorioError):
            ix.cache_config(8)                             # below one set
    finally:
        ix.close()


# ------------------------------------------------------------------ config 3 (SIFT1M-shaped)
def test_config3_scaled_with_latency_bit_exact(gorio):
    w = make_config(3, scale=0.05, nq=1500)
    ref = OracleIndex.from_workload(w).search(w.queries, w.K, w.L, w.W, threads=8, want_union=True)
    got = _gpu_search(gorio, w, w.cache_pages, remote_latency_ns=20000, max_outstanding=256)
    _assert_exact(got, ref)
    _check_stats_invariants(got["stats"], ref["counters"], 256, union_pages=int(ref["page_union"].sum()))


@pytest.fixture(scope="module")
def cfg3_full():
    return make_config(3)


def test_config3_full_size_every_query_bit_exact(gorio, cfg3_full):
    """1M nodes, 10,000 queries, 20% cache, 20 us, <=256 outstanding -- the configuration the
    benchmark times; the oracle checks every query's ids, distances and counters."""
    w = cfg3_full
    assert w.N == 1_000_000 and w.n_pages == 100_000 and w.node_bytes == 388
    ref = OracleIndex.from_workload(w).search(w.queries, w.K, w.L, w.W, threads=THREADS, want_union=True)
    got = _gpu_search(gorio, w, w.cache_pages, remote_latency_ns=20000, max_outstanding=256)
    _assert_exact(got, ref)
    _check_stats_invariants(got["stats"], ref["counters"], 256, union_pages=int(ref["page_union"].sum()))
    # properties that hold at any size: sorted unique output, distances recomputable
    ids, dd = got["ids"], got["dists"]
    keys = dd.astype(np.uint64) << np.uint64(32) | ids.astype(np.uint64)
    assert (keys[:, 1:] > keys[:, :-1]).all()
    for r in range(0, w.nq, 97):
        diff = w.data[ids[r]].astype(np.int64) - w.queries[r].astype(np.int64)
        assert ((diff * diff).sum(1) == dd[r]).all()
    assert recall_at_k(ids, w.gt) == recall_at_k(ref["ids"], w.gt)


# ------------------------------------------------------------------ hash-set visited / page sets
def test_hash_set_visited_and_page_sets_under_misses_bit_exact(gorio, cfg3_full):
    """The per-query visited set and distinct-page set are bitmaps when those are small and
    open-addressing hash sets otherwise.  Every other uint8 test takes the bitmaps; this one
    forces both hash sets (1M nodes stored 3 per page: 31,250 and 10,417 bitmap words against a
    capacity of 8,192 entries) with a cold 10 % cache and 20 us misses, at page and at record
    granularity, and compares every query with the oracle."""
    w = cfg3_full
    npp, L, W, nq, cap_entries = 3, 64, 4, 3000, 8192
    pages3 = write_page_store(w.data, w.deg, w.nbrs, npp)
    n_pages = pages3.shape[0]
    assert (w.N + 31) // 32 > cap_entries and (n_pages + 31) // 32 > cap_entries      # neither bitmap fits
    q = w.queries[:nq]
    ref = OracleIndex(pages3, w.N, w.d, w.dtype, w.R, npp, w.entry).search(q, w.K, L, W, threads=THREADS, want_union=True)
    assert int(ref["counters"][:, 3].max()) < cap_entries - 64, "the workload must fit the forced capacity"
    ix = gorio.Index(pages3, w.N, w.d, w.dtype, w.R, npp, w.entry)
    try:
        ix.set_tuning(visited_capacity=cap_entries)
        qd = torch.as_tensor(q).cuda()
        for gran in ("page", "record"):
            ix.cache_config(n_pages // 10, remote_latency_ns=20000, max_outstanding=256, timeout_ms=120000, granularity=gran)
            ix.stats_reset()
            out = ix.search(qd, w.K, L, W)
            torch.cuda.synchronize()
            got = dict(ids=_u32(out["ids"]), dists=_u32(out["dists"]), counters=_u32(out["counters"]),
                       pages=_u32(out["pages_distinct"]))
            _assert_exact(got, ref)
            st = ix.stats()
            assert st["pages_missed"] > 0 and st["evictions"] > 0 and st["resumes"] > 0 and st["queries_done"] == nq
            if gran == "page":
                _check_stats_invariants(st, ref["counters"], 256, union_pages=int(ref["page_union"].sum()))
    finally:
        ix.close()


# ------------------------------------------------------------------ config 4 (PQ navigation)
@pytest.fixture(scope="module")
def cfg4_small():
    w = make_config(3, scale=0.05, nq=300)
    w.pq_centroids, w.pq_codes = train_pq(w.data, m=32, sample=16384, iters=6)
    return w


@pytest.mark.parametrize("L", [50, 100, 200])
@pytest.mark.parametrize("W", [1, 4, 8])
def test_config4_pq_sweep_bit_exact(gorio, cfg4_small, L, W):
    w = cfg4_small
    ref = OracleIndex.from_workload(w, use_pq=True).search(w.queries, w.K, L, W, threads=8)
    for frac, preload in ((0.05, False), (0.20, False), (1.0, True)):
        cap = max(16, int(frac * w.n_pages))
        got = _gpu_search(gorio, w, cap, L=L, W=W, use_pq=True, preload=preload,
                          remote_latency_ns=20000 if not preload else 0)
        _assert_exact(got, ref)


@pytest.fixture(scope="module")
def cfg4_full(cfg3_full):
    w = cfg3_full
    if w.pq_centroids is None:
        w.pq_centroids, w.pq_codes = train_pq(w.data, m=32)
    return w


@pytest.mark.parametrize("L", [50, 100, 200])
@pytest.mark.parametrize("W", [1, 4, 8])
def test_config4_full_size_every_sweep_point_bit_exact(gorio, cfg4_full, L, W):
    """The PQ sweep on the 1M-node index itself: for each (L, W) the oracle's answers to all
    10,000 queries, against the CUDA path at 5 %, 20 % (cold, 20 us misses) and 100 % (preloaded)
    cache -- 27 points, every query's ids, exact distances and counters."""
    w = cfg4_full
    ref = OracleIndex.from_workload(w, use_pq=True).search(w.queries, w.K, L, W, threads=THREADS)
    ix = gorio.Index.from_workload(w, use_pq=True)
    try:
        qd = torch.as_tensor(w.queries).cuda()
        for frac in (0.05, 0.20, 1.0):
            preload = frac >= 1.0
            ix.cache_config(int(frac * w.n_pages), remote_latency_ns=0 if preload else 20000, max_outstanding=256,
                            preload=preload, timeout_ms=120000)
            ix.stats_reset()
            out = ix.search(qd, w.K, L, W)
            torch.cuda.synchronize()
            got = dict(ids=_u32(out["ids"]), dists=_u32(out["dists"]), counters=_u32(out["counters"]),
                       pages=_u32(out["pages_distinct"]))
            _assert_exact(got, ref)
            st = ix.stats()
            assert st["queries_done"] == w.nq and (st["pages_fetched"] == 0) == preload
    finally:
        ix.close()


# ------------------------------------------------------------------ config 5 (fp32)
def test_config5_scaled_fp32_tolerance(gorio):
    w = make_config(5, scale=0.02, nq=2000)          # 200,000 nodes, 6 per page, 10% cache
    ref = OracleIndex.from_workload(w).search(w.queries, w.K, w.L, w.W, threads=8)
    got = _gpu_search(gorio, w, w.cache_pages, remote_latency_ns=20000, max_outstanding=256)
    _fp32_parity(w, got, ref)


def test_config5_full_size_every_query_fp32_tolerance(gorio):
    """10,000,000 x 96 fp32 nodes, 6 per page (1,666,667 pages, 6.8 GB pinned), 10,000 queries,
    K=10 L=128 W=4, 10 % cache, 20 us; the oracle checks every query."""
    w = make_config(5)
    assert w.N == 10_000_000 and w.n_pages == 1_666_667 and w.node_bytes == 644
    ref = OracleIndex.from_workload(w).search(w.queries, w.K, w.L, w.W, threads=THREADS)
    got = _gpu_search(gorio, w, w.cache_pages, remote_latency_ns=20000, max_outstanding=256, timeout_ms=120000)
    _fp32_parity(w, got, ref)
    assert got["stats"]["queries_done"] == w.nq and got["stats"]["max_outstanding_seen"] <= 256
    # properties at full size: reported distances recomputable in double within fp32 rounding
    for r in range(0, w.nq, 211):
        ids = got["ids"][r]
        dd = ((w.data[ids].astype(np.float64) - w.queries[r].astype(np.float64)) ** 2).sum(1)
        np.testing.assert_allclose(got["dists"][r], dd, rtol=2e-6)
        assert (np.diff(dd) >= -1e-5 * dd[1:]).all()


# ------------------------------------------------------------------ scoring paths off the standard shapes
@pytest.mark.parametrize("kind,d,R", [
    ("u8", 20, 12),      # 20-byte vectors: not whole 16-byte chunks -> 4-byte-per-lane path
    ("u8", 256, 24),     # 16 chunks: two chunks per lane in the 128-bit path
    ("u8", 512, 8),      # longer than the 128-bit path handles -> one-at-a-time path
    ("f32", 36, 16),     # 144-byte vectors: 9 chunks
    ("f32", 200, 20),    # 800-byte vectors -> one-at-a-time path
])
def test_other_dimensions_match_oracle(gorio, kind, d, R):
    from workloads import node_bytes as nbytes
    nb = nbytes(d, np.uint8 if kind == "u8" else np.float32, R)
    npp = max(1, 4096 // nb)
    w = make_workload("odd", kind, 6000, 6, 300, d, R - 4, 4, npp, clustered_knn=True, cross_only=False,
                      K=10, L=48, W=3)
    ref = OracleIndex.from_workload(w).search(w.queries, w.K, w.L, w.W, threads=4)
    got = _gpu_search(gorio, w, max(16, w.n_pages // 5), remote_latency_ns=2000)
    if kind == "u8":
        _assert_exact(got, ref)
    else:
        _fp32_parity(w, got, ref)


def test_queries_not_16_byte_aligned_take_the_narrow_path(gorio, cfg1):
    w, ref = cfg1
    ix = gorio.Index.from_workload(w)
    try:
        ix.cache_config(1500)
        buf = torch.zeros(4 + 200 * w.d, dtype=torch.uint8, device="cuda")
        q = buf[4:].view(200, w.d)                       # data pointer is 4 bytes past a 16-byte boundary
        q.copy_(torch.as_tensor(w.queries[:200]))
        assert q.data_ptr() % 16 == 4 and q.is_contiguous()
        out = ix.search(q, w.K, w.L, w.W)
        assert (_u32(out["ids"]) == ref["ids"][:200]).all() and (_u32(out["dists"]) == ref["dists"][:200]).all()
        assert (_u32(out["counters"]) == ref["counters"][:200]).all()
    finally:
        ix.close()


def test_sixteen_thousand_queries_join_the_entry_page_at_once_repeatedly(gorio, cfg1):
    """Every query's first item is the entry node, so a batch opens with all of its queries
    joining one page's waiter list through compare-and-swap on one word.  Ten cold searches of
    16,384 queries each must all come out exact."""
    w, ref = cfg1
    reps = -(-16384 // w.nq)
    q = np.tile(w.queries, (reps, 1))[:16384]
    rows = np.arange(16384) % w.nq
    ix = gorio.Index.from_workload(w)
    try:
        qd = torch.as_tensor(q).cuda()
        for it in range(10):
            ix.cache_config(500, remote_latency_ns=(0, 20000)[it % 2], max_outstanding=256, timeout_ms=60000)
            out = ix.search(qd, w.K, w.L, w.W)
            assert (_u32(out["ids"]) == ref["ids"][rows]).all()
            assert (_u32(out["counters"]) == ref["counters"][rows]).all()
    finally:
        ix.close()


def test_two_threads_on_one_index_are_serialised(gorio, cfg1):
    """Calls on one index are serialised by the library: two caller threads searching at the
    same time both get the oracle's answers."""
    import threading
    w, ref = cfg1
    ix = gorio.Index.from_workload(w)
    results, errors = {}, []
    try:
        ix.cache_config(1000, remote_latency_ns=5000)
        q = torch.as_tensor(w.queries).cuda()

        def work(tag):
            try:
                for _ in range(3):
                    s = torch.cuda.Stream()
                    out = ix.search(q, w.K, w.L, w.W, stream=s)
                    s.synchronize()
                    results.setdefault(tag, []).append(_u32(out["ids"]).copy())
            except Exception as e:                       # noqa: BLE001
                errors.append(e)

        ts = [threading.Thread(target=work, args=(i,)) for i in range(2)]
        for t in ts:
            t.start()
        for t in ts:
            t.join()
    finally:
        ix.close()
    assert not errors, errors
    assert all((ids == ref["ids"]).all() for tag in results for ids in results[tag]) and len(results) == 2


def test_second_search_reuses_the_warm_cache(gorio, cfg1):
    w, ref = cfg1
    ix = gorio.Index.from_workload(w)
    try:
        ix.cache_config(w.n_pages, preload=False)         # room for everything, cold
        q = torch.as_tensor(w.queries).cuda()
        a = ix.search(q, w.K, w.L, w.W)
        f1 = ix.stats()["pages_fetched"]
        b = ix.search(q, w.K, w.L, w.W)                   # same index, no cache_config in between
        f2 = ix.stats()["pages_fetched"] - f1
        for out in (a, b):
            assert (_u32(out["ids"]) == ref["ids"]).all() and (_u32(out["counters"]) == ref["counters"]).all()
        assert f1 == int(ref["page_union"].sum()) and f2 == 0
    finally:
        ix.close()


# ------------------------------------------------------------------ randomized configurations
@pytest.mark.parametrize("seed", list(range(int(os.environ.get("GORIO_FUZZ_SEEDS", "24")))))
def test_randomized_configurations_match_oracle(gorio, seed):
    """Small random indexes under random search, cache, proxy and scheduler settings: whatever
    the interleaving of misses, arrivals, evictions and resumes, uint8 results are bit-exact."""
    from workloads import node_bytes as nbytes
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([16, 32, 48, 64, 128]))
    R = int(rng.integers(4, 33))
    nb = nbytes(d, np.uint8, R)
    npp = int(rng.integers(1, 4096 // nb + 1))
    N = int(rng.integers(400, 5000))
    C = int(rng.integers(1, 6))
    nq = int(rng.integers(1, 500))
    k = int(rng.integers(2, R))
    L = int(rng.integers(4, 129))
    W = int(rng.integers(1, min(9, 1024 // R)))
    K = int(rng.integers(1, min(L, 20) + 1))
    w = make_workload(f"rnd{seed}", "u8", N, C, nq, d, k, R - k, npp, clustered_knn=bool(rng.integers(0, 2)),
                      cross_only=False, with_gt=False, K=K, L=L, W=W)
    ref = OracleIndex.from_workload(w).search(w.queries, K, L, W, threads=4)
    cap = int(rng.integers(16, max(17, w.n_pages + 1)))
    tuning = dict(warps_per_block=int(rng.integers(2, 17)), max_inflight=int(rng.choice([0, 8, 64])),
                  stash_entries=int(rng.choice([0, 1, 64, 256])), blocking=int(rng.integers(0, 2)),
                  request_backlog=int(rng.choice([0, 1, 16, 4096])), shared_pull=int(rng.integers(0, 3) == 0))
    preload, lat, depth = bool(rng.integers(0, 4) == 0), int(rng.choice([0, 2000, 20000])), int(rng.choice([1, 8, 256]))
    copy_engine, gran = bool(rng.integers(0, 4) == 0), str(rng.choice(["page", "page", "record"]))
    got = _gpu_search(gorio, w, cap, K=K, L=L, W=W, tuning=tuning, preload=preload and gran == "page",
                      remote_latency_ns=lat, max_outstanding=depth, copy_engine=copy_engine, granularity=gran)
    _assert_exact(got, ref)
    assert got["stats"]["queries_done"] == nq


@pytest.mark.parametrize("seed", list(range(8)))
def test_randomized_fp32_and_pq_configurations(gorio, seed):
    from workloads import node_bytes as nbytes
    rng = np.random.default_rng(5000 + seed)
    pq = seed % 2 == 1
    R = int(rng.integers(6, 25))
    if pq:
        kind, d = "u8", int(rng.choice([32, 64, 128]))          # 8 / 16 / 32 ... subspaces of 4 bytes
    else:
        kind, d = "f32", int(rng.choice([8, 24, 40, 96]))
    nb = nbytes(d, np.uint8 if kind == "u8" else np.float32, R)
    npp = int(rng.integers(1, 4096 // nb + 1))
    N, nq = int(rng.integers(1500, 6000)), int(rng.integers(20, 300))
    L, W = int(rng.integers(16, 100)), int(rng.integers(1, 6))
    w = make_workload(f"rnd{seed}", kind, N, 4, nq, d, R - 3, 3, npp, clustered_knn=True, cross_only=False,
                      with_gt=not pq, K=8, L=L, W=W)
    if pq:
        w.pq_centroids, w.pq_codes = train_pq(w.data, m=d // 4, sample=2048, iters=3)
    ref = OracleIndex.from_workload(w, use_pq=pq).search(w.queries, 8, L, W, threads=4)
    cap = int(rng.integers(16, max(17, w.n_pages // 2)))
    got = _gpu_search(gorio, w, cap, K=8, L=L, W=W, use_pq=pq, remote_latency_ns=int(rng.choice([0, 5000])),
                      max_outstanding=int(rng.choice([4, 256])), tuning=dict(max_inflight=int(rng.choice([0, 32]))))
    if pq:
        _assert_exact(got, ref)
    else:
        _fp32_parity(w, got, ref)
