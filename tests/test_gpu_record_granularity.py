"""GPU parity for selective materialisation (Section 7.2, third direction): a miss fetches only the
wanted node's record and the cache holds records.  Results and per-query counters must be the
oracle's, exactly as at page granularity; only the remote traffic changes."""
import numpy as np
import pytest
import torch

from oracle import OracleIndex
from workloads import make_config, make_workload, train_pq, write_page_store
from workloads import node_bytes as nbytes

from helpers import fp32_parity as _fp32_parity
from test_gpu_parity import _assert_exact, _check_stats_invariants, _gpu_search, _u32, gorio  # noqa: F401

pytestmark = pytest.mark.gpu


def _slot_bytes(w):
    return (w.node_bytes + 12 + 15) // 16 * 16


@pytest.fixture(scope="module")
def cfg1():
    w = make_config(1)
    ref = OracleIndex.from_workload(w).search(w.queries, w.K, w.L, w.W, threads=8, want_union=True)
    return w, ref


def _node_union(w, K, L, W):
    """Distinct nodes all queries touch: the page union of the same graph stored one node per page."""
    one = OracleIndex(write_page_store(w.data, w.deg, w.nbrs, 1), w.N, w.d, w.dtype, w.R, 1, w.entry)
    return int(one.search(w.queries, K, L, W, threads=8, want_union=True)["page_union"].sum())


def test_config2_record_granularity_bit_exact(gorio, cfg1):
    w, ref = cfg1
    cap = int(0.10 * w.n_pages) // 5              # 200 pages' worth of HBM = 2,048 record slots for 10,000 nodes
    got = _gpu_search(gorio, w, cap, remote_latency_ns=0, max_outstanding=256, granularity="record")
    _assert_exact(got, ref)                       # pages_distinct still counts index pages
    st = got["stats"]
    assert st["pages_missed"] > 0 and st["evictions"] > 0 and st["resumes"] > 0
    assert st["fetched_bytes"] == st["pages_fetched"] * _slot_bytes(w) and _slot_bytes(w) == 272    # 260-byte records
    assert st["pages_fetched"] <= st["pages_missed"] and st["max_outstanding_seen"] <= 256
    assert st["n_eval"] == int(ref["counters"][:, 3].sum()) and st["queries_done"] == w.nq
    assert st["pages_fetched"] >= _node_union(w, w.K, w.L, w.W)


def test_record_cache_with_room_for_every_node_fetches_each_node_once(gorio, cfg1):
    """Dedupe at record granularity: nothing is evicted, so the records fetched are exactly the
    distinct nodes that any query scored or expanded."""
    w, ref = cfg1
    got = _gpu_search(gorio, w, w.n_pages, granularity="record")     # 4096 / 400 slots per page > npp
    _assert_exact(got, ref)
    assert got["stats"]["evictions"] == 0
    assert got["stats"]["pages_fetched"] == _node_union(w, w.K, w.L, w.W)


def test_fewer_bytes_cross_the_link_than_at_page_granularity(gorio, cfg1):
    w, ref = cfg1
    cap = 200
    page = _gpu_search(gorio, w, cap, remote_latency_ns=5000)
    rec = _gpu_search(gorio, w, cap, remote_latency_ns=5000, granularity="record")
    _assert_exact(page, ref)
    _assert_exact(rec, ref)
    assert page["stats"]["fetched_bytes"] == page["stats"]["pages_fetched"] * 4096
    assert rec["stats"]["fetched_bytes"] == rec["stats"]["pages_fetched"] * _slot_bytes(w)
    assert rec["stats"]["fetched_bytes"] * 2 < page["stats"]["fetched_bytes"]


@pytest.mark.parametrize("cfg", [
    dict(capacity=16), dict(capacity=64, max_outstanding=1), dict(capacity=1000, remote_latency_ns=20000),
    dict(capacity=1000, remote_latency_ns=200000, max_outstanding=32),
    dict(capacity=2500, tuning=dict(warps_per_block=4)), dict(capacity=2500, tuning=dict(max_inflight=48)),
    dict(capacity=1000, remote_latency_ns=20000, tuning=dict(blocking=1)),
    dict(capacity=1000, tuning=dict(stash_entries=1)), dict(capacity=1000, max_outstanding=8, tuning=dict(request_backlog=8)),
], ids=lambda c: "-".join(f"{k}={v}" for k, v in c.items() if k != "tuning") + ("-tuned" if "tuning" in c else ""))
def test_record_mode_results_do_not_depend_on_cache_proxy_or_geometry(gorio, cfg1, cfg):
    w, ref = cfg1
    cfg = dict(cfg)
    cap = cfg.pop("capacity")
    nq = 200 if cap < 100 else 1000
    got = _gpu_search(gorio, w, cap, queries=w.queries[:nq], granularity="record", **cfg)
    _assert_exact(got, ref, rows=slice(0, nq))
    assert got["stats"]["max_outstanding_seen"] <= cfg.get("max_outstanding", 256)


def test_config3_scaled_record_granularity_bit_exact(gorio):
    w = make_config(3, scale=0.05, nq=1500)
    ref = OracleIndex.from_workload(w).search(w.queries, w.K, w.L, w.W, threads=8)
    got = _gpu_search(gorio, w, w.cache_pages, remote_latency_ns=20000, max_outstanding=256, granularity="record")
    _assert_exact(got, ref)


def test_config4_pq_record_granularity_bit_exact(gorio):
    w = make_config(3, scale=0.05, nq=300)
    w.pq_centroids, w.pq_codes = train_pq(w.data, m=32, sample=16384, iters=6)
    ref = OracleIndex.from_workload(w, use_pq=True).search(w.queries, w.K, 100, 4, threads=8)
    got = _gpu_search(gorio, w, max(16, int(0.05 * w.n_pages)), L=100, W=4, use_pq=True, remote_latency_ns=20000,
                      granularity="record")
    _assert_exact(got, ref)


def test_config5_scaled_fp32_record_granularity(gorio):
    w = make_config(5, scale=0.02, nq=2000)
    ref = OracleIndex.from_workload(w).search(w.queries, w.K, w.L, w.W, threads=8)
    got = _gpu_search(gorio, w, w.cache_pages, remote_latency_ns=20000, max_outstanding=256, granularity="record")
    _fp32_parity(w, got, ref)
    assert got["stats"]["fetched_bytes"] == got["stats"]["pages_fetched"] * 656      # 644-byte records


@pytest.mark.parametrize("kind,d,R,npp", [
    ("u8", 20, 12, 0),       # 72-byte records, 56 per page
    ("u8", 256, 24, 0),      # 356-byte records
    ("u8", 512, 8, 3),       # fewer nodes per page than would fit
    ("u8", 3968, 30, 1),     # a record that nearly fills the page: 4092 bytes, 256 chunks
    ("f32", 36, 16, 0),
    ("f32", 200, 20, 0),
])
def test_record_mode_other_record_sizes(gorio, kind, d, R, npp):
    nb = nbytes(d, np.uint8 if kind == "u8" else np.float32, R)
    npp = npp or max(1, 4096 // nb)
    N = 6000 if d < 1000 else 1200
    w = make_workload("odd", kind, N, 6, 200, d, R - 4, 4, npp, clustered_knn=True, cross_only=False, K=10, L=48, W=3)
    ref = OracleIndex.from_workload(w).search(w.queries, w.K, w.L, w.W, threads=4)
    got = _gpu_search(gorio, w, max(16, w.n_pages // 5), remote_latency_ns=2000, granularity="record")
    if kind == "u8":
        _assert_exact(got, ref)
    else:
        _fp32_parity(w, got, ref)


def test_last_record_of_the_store_is_not_read_past_its_page(gorio):
    """The span fetched for a record is clipped to the record: the final node of the final page is
    fetched without touching bytes beyond the pinned store."""
    w = make_workload("tail", "u8", 1003, 2, 50, 128, 20, 4, 10, clustered_knn=True, cross_only=False, K=5, L=32, W=2)
    assert w.N % w.npp != 0
    q = np.concatenate([w.queries, w.data[-3:]])               # queries that land on the last nodes
    ref = OracleIndex.from_workload(w).search(q, 5, 32, 2, threads=2)
    got = _gpu_search(gorio, w, 16, queries=q, K=5, L=32, W=2, granularity="record")
    _assert_exact(got, ref)
    assert (got["ids"][-3:, 0] == np.arange(w.N - 3, w.N)).all()


def test_record_mode_rejects_preload_and_unknown_granularity(gorio, cfg1):
    w, _ = cfg1
    ix = gorio.Index.from_workload(w)
    try:
        with pytest.raises(gorio.GorioError) as e:
            ix.cache_config(64, preload=True, granularity="record")
        assert e.value.status == 1
        ix.cache_config(64, granularity="record")                 # and the index stays usable
        q = torch.as_tensor(w.queries[:8]).cuda()
        ix.search(q, 10, 64, 4)
        ix.cache_config(64)                                       # back to pages on the same handle
        ix.search(q, 10, 64, 4)
    finally:
        ix.close()


@pytest.mark.parametrize("seed", list(range(12)))
def test_randomized_record_mode_configurations(gorio, seed):
    rng = np.random.default_rng(9000 + seed)
    d = int(rng.choice([16, 32, 48, 64, 128]))
    R = int(rng.integers(4, 33))
    nb = nbytes(d, np.uint8, R)
    npp = int(rng.integers(1, 4096 // nb + 1))
    N, nq = int(rng.integers(400, 5000)), int(rng.integers(1, 400))
    k = int(rng.integers(2, R))
    L, W = int(rng.integers(4, 129)), int(rng.integers(1, min(9, 1024 // R)))
    K = int(rng.integers(1, min(L, 20) + 1))
    w = make_workload(f"rec{seed}", "u8", N, int(rng.integers(1, 6)), nq, d, k, R - k, npp,
                      clustered_knn=bool(rng.integers(0, 2)), cross_only=False, with_gt=False, K=K, L=L, W=W)
    ref = OracleIndex.from_workload(w).search(w.queries, K, L, W, threads=4)
    cap = int(rng.integers(16, max(17, w.n_pages + 1)))
    tuning = dict(warps_per_block=int(rng.integers(2, 17)), max_inflight=int(rng.choice([0, 8, 64])),
                  stash_entries=int(rng.choice([0, 1, 64, 256])), blocking=int(rng.integers(0, 2)),
                  request_backlog=int(rng.choice([0, 1, 16, 4096])))
    got = _gpu_search(gorio, w, cap, K=K, L=L, W=W, tuning=tuning, granularity="record",
                      remote_latency_ns=int(rng.choice([0, 2000, 20000])), max_outstanding=int(rng.choice([1, 8, 256])))
    _assert_exact(got, ref)
    assert got["stats"]["queries_done"] == nq
