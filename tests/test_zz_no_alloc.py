"""The allocation-free entry point, for callers that may not call cudaMalloc (fixed-arena
services, latency-critical loops, plugins of hosts that forbid allocation after start-up).

It must return what the CPU oracle returns -- and therefore what the ordinary open /
cache_config / search path returns -- on two calls in a row (the second call reuses the
library's fixed scratch array with the first call's leftovers in it), and must refuse inputs
larger than that array with a clear error.
Collected last on purpose: if it fails under `pytest -x`, every other test has already run.
"""
import numpy as np
import pytest
import torch

from helpers import fp32_parity
from oracle import OracleIndex
from workloads import make_config

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gorio():
    from paper_2607_04415_b200 import build
    build.build()
    import paper_2607_04415_b200 as g
    return g


def _u32(t):
    return t.cpu().numpy().view(np.uint32)


def _noalloc(g, w, pages_dev, q, K, L, W):
    out = g.search_resident_noalloc(pages_dev, w.N, w.d, w.dtype, w.R, w.npp, w.entry, q, K, L, W)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("which,nq", [(1, 300), (3, 150)])
def test_noalloc_entry_matches_oracle_and_regular_entry_twice_in_a_row(gorio, which, nq):
    scale = 0.5 if which == 1 else 0.02            # 5,000 pages (1 node each) / 2,000 pages (10 nodes each)
    w = make_config(which, scale=scale, nq=nq, with_gt=False)
    assert w.n_pages <= 32768
    orc = OracleIndex.from_workload(w)
    ref = orc.search(w.queries, w.K, w.L, w.W, threads=4)
    q = torch.as_tensor(w.queries).cuda()
    ix = gorio.Index.from_workload(w)
    try:
        ix.cache_config(w.n_pages, preload=True)
        reg = ix.search(q, w.K, w.L, w.W)
        reg = {k: _u32(reg[k]) for k in ("ids", "dists", "pages_distinct")}
    finally:
        ix.close()
    pages_dev = torch.as_tensor(w.pages).cuda()
    for call in range(2):
        out = _noalloc(gorio, w, pages_dev, q, w.K, w.L, w.W)
        # uint8 data: bit-exact against the oracle, as in the parity tests
        assert (_u32(out["ids"]) == ref["ids"]).all(), f"ids differ from the oracle on call {call}"
        assert (_u32(out["dists"]) == ref["dists"]).all(), f"distances differ from the oracle on call {call}"
        assert (_u32(out["pages_distinct"]) == ref["counters"][:, 0]).all(), f"page counts differ on call {call}"
        for k in ("ids", "dists", "pages_distinct"):
            assert (_u32(out[k]) == reg[k]).all(), f"{k} differs from the regular entry on call {call}"
    # more queries than in-flight slots, other parameters, same scratch: still exact
    ref2 = orc.search(w.queries, 5, 40, 2, threads=4)
    out2 = _noalloc(gorio, w, pages_dev, q, 5, 40, 2)
    assert (_u32(out2["ids"]) == ref2["ids"]).all() and (_u32(out2["dists"]) == ref2["dists"]).all()
    assert (_u32(out2["pages_distinct"]) == ref2["counters"][:, 0]).all()


def test_noalloc_entry_fp32_within_tolerance_twice_in_a_row(gorio):
    w = make_config(5, scale=0.01, nq=400)          # 100,000 x 96 fp32 nodes, 6 per page: 16,667 pages
    assert w.n_pages <= 32768 and w.dtype == "f32"
    ref = OracleIndex.from_workload(w).search(w.queries, w.K, w.L, w.W, threads=4)
    assert int(ref["counters"][:, 3].max()) < 16384  # within the fixed per-query visited set
    q = torch.as_tensor(w.queries).cuda()
    pages_dev = torch.as_tensor(w.pages).cuda()
    for _ in range(2):
        out = _noalloc(gorio, w, pages_dev, q, w.K, w.L, w.W)
        got = dict(ids=_u32(out["ids"]), dists=out["dists"].cpu().numpy(), counters=None)
        fp32_parity(w, got, ref)
        same = (got["ids"] == ref["ids"]).all(1)
        assert (_u32(out["pages_distinct"])[same] == ref["counters"][same, 0]).mean() >= 0.999


def test_noalloc_entry_with_far_more_queries_than_slots(gorio):
    """64 queries are in flight at a time whatever nq is; a batch of 12,000 (more than 64 per SM)
    must come out exact and well inside the call's fixed 60 s budget."""
    import time
    w = make_config(1, scale=0.5, nq=500, with_gt=False)
    ref = OracleIndex.from_workload(w).search(w.queries, w.K, w.L, w.W, threads=4)
    rows = np.arange(12000) % w.nq
    q = torch.as_tensor(w.queries[rows]).cuda()
    pages_dev = torch.as_tensor(w.pages).cuda()
    _noalloc(gorio, w, pages_dev, q[:8], w.K, w.L, w.W)          # first call on the device: set-up
    t0 = time.perf_counter()
    out = _noalloc(gorio, w, pages_dev, q, w.K, w.L, w.W)
    dt = time.perf_counter() - t0
    assert (_u32(out["ids"]) == ref["ids"][rows]).all() and (_u32(out["dists"]) == ref["dists"][rows]).all()
    assert dt < 20.0, f"12,000 resident queries took {dt:.1f} s"


def test_noalloc_entry_rejects_what_does_not_fit_its_scratch(gorio):
    w = make_config(1, scale=0.05, nq=8, with_gt=False)
    q = torch.as_tensor(w.queries).cuda()
    pages_dev = torch.as_tensor(w.pages).cuda()
    with pytest.raises(gorio.GorioError) as e:          # claims more pages than the array can track
        gorio.search_resident_noalloc(torch.zeros(40000 * 4096, dtype=torch.uint8, device="cuda"), 40000, w.d, w.dtype,
                                      w.R, 1, 0, q, 10, 64, 4)
    assert e.value.status == 1 and "32768 pages" in str(e.value)
    with pytest.raises(gorio.GorioError) as e:          # W * max_degree beyond the per-query buffers
        gorio.search_resident_noalloc(pages_dev, w.N, w.d, w.dtype, w.R, w.npp, w.entry, q, 10, 64, 16)
    assert e.value.status == 1 and "W*max_degree" in str(e.value)
    with pytest.raises(gorio.GorioError) as e:          # a page buffer smaller than the description says
        gorio.search_resident_noalloc(pages_dev.view(-1)[: 4096 * (w.n_pages - 1)], w.N, w.d, w.dtype, w.R, w.npp, w.entry, q, 10, 64, 4)
    assert e.value.status == 1
    with pytest.raises(gorio.GorioError) as e:          # queries of the wrong width
        gorio.search_resident_noalloc(pages_dev, w.N, w.d, w.dtype, w.R, w.npp, w.entry, q[:, :64].contiguous(), 10, 64, 4)
    assert e.value.status == 1
    # and it still works afterwards
    out = gorio.search_resident_noalloc(pages_dev, w.N, w.d, w.dtype, w.R, w.npp, w.entry, q, 10, 64, 4)
    assert _u32(out["ids"]).shape == (8, 10)
