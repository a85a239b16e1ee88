"""The allocation-free entry point, for callers that may not call cudaMalloc (fixed-arena
services, latency-critical loops, plugins of hosts that forbid allocation after start-up).

It must return exactly what the ordinary open / cache_config / search path returns, on two
calls in a row (the second call reuses the library's fixed scratch array with the first
call's leftovers in it), and must refuse inputs larger than that array with a clear error.
Collected last on purpose: if it fails under `pytest -x`, every other test has already run.
"""
import ctypes

import numpy as np
import pytest
import torch

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


@pytest.mark.parametrize("which,nq", [(1, 300), (3, 150)])
def test_noalloc_entry_matches_regular_entry_twice_in_a_row(gorio, which, nq):
    scale = 0.5 if which == 1 else 0.02            # 5,000 pages (1 node each) / 2,000 pages (10 nodes each)
    w = make_config(which, scale=scale, nq=nq, with_gt=False)
    assert w.n_pages <= 32768
    q = torch.as_tensor(w.queries).cuda()
    ix = gorio.Index.from_workload(w)
    try:
        ix.cache_config(w.n_pages, preload=True)
        ref = ix.search(q, w.K, w.L, w.W)
        ref = {k: _u32(ref[k]) for k in ("ids", "dists", "pages_distinct")}
    finally:
        ix.close()
    pages_dev = torch.as_tensor(w.pages).cuda()
    for call in range(2):
        out = gorio.search_resident_noalloc(pages_dev, w.N, w.d, w.dtype, w.R, w.npp, w.entry, q, w.K, w.L, w.W)
        torch.cuda.synchronize()
        for k in ("ids", "dists", "pages_distinct"):       # uint8 data: bit-exact, as in the parity tests
            assert (_u32(out[k]) == ref[k]).all(), f"{k} differs on call {call}"
    # more queries than in-flight slots, other parameters, same scratch: still exact
    ix = gorio.Index.from_workload(w)
    try:
        ix.cache_config(w.n_pages, preload=True)
        ref2 = ix.search(q, 5, 40, 2)
        out2 = gorio.search_resident_noalloc(pages_dev, w.N, w.d, w.dtype, w.R, w.npp, w.entry, q, 5, 40, 2)
        assert (_u32(out2["ids"]) == _u32(ref2["ids"])).all() and (_u32(out2["dists"]) == _u32(ref2["dists"])).all()
    finally:
        ix.close()


def test_noalloc_entry_rejects_what_does_not_fit_its_scratch(gorio):
    w = make_config(1, scale=0.05, nq=8, with_gt=False)
    q = torch.as_tensor(w.queries).cuda()
    pages_dev = torch.as_tensor(w.pages).cuda()
    with pytest.raises(gorio.GorioError) as e:          # claims more pages than the array can track
        gorio.search_resident_noalloc(pages_dev, 40000, w.d, w.dtype, w.R, 1, 0, q, 10, 64, 4)
    assert e.value.status == 1 and "32768 pages" in str(e.value)
    with pytest.raises(gorio.GorioError) as e:          # W * max_degree beyond the per-query buffers
        gorio.search_resident_noalloc(pages_dev, w.N, w.d, w.dtype, w.R, w.npp, w.entry, q, 10, 64, 16)
    assert e.value.status == 1 and "W*max_degree" in str(e.value)
    # and it still works afterwards
    out = gorio.search_resident_noalloc(pages_dev, w.N, w.d, w.dtype, w.R, w.npp, w.entry, q, 10, 64, 4)
    assert _u32(out["ids"]).shape == (8, 10)
