"""Host-side checks that need no GPU: the C-ABI library loads and exports every function the
header declares, argument validation that precedes any CUDA call, and the query-sharding
logic under a 2-rank gloo group."""
import ctypes
import os
import re
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2607_04415_b200 import build
    build.build()
    import paper_2607_04415_b200 as g
    return g.load_library()


def test_library_exports_every_declared_entry_point(lib):
    import paper_2607_04415_b200 as g
    header = open(os.path.join(ROOT, "include", "gorio.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(gorio_[a-z_]+)\s*\(", header))
    assert declared, "no declarations parsed"
    assert declared == set(g.EXPORTED_SYMBOLS)
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in gorio.h but not exported"


def test_status_strings(lib):
    seen = {lib.gorio_status_str(i) for i in range(9)}
    assert len(seen) == 9 and all(s for s in seen)
    assert lib.gorio_status_str(12345) == b"unknown status"


def test_argument_validation_happens_before_any_cuda_call(lib):
    import paper_2607_04415_b200.binding as b
    h = ctypes.c_void_p()
    assert lib.gorio_index_open(None, 0, ctypes.byref(h)) == 1
    pages = np.zeros((4, 4096), dtype=np.uint8)
    d = b._IndexDesc()
    d.n_nodes, d.dim, d.dtype, d.max_degree, d.nodes_per_page, d.page_bytes = 4, 128, 0, 32, 1, 4096
    d.entry_id, d.host_pages = 0, pages.ctypes.data
    for field, bad in (("page_bytes", 8192), ("dim", 130), ("nodes_per_page", 20), ("entry_id", 4),
                       ("max_degree", 0), ("dtype", 2), ("n_nodes", 0)):
        old = getattr(d, field)
        setattr(d, field, bad)
        assert lib.gorio_index_open(ctypes.byref(d), 0, ctypes.byref(h)) == 1, field
        setattr(d, field, old)
    d.pq_m = 32                                            # PQ without device arrays
    assert lib.gorio_index_open(ctypes.byref(d), 0, ctypes.byref(h)) == 1
    assert lib.gorio_cache_config(None, None) == 1
    assert lib.gorio_stats(None, None) == 1
    assert lib.gorio_index_close(None) == 1
    assert not h.value


def test_missing_library_fails_loudly(monkeypatch):
    import paper_2607_04415_b200.binding as b
    monkeypatch.setattr(b, "_LIB", None)
    monkeypatch.setattr(b, "lib_path", lambda: "/nonexistent/libgorio.so")
    with pytest.raises(b.GorioError):
        b.load_library()


def test_shard_ranges_cover_every_query_once():
    from paper_2607_04415_b200.shard import shard_range
    for nq in (1, 7, 10_000, 10_001):
        for world in (1, 2, 3, 8):
            cover = []
            for r in range(world):
                b, e = shard_range(nq, r, world)
                cover.extend(range(b, e))
            assert cover == list(range(nq))


def _rank_main(rank, world, port, nq, out):
    from paper_2607_04415_b200.shard import gather_results, shard_range
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    b, e = shard_range(nq, rank, world)
    local = torch.arange(b, e, dtype=torch.int32)[:, None] * torch.tensor([[1, 10]], dtype=torch.int32)
    full = gather_results(local, nq)
    # max-over-ranks timing reduction used by the benchmark
    t = torch.tensor([float(rank + 1)])
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        out.put((full.tolist(), float(t)))
    dist.destroy_process_group()


def test_two_rank_gloo_gather_restores_global_order():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    nq = 11
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, nq, out)) for r in range(2)]
    for p in procs:
        p.start()
    full, tmax = out.get(timeout=120)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert full == [[i, 10 * i] for i in range(nq)]
    assert tmax == 2.0


def test_bench_reference_arm_prints_the_contract_line_on_cpu():
    """`bench.py --impl reference` times the oracle and needs no GPU: one JSON line with the
    contract's keys, on a shrunken workload so that the CPU suite stays short."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--config", "3",
                          "--scale", "0.01", "--nq", "64", "--steps", "1", "--warmup", "1"],
                         capture_output=True, text=True, timeout=300, cwd=root)
    assert out.returncode == 0, out.stderr[-800:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["impl"] == "reference" and line["value"] > 0 and line["vs_baseline"] is None
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
