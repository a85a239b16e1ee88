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


def test_binding_rejects_wrong_shapes_types_and_sizes_before_any_pointer_is_passed():
    """The library sees raw pointers only, so the binding checks what it cannot: a wrong-shaped,
    wrong-typed, non-contiguous, misplaced or misaligned tensor is an INVALID_ARG error, never
    an out-of-bounds device access."""
    import paper_2607_04415_b200.binding as b
    good = torch.zeros((8, 128), dtype=torch.uint8)
    for bad in (torch.zeros(128, dtype=torch.uint8),                  # not 2-D
                torch.zeros((8, 64), dtype=torch.uint8),              # wrong width
                torch.zeros((8, 128), dtype=torch.float32),           # wrong element type
                torch.zeros((128, 8), dtype=torch.uint8).t(),         # right shape, not contiguous
                good):                                                # not on a CUDA device
        with pytest.raises(b.GorioError) as e:
            b.check_queries(bad, 128, "u8", 0)
        assert e.value.status == 1
    with pytest.raises(b.GorioError) as e:
        b.check_queries(torch.zeros((8, 96), dtype=torch.uint8), 96, "f32")
    assert e.value.status == 1
    cpu = torch.device("cpu")
    pages = torch.zeros(4 * 4096, dtype=torch.uint8)
    for args in ((pages, 0, 1), (pages, 4, 0), (pages.to(torch.int32), 4, 1), (pages[::2], 2, 1)):
        with pytest.raises(b.GorioError) as e:
            b.check_resident_pages(args[0], args[1], args[2], cpu)
        assert e.value.status == 1


def test_c_entries_reject_misaligned_pointers_and_oversized_indexes_without_a_gpu(lib):
    import paper_2607_04415_b200.binding as b
    d = b._IndexDesc()
    d.n_nodes, d.dim, d.dtype, d.max_degree, d.nodes_per_page, d.page_bytes, d.entry_id = 100, 128, 0, 32, 1, 4096, 0
    fake = 0x10000                                        # never dereferenced: validation fails first
    call = lambda desc, pages, q, ids: lib.gorio_search_resident_noalloc(ctypes.byref(desc), pages, q, 4, 10, 64, 4,
                                                                         ids, fake, None, None)
    assert call(d, fake + 2, fake, fake) == 1             # pages not 4-byte aligned
    assert call(d, fake, fake + 1, fake) == 1             # queries not 4-byte aligned
    assert call(d, fake, fake, fake + 2) == 1             # outputs not 4-byte aligned
    assert b"aligned" in lib.gorio_last_error(None)
    d.n_nodes = 1 << 31                                   # the list key keeps ids in 31 bits
    assert call(d, fake, fake, fake) == 1
    d.n_nodes = (1 << 64) - 1                             # n_nodes + nodes_per_page - 1 must not wrap
    assert call(d, fake, fake, fake) == 1


def _stub_rank_script(tmp_path):
    p = tmp_path / "stub_rank.py"
    p.write_text(
        "import os, sys, torch, torch.distributed as dist\n"
        "dist.init_process_group('gloo')\n"
        "r, w = dist.get_rank(), dist.get_world_size()\n"
        "assert r == int(os.environ['RANK']) and w == int(os.environ['WORLD_SIZE']) == int(sys.argv[1])\n"
        "assert int(os.environ['LOCAL_RANK']) == r and os.environ['MASTER_ADDR'] == '127.0.0.1'\n"
        "t = torch.tensor([float(r + 1)]); dist.all_reduce(t, op=dist.ReduceOp.MAX)\n"
        "open(os.path.join(sys.argv[2], f'rank{r}.txt'), 'w').write(f'{w} {t.item()}')\n"
        "dist.destroy_process_group()\n"
        "sys.exit(3 if (len(sys.argv) > 3 and r == 1) else 0)\n")
    return str(p)


def test_spawn_ranks_starts_one_process_per_rank_with_the_launcher_environment(tmp_path):
    from paper_2607_04415_b200.shard import spawn_ranks
    script = _stub_rank_script(tmp_path)
    assert spawn_ranks(2, script, ["2", str(tmp_path)], timeout=300) == 0
    for r in range(2):
        assert (tmp_path / f"rank{r}.txt").read_text() == "2 2.0"
    # a failing rank makes the launch fail
    assert spawn_ranks(2, script, ["2", str(tmp_path), "fail"], timeout=300) != 0


def test_bench_reference_arm_with_two_gpus_still_prints_one_line():
    import json
    import subprocess
    import sys
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--config", "3",
                          "--scale", "0.01", "--nq", "64", "--steps", "1", "--warmup", "1"],
                         capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-800:]
    lines = [ln for ln in out.stdout.strip().splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0


def test_bench_refuses_a_world_size_that_differs_from_gpus():
    import subprocess
    import sys
    env = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--steps", "1"],
                         capture_output=True, text=True, timeout=300, cwd=ROOT, env=env)
    assert out.returncode != 0 and "--gpus 4" in (out.stderr + out.stdout)


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


def test_bind_to_gpu_cpus_follows_sysfs_and_is_a_no_op_when_it_cannot_help(tmp_path):
    """The rank-to-socket binding reads the PCI device's local_cpulist: it narrows the affinity to the
    CPUs named there that this process may use, and leaves it alone when the file is missing, names
    none of them, or names all of them."""
    import os
    from paper_2607_04415_b200.shard import bind_to_gpu_cpus, parse_cpulist
    assert parse_cpulist("0-3,8,10-11\n") == {0, 1, 2, 3, 8, 10, 11}
    allowed = os.sched_getaffinity(0)
    dev = tmp_path / "bus/pci/devices/0000:aa:00.0"
    dev.mkdir(parents=True)
    try:
        assert not bind_to_gpu_cpus("0000:bb:00.0", str(tmp_path))                 # no such device
        (dev / "local_cpulist").write_text(",".join(str(c) for c in sorted(allowed)) + "\n")
        assert not bind_to_gpu_cpus("0000:aa:00.0", str(tmp_path))                 # names every allowed CPU
        (dev / "local_cpulist").write_text(str(max(allowed) + 1000) + "\n")
        assert not bind_to_gpu_cpus("0000:aa:00.0", str(tmp_path))                 # names none of them
        assert os.sched_getaffinity(0) == allowed
        if len(allowed) > 1:
            one = min(allowed)
            (dev / "local_cpulist").write_text(f"{one}\n")
            assert bind_to_gpu_cpus("0000:aa:00.0", str(tmp_path))
            assert os.sched_getaffinity(0) == {one}
    finally:
        os.sched_setaffinity(0, allowed)
