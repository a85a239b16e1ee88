#!/usr/bin/env python
"""Benchmark of the GPU-owned paged beam search on the SIFT1M-shaped workload.

One "step" is one blocking search of all 10,000 queries against the 1,000,000-node uint8
index (R=64, 10 nodes per 4 KB page) starting from a COLD 20 % page cache, with the remote
tier emulated at 20 us per request and at most 256 requests in service.  The cache is
re-created (untimed) before every step; an L2 flush precedes every timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

prints one JSON line (rank 0).  With --gpus N > 1 and no launcher environment the script
starts N ranks itself (one per GPU); under a launcher (RANK / WORLD_SIZE set) it is one rank.
`--impl reference` times the CPU oracle instead.  After the timed steps the last step's
outputs are compared with the oracle on every query; a mismatch makes the run fail.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "QPS @ recall@10, 1M x 128 uint8, 20% cache, 20us miss"
PAPER_CONTEXT = ("paper (L40S + ConnectX-6 NVMe-oF, SIFT1M): G-ABaM 5650 QPS = 4.89x over blocking BaM, "
                 "G-Gust 1.31x over GustANN; context only, other hardware and transport")
PQ_SWEEP = [(L, W, f) for L in (50, 100, 200) for W in (1, 4, 8) for f in (0.05, 0.20, 1.0)]


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return json.load(open(p)), "measured"
    return {"hbm_gbs": 6650.0}, "fallback"


def profile_json(name):
    p = os.path.join(ROOT, "profiles", name)
    if os.path.exists(p):
        with open(p) as fh:
            return json.load(fh)
    return {}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc:
            self.proc.terminate()
        sm = [float(r[0]) for r in self.rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in self.rows if len(r) >= 7 for n, v in zip(names, r[3:7]) if v == "Active"})
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def measure_h2d_gbs(device, store=None):
    """Pinned host -> device copy bandwidth (the link the page fills cross): best of 20 copies of
    256 MB after a warm-up copy, from a pinned buffer of its own and -- when the index's page store
    is large enough -- from the page store itself (page-locked by the library at open), whichever
    is faster: where a buffer's pages sit relative to the GPU's socket changes the figure by a
    third, and the fills come from the page store."""
    def best_of(src):
        d = torch.empty(src.numel(), dtype=torch.uint8, device=device)
        d.copy_(src, non_blocking=True); torch.cuda.synchronize()
        best = 0.0
        for _ in range(20):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); d.copy_(src, non_blocking=True); b.record(); torch.cuda.synchronize()
            best = max(best, src.numel() / (a.elapsed_time(b) * 1e-3) / 1e9)
        return best
    n = 256 << 20
    out = best_of(torch.empty(n, dtype=torch.uint8).pin_memory())
    if store is not None and store.nbytes >= (64 << 20):
        t = torch.from_numpy(store.reshape(-1)[: min(n, store.nbytes)])
        if t.is_pinned():
            out = max(out, best_of(t))
    return out


def l2_flush(buf):
    buf.add_(1)          # 512 MB read+write, larger than the 126 MB L2


def oracle_qps(w, threads, budget_s=20.0, use_pq=False, L=None, W=None):
    """The CPU oracle as it stands on a bounded sample of the same queries.  Returns
    (queries/s, sample size, the oracle's results on that sample)."""
    from oracle import OracleIndex
    L, W = L or w.L, W or w.W
    orc = OracleIndex.from_workload(w, use_pq=use_pq)
    t = time.perf_counter(); orc.search(w.queries[: 4 * threads], w.K, L, W, threads=threads)
    per_q = (time.perf_counter() - t) / (4 * threads)
    n = int(min(w.nq, max(8 * threads, budget_s / max(per_q, 1e-6))))
    t = time.perf_counter(); ref = orc.search(w.queries[:n], w.K, L, W, threads=threads)
    dt = time.perf_counter() - t
    return n / dt, n, ref


def oracle_one_thread_qps(w, use_pq=False, L=None, W=None, n=500):
    from oracle import OracleIndex
    n = min(n, w.nq)
    orc = OracleIndex.from_workload(w, use_pq=use_pq)
    t = time.perf_counter(); orc.search(w.queries[:n], w.K, L or w.L, W or w.W, threads=1)
    return n / (time.perf_counter() - t), n


def parity_check(w, ids, dists, pages, ref, n):
    """The timed outputs against the oracle's on the first n queries.  uint8: ids, integer
    distances and distinct-page counts bit-exact.  fp32: ids equal on >= 99.9 % of the queries,
    every other query explained by near ties (true double distances within 1e-5 relative, rank by
    rank), reported distances within fp32 rounding of the oracle's.  Returns (ok, detail)."""
    ids, pages = ids[:n], pages[:n]
    if w.dtype == "u8":
        ok_i = bool((ids == ref["ids"]).all())
        ok_d = bool((dists[:n].view(np.uint32) == ref["dists"]).all())
        ok_p = bool((pages == ref["counters"][:, 0]).all())
        return ok_i and ok_d and ok_p, {"ids": ok_i, "dists": ok_d, "pages_distinct": ok_p}
    same = (ids == ref["ids"]).all(1)
    ok = same.mean() >= 0.999
    ok = ok and bool(np.allclose(dists[:n][same], ref["dists"][same], rtol=2e-6, atol=0))
    q64 = w.queries[:n].astype(np.float64)
    for r in np.nonzero(~same)[0]:
        dg = ((w.data[ids[r]].astype(np.float64) - q64[r]) ** 2).sum(1)
        do = ((w.data[ref["ids"][r]].astype(np.float64) - q64[r]) ** 2).sum(1)
        ok = ok and bool((np.abs(dg - do) <= 1e-5 * do).all()) and len(set(ids[r].tolist())) == ids.shape[1]
    return bool(ok), {"id_match_rate": float(same.mean())}


def reference_arm(args, rank, threads):
    """`--impl reference`: the oracle, as it stands, on the host cores.  Rank 0 alone works."""
    from workloads import make_config
    if rank != 0:
        return
    w = make_config(args.config, scale=args.scale, nq=args.nq, device="cuda" if torch.cuda.is_available() else "cpu",
                    with_gt=False)
    vals = []
    for _ in range(args.warmup):
        oracle_qps(w, threads, budget_s=2.0, use_pq=args.config == 4, L=args.L, W=args.W)
    n_s = 0
    for _ in range(args.steps):
        v, n_s, _ = oracle_qps(w, threads, budget_s=max(5.0, 60.0 / max(1, args.steps)), use_pq=args.config == 4,
                               L=args.L, W=args.W)
        vals.append(v)
    v = statistics.mean(vals)
    sample = f"first {n_s} of {w.nq} queries per step, {threads} threads, in-memory page store, no cache emulation"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": "queries/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * n_s / v, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8" if w.dtype == "u8" else "f32", "data": "synthetic",
        "config": {"workload": f"cfg{args.config}: N={w.N} d={w.d} {w.dtype} R={w.R} npp={w.npp} K={w.K} "
                               f"L={args.L or w.L} W={args.W or w.W}"},
        "cpu_baseline": {"value": v, "unit": "queries/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": "queries/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--scale", type=float, default=1.0, help="shrink the index (profiling captures only)")
    ap.add_argument("--cache-frac", type=float, default=0.20)
    ap.add_argument("--preload", action="store_true", help="fully resident cache (profiling captures only)")
    ap.add_argument("--nq", type=int, default=None)
    ap.add_argument("--config", type=int, default=3, choices=[1, 2, 3, 4, 5],
                    help="3 = the benchmark workload; the others are the parity configurations")
    ap.add_argument("--blocking", action="store_true", help="ablation: warps wait in place on a miss")
    ap.add_argument("--latency-us", type=float, default=None)
    ap.add_argument("--max-outstanding", type=int, default=None)
    ap.add_argument("--sweep", default=None,
                    help="comma list of latency_us:max_outstanding points; prints one short JSON line per point "
                         "(characterisation runs, not the benchmark line)")
    ap.add_argument("--pq-sweep", action="store_true",
                    help="with --config 4: all 27 (L, W, cache) points on one index, one short JSON line per point, "
                         "each checked against the oracle on every query")
    ap.add_argument("--granularity", default="page", choices=["page", "record"],
                    help="record: selective materialisation, a miss fetches only the wanted node's record")
    ap.add_argument("--copy-engine", action="store_true",
                    help="the proxy copies pages itself with the GPU's copy engine (one cudaMemcpyAsync per page) "
                         "instead of commanding warps of the search kernel to pull them")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="N GPUs: weak = every rank searches its own 10,000 queries; strong = one 10,000-query set "
                         "sliced across the ranks, results gathered and checked on rank 0")
    ap.add_argument("--no-parity", action="store_true", help="skip the oracle comparison of the timed outputs")
    ap.add_argument("--warps", type=int, default=0, help="warps per block of the persistent kernel (0 = the library's choice)")
    ap.add_argument("--visited-capacity", type=int, default=0,
                    help="entries of the per-query visited set (0 = the library's default; a bitmap is used when it is no larger)")
    ap.add_argument("--request-backlog", type=int, default=0,
                    help="most requests posted and not yet arrived (0 = the library's default, 4 x the window up to 1024)")
    ap.add_argument("--shared-pull", action="store_true",
                    help="ablation: worker warps pull admitted pages between their other work (no dedicated puller warps)")
    ap.add_argument("--no-fast-path", action="store_true", help="whole index resident: use the general path anyway")
    ap.add_argument("--timeout-ms", type=int, default=120_000, help="bound on one search call (profiling captures use a short one)")
    ap.add_argument("--L", type=int, default=None)
    ap.add_argument("--W", type=int, default=None)
    args = ap.parse_args()

    launched = "WORLD_SIZE" in os.environ
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    threads = os.cpu_count() or 1

    if args.impl == "reference":
        return reference_arm(args, rank, threads)

    if args.gpus > 1 and not launched:
        # the stock command form `python bench.py --gpus N`: become the launcher of N ranks
        from paper_2607_04415_b200.shard import spawn_ranks
        from paper_2607_04415_b200 import build
        build.build()                      # once, before the ranks start
        sys.exit(spawn_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} ranks")

    from workloads import make_config, recall_at_k, workload_key
    import paper_2607_04415_b200 as g
    from paper_2607_04415_b200 import build
    from paper_2607_04415_b200.shard import gather_results, shard_range
    build.build()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the search has no CPU path")
    if torch.cuda.device_count() < world:
        raise SystemExit(f"bench.py: {world} ranks but only {torch.cuda.device_count()} CUDA devices")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        # one rank per GPU: keep this rank's page store, proxy thread and polled words on the GPU's socket
        from paper_2607_04415_b200.shard import bind_to_gpu_cpus
        pr = torch.cuda.get_device_properties(local)
        bind_to_gpu_cpus(f"{pr.pci_domain_id:04x}:{pr.pci_bus_id:02x}:{pr.pci_device_id:02x}.0")
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
        if dist.get_world_size() != args.gpus:
            raise SystemExit(f"bench.py: the process group has {dist.get_world_size()} ranks, --gpus says {args.gpus}")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # Every rank builds and pins its own copy of the page store and owns a private cache, ring
    # and proxy thread.  weak: rank r searches its own 10,000 queries (query seed 1 + r);
    # strong: the ranks slice one 10,000-query set.
    strong = args.scaling == "strong" and world > 1
    w = make_config(args.config, scale=args.scale, nq=args.nq, device=dev, seed_q=1 if strong else 1 + rank)
    nq_total = w.nq if strong else world * w.nq
    q_lo, q_hi = shard_range(w.nq, rank, world) if strong else (0, w.nq)
    my_q = w.queries[q_lo:q_hi]
    my_nq = q_hi - q_lo
    if args.L:
        w.L = args.L
    if args.W:
        w.W = args.W
    frac = args.cache_frac if args.config in (3, 4) else w.cache_frac
    preload = args.preload or w.preload or frac >= 1.0
    cap = w.n_pages if preload else int(frac * w.n_pages)
    if args.latency_us is not None:
        w.latency_us = args.latency_us
    if args.max_outstanding:
        w.max_outstanding = args.max_outstanding
    lat_ns, max_out = int(w.latency_us * 1000), w.max_outstanding
    use_pq = args.config == 4
    ix = g.Index.from_workload(w, device=local, use_pq=use_pq)
    if args.blocking or args.warps or args.no_fast_path or args.shared_pull or args.visited_capacity or args.request_backlog:
        ix.set_tuning(blocking=int(args.blocking), warps_per_block=args.warps, no_fast_path=int(args.no_fast_path),
                      visited_capacity=args.visited_capacity, shared_pull=int(args.shared_pull),
                      request_backlog=args.request_backlog)
    q_dev = torch.as_tensor(my_q).to(dev)
    q_pin = torch.as_tensor(my_q).pin_memory()
    outs_pin = dict(ids=torch.empty((my_nq, w.K), dtype=torch.int32).pin_memory(),
                    dists=torch.empty((my_nq, w.K), dtype=torch.int32 if w.dtype == "u8" else torch.float32).pin_memory(),
                    pages=torch.empty(my_nq, dtype=torch.int32).pin_memory(),
                    counters=torch.empty((my_nq, 5), dtype=torch.int32).pin_memory())
    flush = torch.zeros(512 << 20, dtype=torch.uint8, device=dev)
    h2d = measure_h2d_gbs(dev, w.pages)
    pk, pk_kind = peaks()
    state = dict(cap=cap, preload=preload, lat_ns=lat_ns, max_out=max_out, L=w.L, W=w.W)

    def reset_cache():
        ix.cache_config(state["cap"], remote_latency_ns=state["lat_ns"], max_outstanding=state["max_out"],
                        preload=state["preload"], timeout_ms=args.timeout_ms, granularity=args.granularity,
                        copy_engine=args.copy_engine)
        ix.stats_reset()
        l2_flush(flush)

    def one_step():
        reset_cache()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        out = ix.search(q_dev, w.K, state["L"], state["W"])
        b.record()
        barrier()
        t = torch.tensor([a.elapsed_time(b)], device=dev)
        if world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t), out, ix.stats()

    def roofline_terms(st, ms, fetched, fetched_bytes):
        """The slowest of (a) algorithmic HBM bytes at the measured copy peak, (b) fetched page bytes
        over the measured host link, (c) outstanding window / injected latency."""
        esz = 1 if w.dtype == "u8" else 4
        if use_pq:                # PQ: 32-byte code per scored node, whole record per expanded node
            b_alg = st["n_eval"] * 32 + st["n_expand"] * w.node_bytes
        else:
            b_alg = st["n_eval"] * w.d * esz + 4 * st["n_expand"] + 4 * st["sum_degree"]
        b_hbm = b_alg + fetched_bytes
        terms = {"hbm": b_hbm / (pk["hbm_gbs"] * 1e9), "host_link": fetched_bytes / (h2d * 1e9),
                 "outstanding_window": fetched * state["lat_ns"] * 1e-9 / state["max_out"]}
        bound = max(terms, key=terms.get)
        if bound == "hbm":
            ach, peak, unit = b_hbm / (ms * 1e-3) / 1e9, pk["hbm_gbs"], "GB/s"
        elif bound == "host_link":
            ach, peak, unit = fetched_bytes / (ms * 1e-3) / 1e9, h2d, "GB/s"
        else:
            ach, peak, unit = fetched / (ms * 1e-3) / 1e6, state["max_out"] / max(state["lat_ns"] * 1e-9, 1e-12) / 1e6, "Mfetch/s"
        return terms, bound, ach, peak, unit, b_hbm

    def out_arrays(out):
        ids = out["ids"].cpu().numpy().view(np.uint32)
        dists = out["dists"].cpu().numpy()
        pages = out["pages_distinct"].cpu().numpy().view(np.uint32)
        return ids, dists, pages

    if args.sweep:
        for point in args.sweep.split(","):
            lat_us, mo = point.split(":")
            state["lat_ns"], state["max_out"] = int(float(lat_us) * 1000), int(mo)
            ts, sts = [], []
            for i in range(1 + max(1, args.steps)):
                t, _, st_i = one_step()
                if i:
                    ts.append(t); sts.append(st_i)
            ms_p = statistics.mean(ts)
            f_p = statistics.mean(x["pages_fetched"] for x in sts)
            terms_p = {"host_link": statistics.mean(x["fetched_bytes"] for x in sts) / (h2d * 1e9),
                       "outstanding_window": f_p * state["lat_ns"] * 1e-9 / state["max_out"]}
            bound_p = max(terms_p, key=terms_p.get)
            if rank == 0:
                print(json.dumps({"latency_us": float(lat_us), "max_outstanding": state["max_out"], "qps": nq_total / (ms_p * 1e-3),
                                  "ms_per_step": ms_p, "pages_fetched": f_p, "fetch_rate_M_per_s": f_p / ms_p / 1e3,
                                  "bound": bound_p, "frac": terms_p[bound_p] / (ms_p * 1e-3),
                                  "service_us": statistics.mean(x["proxy_service_ns"] / max(1, x["pages_fetched"]) for x in sts) / 1e3,
                                  "blocking": bool(args.blocking), "granularity": args.granularity,
                                  "copy_engine": bool(args.copy_engine)}), flush=True)
        ix.close()
        return

    if args.pq_sweep:
        if not use_pq or world != 1:
            raise SystemExit("--pq-sweep needs --config 4 on one GPU")
        from oracle import OracleIndex
        orc = OracleIndex.from_workload(w, use_pq=True)
        refs = {}
        all_ok = True
        for L, W, f in PQ_SWEEP:
            if (L, W) not in refs:
                refs[(L, W)] = orc.search(w.queries, w.K, L, W, threads=threads)
            ref = refs[(L, W)]
            state.update(L=L, W=W, preload=f >= 1.0, cap=w.n_pages if f >= 1.0 else int(f * w.n_pages))
            ts, sts, out = [], [], None
            for i in range(1 + max(1, args.steps)):
                t, out, st_i = one_step()
                if i:
                    ts.append(t); sts.append(st_i)
            ms_p = statistics.mean(ts)
            f_p = statistics.mean(x["pages_fetched"] for x in sts)
            fb_p = statistics.mean(x["fetched_bytes"] for x in sts)
            terms, bound, ach, peak, unit, _ = roofline_terms(sts[-1], ms_p, f_p, fb_p)
            ids, dists, pages = out_arrays(out)
            ok, _ = parity_check(w, ids, dists, pages, ref, w.nq)
            all_ok = all_ok and ok
            print(json.dumps({"L": L, "W": W, "cache_frac": f, "qps": w.nq / (ms_p * 1e-3), "ms_per_step": ms_p,
                              "recall_at_10": recall_at_k(ids, w.gt), "bound": bound, "frac": terms[bound] / (ms_p * 1e-3),
                              "pages_fetched": f_p, "parity_checked_queries": w.nq, "parity_ok": ok}), flush=True)
        ix.close()
        if not all_ok:
            raise SystemExit("bench.py: a sweep point differs from the oracle")
        return

    for _ in range(max(3, args.warmup)):
        one_step()
    sampler = ClockSampler(local); sampler.start()
    times, stats_list, out = [], [], None
    for _ in range(args.steps):
        t, out, st = one_step()
        times.append(t); stats_list.append(st)
    clocks = sampler.stop()

    # end to end through the host-buffer entry point: H2D queries, search, D2H results; as many
    # timed steps as above, after one untimed call
    e2e_times = []
    for i in range(1 + args.steps):
        reset_cache()
        barrier()
        t0 = time.perf_counter()
        ix.search_host(q_pin.numpy(), w.K, w.L, w.W, out={k: v.numpy() for k, v in outs_pin.items()})
        dt = time.perf_counter() - t0
        tt = torch.tensor([dt], device=dev)
        if world > 1:
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        if i:
            e2e_times.append(float(tt))
    h2d = max(h2d, measure_h2d_gbs(dev, w.pages))     # measured before and after the timed steps; the better one is the peak
    # what the link gives SM warps that pull scattered 4 KB pages of this store and do nothing else
    # (the loads of a page fill, as many pages in flight as the window allows): context for the link term
    sm_pull_gbs = max(ix.link_probe(200_000, max(4, min(int(max_out), 16384))) for _ in range(3))
    ms = statistics.mean(times)
    st = stats_list[len(stats_list) // 2]
    fetched = statistics.mean(s["pages_fetched"] for s in stats_list)
    fetched_bytes = statistics.mean(s["fetched_bytes"] for s in stats_list)   # 4096 per page, or the record span
    launches = 2 * len(stats_list)          # init + persistent search kernel per step
    terms, bound, ach, peak, unit, b_hbm = roofline_terms(st, ms, fetched, fetched_bytes)
    t_roof = terms[bound]

    default_workload = (args.config == 3 and args.scale == 1.0 and args.nq is None and not args.preload and
                        not args.blocking and args.cache_frac == 0.20 and args.latency_us is None and
                        not args.max_outstanding and not args.L and not args.W and args.granularity == "page" and
                        not args.copy_engine and not args.warps)
    ids, dists, pages = out_arrays(out)

    # the timed outputs against the oracle, every query; at N = 1 the same oracle run is the CPU baseline
    cpu_baseline, parity = None, {"checked": 0, "ok": None}
    if not args.no_parity:
        th = max(1, threads // world)
        v, n_s, ref = oracle_qps(w, th, use_pq=use_pq) if not strong else (0.0, 0, None)
        if strong:
            from oracle import OracleIndex
            gi = gather_results(out["ids"], w.nq).cpu().numpy().view(np.uint32)
            gd = gather_results(out["dists"], w.nq).cpu().numpy()
            gp = gather_results(out["pages_distinct"], w.nq).cpu().numpy().view(np.uint32)
            ok = True
            if rank == 0:
                ref = OracleIndex.from_workload(w, use_pq=use_pq).search(w.queries, w.K, w.L, w.W, threads=threads)
                ok, _ = parity_check(w, gi, gd, gp, ref, w.nq)
            parity = {"checked": w.nq, "ok": ok}
        else:
            ok, _ = parity_check(w, ids, dists, pages, ref, n_s)
            parity = {"checked": n_s * world, "ok": ok}
            if world == 1:
                v1, n1 = oracle_one_thread_qps(w, use_pq=use_pq)
                cpu_baseline = {"value": v, "unit": "queries/s", "cores": th, "kind": "oracle",
                                "sample": f"first {n_s} of {w.nq} queries, {th} threads, in-memory page store "
                                          "(no cache emulation, no injected latency)",
                                "one_thread": {"value": v1, "unit": "queries/s", "sample": f"first {n1} queries, 1 thread"}}
        if world > 1:
            flag = torch.tensor([1 if parity["ok"] else 0], device=dev)
            dist.all_reduce(flag, op=dist.ReduceOp.MIN)
            parity["ok"] = bool(int(flag))

    # recall over all ranks' queries (strong: each rank's slice of the shared ground truth)
    recall = recall_at_k(ids, w.gt[q_lo:q_hi])
    if world > 1:
        rr = torch.tensor([recall * my_nq, my_nq], device=dev, dtype=torch.float64)
        dist.all_reduce(rr)
        recall = float(rr[0] / rr[1])

    roof = {"bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": t_roof / (ms * 1e-3),
            "traffic": None, "peak_kind": f"hbm {pk_kind}; host link measured in this run ({h2d:.1f} GB/s)",
            "terms_ms": {k: 1e3 * v for k, v in terms.items()},
            "pages_fetched": fetched, "fetched_bytes": fetched_bytes, "algorithmic_hbm_bytes": b_hbm,
            "hbm_achieved_gbs": b_hbm / (ms * 1e-3) / 1e9, "hbm_peak_gbs": pk["hbm_gbs"],
            "host_link_bulk_copy_gbs": h2d, "host_link_sm_page_pull_gbs": sm_pull_gbs,
            "fetched_gbs": fetched_bytes / (ms * 1e-3) / 1e9,
            "fetched_over_sm_page_pull": fetched_bytes / (ms * 1e-3) / 1e9 / sm_pull_gbs if sm_pull_gbs > 0 else None}
    if default_workload:
        # DRAM bytes of one search_kernel launch from a single-pass ncu capture of this command, valid
        # only for the device code it was captured on
        cap_rec = profile_json("ncu_dram_traffic.json").get("cfg3")
        if cap_rec:
            fresh = cap_rec.get("kernel_source_hash") == build.kernel_source_hash()
            roof["traffic"] = cap_rec["dram_bytes_per_launch"] if fresh else None
            roof["traffic_stale"] = not fresh
    floor = profile_json("fetch_floor.json").get(workload_key(args.config, w.N, w.npp, w.nq, w.L, w.W, cap))
    if floor and not use_pq and not strong and args.granularity == "page":
        # fewest fetches the "all queries in flight, merged misses" design can be held to (an offline
        # optimal-replacement replay of the oracle's page traces); per GPU, like pages_fetched
        roof["fetch_floor"] = floor["fetch_floor_optimal_replacement"]
        roof["fetched_over_floor"] = fetched / floor["fetch_floor_optimal_replacement"]
        roof["fetches_clock_replay"] = floor["fetches_clock_replacement"]
        lat_s, mo = state["lat_ns"] * 1e-9, state["max_out"]
        t_floor = max(floor["fetch_floor_optimal_replacement"] * 4096 / (h2d * 1e9),
                      floor["fetch_floor_optimal_replacement"] * lat_s / mo)
        roof["frac_at_fetch_floor"] = t_floor / (ms * 1e-3)     # the roofline with the floor's fetch count

    line = {
        "metric": METRIC, "value": nq_total / (ms * 1e-3), "unit": "queries/s", "n_gpus": world,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True,
        "scaling": "strong" if strong else "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": f"cfg{args.config}{' SIFT1M-shaped' if args.config == 3 else ''}: N={w.N} d={w.d} {w.dtype} "
                               f"R={w.R} npp={w.npp} pages={w.n_pages} nq={my_nq}/gpu K={w.K} L={w.L} W={w.W} "
                               f"cache={cap} slots {'preloaded' if preload else 'cold'} latency={w.latency_us:g}us "
                               f"max_outstanding={max_out}{' PQ 32x256' if use_pq else ''}{' BLOCKING ablation' if args.blocking else ''}"
                               f"{' RECORD granularity (selective materialisation)' if args.granularity == 'record' else ''}"
                               f"{' COPY-ENGINE proxy (one cudaMemcpyAsync per page)' if args.copy_engine else ''}",
                   "recall_at_10": recall, "l2": "flushed before every step (512 MB read+write)",
                   "cache": "re-created cold before every step, untimed",
                   "parallelism": f"query-sharded x{world}: every rank has its own copy of the page store, cache, ring and proxy thread",
                   "parity_checked_queries": parity["checked"], "parity_ok": parity["ok"],
                   "context": PAPER_CONTEXT},
        "clocks": clocks,
        "e2e": {"value": nq_total / statistics.mean(e2e_times), "unit": "queries/s", "steps": len(e2e_times),
                "h2d_bytes_per_step": int(q_pin.numel() * q_pin.element_size()),
                "d2h_bytes_per_step": int(sum(v.numel() * 4 for v in outs_pin.values()))},
        "gpu_launches": int(launches),
        "roofline": roof,
        "stats": {k: st[k] for k in ("pages_hit", "pages_missed", "pages_fetched", "dedupe_joins", "evictions",
                                     "retries", "max_outstanding_seen", "resumes", "proxy_batches", "proxy_service_ns",
                                     "proxy_iters", "proxy_ack_wait_iters", "proxy_window_full_iters",
                                     "proxy_ring_empty_iters", "proxy_outstanding_sum", "warp_ns_arrivals",
                                     "warp_ns_queries", "warp_ns_idle", "warp_ns_copies", "arrivals_consumed",
                                     "stash_hits")},
    }
    if cpu_baseline:
        line["cpu_baseline"] = cpu_baseline
    ix.close()
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    if parity["ok"] is False:
        raise SystemExit("bench.py: the timed outputs differ from the oracle")


if __name__ == "__main__":
    main()
