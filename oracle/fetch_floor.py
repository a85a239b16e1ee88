#!/usr/bin/env python
"""How few page fetches can a batch get away with?  -- MEASUREMENT INFRASTRUCTURE ONLY.

The benchmark's roofline terms (host link, outstanding window) both scale with the number
of pages the implementation fetched, so the fraction alone cannot tell a frugal run from a
wasteful one.  This script derives, from the CPU oracle's per-query traces and nothing
else, a floor for that number under the model the benchmark configuration implies:

  * all nq queries are in flight and advance in lock step, one search iteration per round;
  * requests for the same page in the same round merge into one fetch (miss dedupe);
  * between rounds the cache keeps `slots` pages chosen with full knowledge of the future
    (furthest-next-use replacement, the offline optimum for unit-size pages);
  * only the pages of newly scored nodes count (an implementation may keep the adjacency
    list of a node from the moment it was scored, so expansions need no page of their own).

A clock-replacement replay of the same rounds (second-chance bits, the policy the CUDA path
uses) is reported beside it.  Neither is a bound over every conceivable schedule (a batch
that is not in lock step sees a different request stream); they pin the fetch count that
the "all queries in flight" design can be held to.

Calls only oracle/ and workloads/.  Usage:

    python oracle/fetch_floor.py [--config 3] [--scale 1.0] [--nq N] [--procs P] [--out profiles/fetch_floor.json]

The result is merged into the JSON file under a key that names the workload.
"""
from __future__ import annotations

import argparse
import json
import multiprocessing as mp
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

_W = None      # the workload, inherited by forked workers


def _query_rounds(args):
    """Pages of the newly scored nodes of every iteration of queries [b, e), from the oracle's
    frontier trace: [(round, page array)], plus self-checks against the oracle's counters."""
    from oracle import OracleIndex
    b, e = args
    w = _W
    orc = OracleIndex.from_workload(w)
    seen = np.zeros(w.N, dtype=bool)
    out = []
    for qi in range(b, e):
        tr = orc.search_trace(w.queries[qi], w.K, w.L, w.W)
        touched = [np.array([w.entry], dtype=np.int64)]
        seen[w.entry] = True
        rounds = [(0, np.array([w.entry // w.npp], dtype=np.int64))]
        for t, (front, _lst) in enumerate(tr["iterations"], start=1):
            f = np.asarray(front, dtype=np.int64)
            nb = w.nbrs[f]                                          # [|F|, R]
            valid = np.arange(w.R)[None, :] < w.deg[f][:, None]
            nb = np.unique(nb[valid].astype(np.int64))
            new = nb[~seen[nb]]
            seen[new] = True
            touched.append(new)
            if new.size:
                rounds.append((t, np.unique(new // w.npp)))
        allv = np.concatenate(touched)
        seen[allv] = False
        cnt = tr["counters"]
        assert allv.size == int(cnt[3]), "re-derived visited set differs from the oracle's n_eval"
        pages = np.unique(np.concatenate([allv, np.concatenate([np.asarray(fr, dtype=np.int64) for fr, _ in tr["iterations"]])]) // w.npp)
        assert pages.size == int(cnt[0]), "re-derived page set differs from the oracle's pages_distinct"
        out.append(rounds)
    return out


def replay_optimal(need: np.ndarray, slots: int) -> int:
    """need[r, p]: page p is wanted in round r.  Fetches with furthest-next-use replacement."""
    n_rounds, n_pages = need.shape
    big = n_rounds + 1
    nxt = np.full((n_rounds + 1, n_pages), big, dtype=np.int32)      # nxt[r, p]: first round >= r that wants p
    for r in range(n_rounds - 1, -1, -1):
        nxt[r] = np.where(need[r], r, nxt[r + 1])
    cache = np.zeros(n_pages, dtype=bool)
    fetched = 0
    for r in range(n_rounds):
        fetched += int((need[r] & ~cache).sum())
        have = cache | need[r]
        idx = np.nonzero(have)[0]
        if idx.size > slots:
            keep = idx[np.argpartition(nxt[r + 1, idx], slots - 1)[:slots]]
            cache[:] = False
            cache[keep] = True
        else:
            cache = have
    return fetched


def replay_clock(need: np.ndarray, slots: int, seed: int = 0) -> int:
    """The same rounds through a clock cache with reference bits; a round's pages are requested
    in a seeded random order (the real order is a matter of timing)."""
    n_rounds, n_pages = need.shape
    rng = np.random.default_rng(seed)
    slot_of = np.full(n_pages, -1, dtype=np.int64)
    page_in = np.full(slots, -1, dtype=np.int64)
    ref = np.zeros(slots, dtype=bool)
    hand, used, fetched = 0, 0, 0
    for r in range(n_rounds):
        pages = np.nonzero(need[r])[0]
        rng.shuffle(pages)
        for p in pages.tolist():
            s = slot_of[p]
            if s >= 0:
                ref[s] = True
                continue
            fetched += 1
            if used < slots:
                s = used
                used += 1
            else:
                while ref[hand]:
                    ref[hand] = False
                    hand = (hand + 1) % slots
                s = hand
                hand = (hand + 1) % slots
                slot_of[page_in[s]] = -1
            page_in[s] = p
            slot_of[p] = s
            ref[s] = True
    return fetched


def main():
    global _W
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=3, choices=[2, 3, 5])
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--nq", type=int, default=None)
    ap.add_argument("--cache-frac", type=float, default=None)
    ap.add_argument("--procs", type=int, default=os.cpu_count() or 1)
    ap.add_argument("--out", default=os.path.join(ROOT, "profiles", "fetch_floor.json"))
    args = ap.parse_args()
    import oracle
    from workloads import make_config, workload_key
    oracle.build()                      # before the workers fork, so that none of them compiles
    t0 = time.time()
    w = make_config(args.config, scale=args.scale, nq=args.nq, with_gt=False)
    frac = args.cache_frac if args.cache_frac is not None else w.cache_frac
    slots = int(np.floor(frac * w.n_pages))
    _W = w
    print(f"workload built in {time.time() - t0:.0f} s: N={w.N} pages={w.n_pages} nq={w.nq} slots={slots}", flush=True)
    step = max(1, w.nq // (4 * args.procs))
    chunks = [(b, min(w.nq, b + step)) for b in range(0, w.nq, step)]
    t0 = time.time()
    with mp.get_context("fork").Pool(args.procs) as pool:
        per_chunk = pool.map(_query_rounds, chunks)
    per_query = [r for ch in per_chunk for r in ch]
    n_rounds = 1 + max(t for rounds in per_query for t, _ in rounds)
    need = np.zeros((n_rounds, w.n_pages), dtype=bool)
    touches = 0
    for rounds in per_query:
        for t, pages in rounds:
            need[t, pages] = True
            touches += pages.size
    print(f"traces of {w.nq} queries in {time.time() - t0:.0f} s: {n_rounds} rounds, {touches} (query, round, page) touches", flush=True)
    merged = int(need.sum())
    floor = replay_optimal(need, slots)
    clock = replay_clock(need, slots)
    res = {"workload": f"cfg{args.config} scale={args.scale}", "n_nodes": w.N, "n_pages": w.n_pages, "nq": w.nq,
           "K": w.K, "L": w.L, "W": w.W, "cache_slots": slots, "rounds": int(n_rounds),
           "page_touches_per_query_round": int(touches), "distinct_pages_touched": int(need.any(0).sum()),
           "fetches_no_cache_merged_per_round": merged, "fetch_floor_optimal_replacement": int(floor),
           "fetches_clock_replacement": int(clock),
           "model": "all queries in flight in lock step, one iteration per round, same-page requests of a round merged, "
                    "pages of newly scored nodes only",
           "made_by": "python oracle/fetch_floor.py " + " ".join(sys.argv[1:])}
    key = workload_key(args.config, w.N, w.npp, w.nq, w.L, w.W, slots)
    allres = {}
    if os.path.exists(args.out):
        with open(args.out) as fh:
            allres = json.load(fh)
    allres[key] = res
    with open(args.out, "w") as fh:
        json.dump(allres, fh, indent=1, sort_keys=True)
        fh.write("\n")
    print(json.dumps({key: res}, indent=1))


if __name__ == "__main__":
    main()
