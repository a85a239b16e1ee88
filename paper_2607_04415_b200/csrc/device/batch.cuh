// Per-query exact sets and the issue of one batch of page items (lookup, inline hits, misses).
// Part of the persistent search kernel; included by search_kernels.cu in this order.
#pragma once
#include "../gorio_internal.h"

namespace gorio {

// ------------------------------------------------------------------------------------------
// per-query exact sets (open addressing, linear probing, 0xFFFFFFFF = empty)
// ------------------------------------------------------------------------------------------

// returns 1 if v was inserted now, 0 if already present, 2 if the table is full
__device__ u32 set_insert(u32 *tab, u32 cap, u32 v) {
  u32 h = hash32(v) & (cap - 1);
  for (u32 p = 0; p < cap; ++p) {
    u32 old = atomicCAS(tab + h, kInvalidId, v);
    if (old == kInvalidId) return 1;
    if (old == v) return 0;
    h = (h + 1) & (cap - 1);
  }
  return 2;
}
// the same over a bitmap (one bit per possible value): never full
__device__ __forceinline__ u32 bit_insert(u32 *bits, u32 v) {
  const u32 bit = 1u << (v & 31u);
  return (atomicOr(bits + (v >> 5), bit) & bit) ? 0u : 1u;
}

// ------------------------------------------------------------------------------------------
// issue a batch of page items for query slot qs
// ------------------------------------------------------------------------------------------
// Items 0..n_items-1 of the current batch: every lane looks its item's page up; hits are
// consumed now (warp cooperative) and validated against the page word afterwards; misses
// leave the item waiting on the page.  Returns true if the whole batch completed inline
// (the caller goes on with the next phase), false if the query is parked: whoever
// consumes its last item pushes it back onto the runnable queue.
template <bool PQ>
__device__ __noinline__ bool issue_batch(const Ctx &c, u32 qs, u32 lane) {
  QHdr *h = c.hdr + qs;
  // qid, phase, (awaiting), n_items sit in the header's first 16 bytes; only this warp writes
  // them while it runs the query, so every lane may read them for itself
  const uint4 h0 = ld_v4((const u32 *)h);
  const u32 qid = h0.x, phase = h0.y, n = h0.w;
  const u64 worst = c.stash_cap ? ld_u64((const u64 *)&h->worst_lo) : 0ull;
  const bool count_pages = (c.pq_m == 0) == (phase == PH_EVAL);
  if (lane == 0) st_u32(&h->awaiting, n + 1u);      // +1: guard held until everything is issued
  __threadfence();
  __syncwarp();
  const u32 *items = c.items + (u64)qs * c.WR;
  u32 *pset = c.pset + (u64)qs * c.pset_cap;
  LaneStats st = {0, 0, 0, 0, 0, 0};
  u32 n_done = 0, new_pages = 0, n_stash = 0;
  u64 tq = c.prof ? globaltimer() : 0;

  for (u32 base = 0; base < n; base += 32) {
    const u32 j = base + lane;
    bool pending = j < n;
    u32 node = 0, page = kInvalidId;      // page: the cache unit looked up (see unit_of)
    u64 w_first = kAbsentWord;
    if (pending) {
      node = ld_u32(items + j);
      page = unit_of(c, node);
      if (!c.identity) w_first = ld_u64(c.ptab + page);    // in flight while the page set is probed
      if (count_pages) {                  // distinct index pages, whatever the cache's unit
        const u32 ipage = node / c.npp;
        u32 r;
        if (c.pset_bitmap) {             // one bit per index page: no probing, and the table stays in L2
          r = bit_insert(pset, ipage);
        } else {
          r = set_insert(pset, c.pset_cap, ipage);
        }
        if (r == 1) new_pages++;
        else if (r == 2) raise(c, 6, 0x81, qs, ipage);
      }
    }
    if (c.stash_cap && phase == PH_EXPAND && c.pq_m == 0) {
      // expansions whose adjacency list was stashed when the node was scored need no page
      u32 e = 0, have = 0;
      if (pending) {
        e = hash32(node) & (c.stash_cap - 1);
        have = ld_u32(c.stash_tag + (u64)qs * c.stash_cap + e) == node ? 1u : 0u;
      }
      const u32 cand_mask = __ballot_sync(0xffffffffu, have != 0u);
      for (u32 m = cand_mask; m; m &= m - 1) {
        const u32 src = __ffs(m) - 1;
        const u32 sj = __shfl_sync(0xffffffffu, j, src), se = __shfl_sync(0xffffffffu, e, src);
        const u32 *from = c.stash + ((u64)qs * c.stash_cap + se) * (c.R + 1u);
        u32 *dst = c.adj + ((u64)qs * c.W + sj) * c.R;
        for (u32 i = lane; i < c.R; i += 32) st_u32(dst + i, ld_u32(from + 1 + i));
        if (lane == 0) st_u32(c.adjdeg + (u64)qs * c.W + sj, ld_u32(from));
      }
      if (cand_mask) {
        __threadfence();
        if (have && ld_u32(c.stash_tag + (u64)qs * c.stash_cap + e) == node) {   // not overwritten meanwhile
          pending = false; n_done++; n_stash++;
        }
      }
    }
    phase_mark(c, tq, S_I_SETUP, lane);
    for (u32 round = 0; __any_sync(0xffffffffu, pending); ++round) {
      u32 code = LK_NONE, slot = 0, gen = 0;
      if (c.identity) {                   // whole index preloaded: unit u sits in slot u for good
        if (pending) { code = LK_HIT; slot = page; }
      } else if (pending) {
        code = page_lookup(c, page, qs * c.WR + j, round ? ld_u64(c.ptab + page) : w_first, slot, gen, st);
      }
      __syncwarp();
      phase_mark(c, tq, S_I_LOOKUP, lane);
      if (code == LK_WAIT) pending = false;
      const u32 hits = __ballot_sync(0xffffffffu, code == LK_HIT);
      if (hits) consume_group<PQ>(c, hits, qs, j, slot, phase, qid, node, worst, lane);
      if (hits && c.identity) {
        if (code == LK_HIT) { st.hit++; n_done++; pending = false; }
      } else if (hits) {
        __threadfence();
        if (code == LK_HIT) {
          // the bytes just read were the page's if its word still names this slot and fill
          const u64 w2 = ld_u64(c.ptab + page);
          const u64 m2 = ld_u64(c.smeta + slot);          // (for the reference bit; loaded alongside)
          const u32 s2 = pw_state(w2);
          if ((s2 == P_RESIDENT || s2 == P_ARRIVED) && pw_slot(w2) == slot && pw_low(w2) == gen) {
            if (!(m2 & 1ull)) atomicCAS((unsigned long long *)(c.smeta + slot), m2, m2 | 1ull);
            st.hit++; n_done++;
            pending = false;
          } else {
            st.retry++;              // evicted under the read: look the page up again
          }
        }
      }
      phase_mark(c, tq, S_I_CONSUME, lane);
      // (no stop check here: every round resolves its items or retries a bounded number of
      // times, and run_query looks at the stop flag between phases)
      if (round > 1024) { if (lane == 0) raise(c, 8, 0x84, qs, base); break; }
    }
  }

#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    n_done += __shfl_xor_sync(0xffffffffu, n_done, o);
    new_pages += __shfl_xor_sync(0xffffffffu, new_pages, o);
    n_stash += __shfl_xor_sync(0xffffffffu, n_stash, o);
    st.hit += __shfl_xor_sync(0xffffffffu, st.hit, o);
    st.missed += __shfl_xor_sync(0xffffffffu, st.missed, o);
    st.joins += __shfl_xor_sync(0xffffffffu, st.joins, o);
    st.evict += __shfl_xor_sync(0xffffffffu, st.evict, o);
    st.retry += __shfl_xor_sync(0xffffffffu, st.retry, o);
    st.posted += __shfl_xor_sync(0xffffffffu, st.posted, o);
  }
  u32 complete = 0;
  if (lane == 0 && new_pages) atomicAdd(&h->pages_distinct, new_pages);   // only this warp touches it while it holds the guard
  __threadfence();
  __syncwarp();
  if (lane == 0) {
    const u32 old = atomicSub(&h->awaiting, n_done + 1u);       // inline hits and the guard
    if (old == n_done + 1u) complete = 1;
    else if (old < n_done + 1u) raise(c, 8, 0x82, qs, old, n_done);
    stat_add(c, S_HIT, st.hit); stat_add(c, S_MISSED, st.missed); stat_add(c, S_JOINS, st.joins);
    stat_add(c, S_EVICT, st.evict); stat_add(c, S_RETRY, st.retry); stat_add(c, S_POSTED, st.posted);
    stat_add(c, S_STASH, n_stash);
  }
  phase_mark(c, tq, S_I_TAIL, lane);
  return __shfl_sync(0xffffffffu, complete, 0) != 0u;
}

}  // namespace gorio
