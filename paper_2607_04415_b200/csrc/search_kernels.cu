// Device side of the GPU-owned paged beam search (sm_100a).
//
// One persistent kernel runs every query of a batch.  Warps are the execution slots: a
// warp pops a runnable query slot from a queue in HBM, advances it by one or more phases,
// and parks it when it has to wait for pages (paper Section 3.3: blocks "claim work,
// execute graph traversal, and either finish a query or mark it pending on a missing page").
//
// Data flow of one query iteration:
//   PH_EVAL  complete -> merge the scored candidates into the sorted L-entry list, pick the
//                        first W unexpanded entries (the frontier), issue their pages
//   PH_EXPAND complete -> read the frontier's adjacency lists, filter through the exact
//                        visited set, issue the pages of the new neighbours (exact mode) or
//                        score them from resident PQ codes (PQ mode)
// "Issuing" a batch of page items means, per item: look the page up in the cache; on a hit
// consume it now; if the page is in flight register as a waiter; if it is absent claim a
// slot (clock eviction), post a request descriptor to the host-visible ring and register.
// A page that arrives is consumed for every registered waiter by whichever warp picks the
// arrival up, using only the waiter's query vector, so no page stays pinned for a query.
// The last item consumed of a batch pushes the query back onto the runnable queue.
#include "gorio_internal.h"

namespace gorio {

// ------------------------------------------------------------------------------------------
// memory access helpers: query/cache state is shared between SMs, so it is always read and
// written at the L2 (relaxed, gpu scope); host-mapped words use system scope.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ u32 ld_u32(const u32 *p) {
  u32 v; asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory"); return v;
}
__device__ __forceinline__ u64 ld_u64(const u64 *p) {
  u64 v; asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory"); return v;
}
__device__ __forceinline__ void st_u32(u32 *p, u32 v) {
  asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void st_u64(u64 *p, u64 v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint4 ld_v4(const u32 *p) {
  uint4 v;
  asm volatile("ld.relaxed.gpu.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint4 ld_sys_v4(const u32 *p) {
  uint4 v;
  asm volatile("ld.volatile.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_sys_u32(u32 *p, u32 v) {
  asm volatile("st.relaxed.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void st_sys_u64(u64 *p, u64 v) {
  asm volatile("st.relaxed.sys.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ u64 globaltimer() {
  u64 t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t;
}
__device__ __forceinline__ u32 lane_id() { return threadIdx.x & 31u; }

// ------------------------------------------------------------------------------------------
// errors and statistics
// ------------------------------------------------------------------------------------------
__device__ __noinline__ void raise(const Ctx &c, u32 status, u32 a = 0, u32 b = 0, u32 d = 0, u32 e = 0) {
  if (atomicCAS(&c.ctl->status, 0u, status) == 0u) {
    c.ctl->dbg[0] = a; c.ctl->dbg[1] = b; c.ctl->dbg[2] = d; c.ctl->dbg[3] = e;
    c.ctl->dbg[4] = blockIdx.x; c.ctl->dbg[5] = threadIdx.x;
    __threadfence();
  }
  st_u32(&c.ctl->stop, 2u);
}
// warp-uniform variants: every lane gets lane 0's view, and the shuffle is a convergence point
__device__ __forceinline__ bool warp_stopped(const Ctx &c) {
  return __shfl_sync(0xffffffffu, ld_u32(&c.ctl->stop), 0) != 0u;
}
__device__ __forceinline__ u32 uld(const u32 *p) { return __shfl_sync(0xffffffffu, ld_u32(p), 0); }
__device__ __forceinline__ void stat_add(const Ctx &c, u32 idx, u32 v) {
  if (v) atomicAdd((unsigned long long *)&c.ctl->stats[idx], (unsigned long long)v);
}
// Debug profile: charge the time since `t` to stats[idx] and restart the clock.
__device__ __forceinline__ void phase_mark(const Ctx &c, u64 &t, u32 idx, u32 lane) {
  if (!c.prof) return;
  const u64 now = globaltimer();
  if (lane == 0) atomicAdd((unsigned long long *)&c.ctl->stats[idx], now - t);
  t = now;
}


// ------------------------------------------------------------------------------------------
// bounded MPMC queue of u32 (cells = sequence << 32 | value); one lane calls these
// ------------------------------------------------------------------------------------------
// Tickets are taken with fetch-and-add on both ends, never with compare-and-swap loops:
// thousands of warps poll these queues, and a CAS on a shared head lets only one of them
// through per L2 round trip.  A signed item count guards the consumer side: a consumer
// first takes one unit of the count (backing out if there was none), and only then a head
// ticket, so a ticket is always for a cell whose producer has at least reserved it; the wait
// for that cell is bounded by the producer's own push.
constexpr u32 kSpinLimit = 1u << 22;

__device__ void q_push(const Ctx &c, const Queue &q, u32 v, bool fence = true) {
  if (fence) __threadfence();   // everything written for the consumer is visible before the cell
  const u32 pos = atomicAdd(q.tail, 1u);
  u64 *cell = (u64 *)q.buf + (pos & q.mask);
  u32 spins = 0;
  while ((u32)(ld_u64(cell) >> 32) != pos) {      // previous lap's consumer not done yet
    if (++spins > kSpinLimit) { raise(c, 8, 0x51, pos); return; }
  }
  st_u64(cell, ((u64)(pos + 1u) << 32) | v);
  atomicAdd(q.count, 1);
}

__device__ bool q_pop(const Ctx &c, const Queue &q, u32 &out) {
  if ((int)ld_u32((const u32 *)q.count) <= 0) return false;
  if (atomicSub(q.count, 1) <= 0) { atomicAdd(q.count, 1); return false; }
  const u32 h = atomicAdd(q.head, 1u);
  u64 *cell = (u64 *)q.buf + (h & q.mask);
  u32 spins = 0;
  u64 v;
  while ((u32)((v = ld_u64(cell)) >> 32) != h + 1u) {
    if (++spins > kSpinLimit) { raise(c, 8, 0x52, h); return false; }
  }
  st_u64(cell, (u64)(h + q.mask + 1u) << 32);
  __threadfence();
  out = (u32)v;
  return true;
}

// warp-level pop: lane 0 pops, the result is broadcast
__device__ __forceinline__ bool warp_pop(const Ctx &c, const Queue &q, u32 &out, u32 lane) {
  u32 ok = 0, v = 0;
  if (lane == 0) ok = q_pop(c, q, v) ? 1u : 0u;
  ok = __shfl_sync(0xffffffffu, ok, 0);
  out = __shfl_sync(0xffffffffu, v, 0);
  return ok != 0u;
}

// ------------------------------------------------------------------------------------------
// page cache and miss tracker
// ------------------------------------------------------------------------------------------
// One 64-bit word per index page is the single point of truth for that page:
//   [state:3][slot:29][low:32]   low = head of the page's waiter list (WANTED, FILLING)
//                                      or the slot's fill generation (ARRIVED, RESIDENT)
//   ABSENT   nobody wants the page               WANTED  waiters, no slot yet (queued in want_q)
//   FILLING  slot assigned, request posted       ARRIVED data present, waiters being served
//   RESIDENT data present, evictable
// It is a hash of page -> slot with the identity hash (page ids are dense and known at open),
// so a lookup is one load and the first miss on a page is decided by one compare-and-swap:
// concurrent misses on the same page, from any lane of any query, can only join its list.
// One 64-bit word per slot ([page:32][generation:31][ref:1]) serves the clock.
enum PageState : u32 { P_ABSENT = 0, P_WANTED = 1, P_FILLING = 2, P_ARRIVED = 3, P_RESIDENT = 4 };
constexpr u64 kAbsentWord = (u64)kNil;
__device__ __forceinline__ u64 mk_pw(u32 state, u32 slot, u32 low) {
  return ((u64)state << 61) | ((u64)slot << 32) | low;
}
__device__ __forceinline__ u32 pw_state(u64 w) { return (u32)(w >> 61); }
__device__ __forceinline__ u32 pw_slot(u64 w) { return (u32)(w >> 32) & 0x1FFFFFFFu; }
__device__ __forceinline__ u32 pw_low(u64 w) { return (u32)w; }
__device__ __forceinline__ u64 mk_sm(u32 page, u32 gen, u32 ref) { return ((u64)page << 32) | ((u64)(gen & 0x7FFFFFFFu) << 1) | ref; }
__device__ __forceinline__ u32 sm_page(u64 m) { return (u32)(m >> 32); }
__device__ __forceinline__ u32 sm_gen(u64 m) { return (u32)(m >> 1) & 0x7FFFFFFFu; }

// The cache unit that holds `node` (a page, or with selective materialisation the node's own
// record), and where the node's record starts inside the slot that holds that unit.
__device__ __forceinline__ u32 unit_of(const Ctx &c, u32 node) { return c.record_mode ? node : node / c.npp; }
__device__ __forceinline__ u32 rec_off(const Ctx &c, u32 node) {
  const u32 off = (node % c.npp) * c.node_bytes;
  return c.record_mode ? (off & 15u) : off;
}
__device__ __forceinline__ const u8 *rec_ptr(const Ctx &c, u32 slot, u32 node) {
  return c.slot_data + (u64)slot * c.slot_bytes + rec_off(c, node);
}

struct LaneStats { u32 hit, missed, joins, evict, retry, posted; };

// Post a request descriptor: one 64-bit word [page:32][slot:24][lap:8] in host-mapped memory.
// The ring holds at least twice as many entries as there are slots, and every pending
// request owns a distinct FILLING slot, so an entry is never overwritten before the proxy
// has consumed it.  (Section 3.2: reserve a descriptor slot atomically, record page id and
// target cache slot, publish through a ready flag -- here the lap tag inside the word.)
__device__ __forceinline__ void post_request(const Ctx &c, u32 page, u32 slot) {
  const u32 idx = atomicAdd(&c.ctl->ring_head, 1u);
  atomicAdd(&c.cs->in_flight, 1);
  const u32 lap = ((idx >> c.ring_shift) % 255u) + 1u;
  const u64 e = ((u64)page << 32) | ((u64)slot << 8) | lap;
  st_u64(c.ring_dev + (idx & c.ring_mask), e);   // device copy: what copy and arrival tickets refer to
  __threadfence_system();      // page word, slot label and device copy before the host can act
  st_sys_u64(c.ring + (idx & c.ring_mask), e);
}

// Requests posted and not yet arrived are kept near a small multiple of the proxy's window:
// anything more would only queue in the ring while holding a slot that could keep a resident
// page instead (with the whole cache in flight it is a buffer pool, not a cache).
__device__ __forceinline__ bool may_post(const Ctx &c) { return (int)ld_u32((const u32 *)&c.cs->in_flight) < (int)c.max_in_flight; }

// Get a slot for a new page: never-used slots first, then the clock (second chance for
// referenced pages); `hint` (a slot the caller has just made evictable) is taken if a short
// sweep finds nothing.  Returns kNil when every slot examined is in flight; otherwise `prev_gen`
// is the generation of the slot's previous fill.  (The backlog gate, may_post, stays with the
// callers: checking it again here made serve_want put pages it had already popped back at the
// tail of the want queue, the queue stopped being first-in first-out, requests were posted
// with far fewer waiters each, and config 3 fetched 9.3 M pages instead of 3.7 M.)
__device__ u32 alloc_slot(const Ctx &c, u32 hint, LaneStats &st, u32 &prev_gen) {
  prev_gen = 0;
  if (ld_u32(&c.cs->bump) < c.n_slots) {
    u32 b = atomicAdd(&c.cs->bump, 1u);
    if (b < c.n_slots) return b;
  }
  const int sweep = hint != kNil ? 6 : 48;
  for (int step = 0; step <= sweep; ++step) {
    const bool use_hint = step == sweep;
    if (use_hint && hint == kNil) break;
    const u32 s = use_hint ? hint : atomicAdd(&c.cs->hand, 1u) % c.n_slots;
    const u64 m = ld_u64(c.smeta + s);
    const u32 pg = sm_page(m);
    if (pg >= c.n_units) continue;                       // slot handed out but not yet labelled
    const u64 w = ld_u64(c.ptab + pg);
    if (pw_state(w) != P_RESIDENT || pw_slot(w) != s) continue;
    if ((m & 1ull) && !use_hint) {                       // referenced: second chance
      atomicCAS((unsigned long long *)(c.smeta + s), m, m & ~1ull);
      continue;
    }
    if (atomicCAS((unsigned long long *)(c.ptab + pg), w, kAbsentWord) == w) {
      st.evict++;
      prev_gen = sm_gen(m);
      return s;
    }
  }
  return kNil;
}

// The page is WANTED and `slot` is exclusively ours: label the slot, move the page to
// FILLING (keeping whatever waiters have queued up meanwhile) and post the descriptor.
// `expect` is what the caller believes the page word to be (0 = not known).
__device__ void assign_and_post(const Ctx &c, u32 page, u32 slot, u32 prev_gen, u64 expect, LaneStats &st) {
  st_u64(c.smeta + slot, mk_sm(page, prev_gen + 1u, 0));
  // (no fence needed here: a clock sweep that sees the new label with the old page word, or
  // the reverse, finds state != RESIDENT or a slot mismatch and moves on; everyone else
  // learns of the slot through the descriptor, which is fenced in post_request)
  u64 w = expect ? expect : ld_u64(c.ptab + page);
  for (u32 spins = 0;; ++spins) {
    if (pw_state(w) != P_WANTED || spins > kSpinLimit) { raise(c, 8, 0x41, page, (u32)(w >> 32), spins); return; }
    const u64 old = atomicCAS((unsigned long long *)(c.ptab + page), w, mk_pw(P_FILLING, slot, pw_low(w)));
    if (old == w) break;
    w = old;
  }
  post_request(c, page, slot);
  st.posted++;
}

// Serve one page from the want queue if a slot can be had (one lane).
__device__ void serve_want(const Ctx &c, u32 hint, LaneStats &st) {
  u32 page, prev_gen = 0;
  if (!may_post(c)) return;
  if (!q_pop(c, c.want, page)) return;
  const u32 slot = alloc_slot(c, hint, st, prev_gen);
  if (slot == kNil) { q_push(c, c.want, page); return; }
  assign_and_post(c, page, slot, prev_gen, 0, st);
}

// Lookup / miss generation for one item by one lane.  g is the item's waiter record.
// Returns LK_HIT with (slot, generation) to be consumed and validated by the caller, or
// LK_WAIT when the item now waits on the page (as first requester or as a joiner).
enum LookupCode : u32 { LK_NONE = 0, LK_HIT = 1, LK_WAIT = 2 };
// `first` is the page word as the caller last saw it (every decision below is re-checked by a
// compare-and-swap or by the caller's validation, so a stale word only costs a retry).
__device__ u32 page_lookup(const Ctx &c, u32 page, u32 g, u64 first, u32 &slot, u32 &gen, LaneStats &st) {
  u64 *pw = c.ptab + page;
  for (u32 tries = 0; tries < 4096; ++tries) {
    const u64 w = tries ? ld_u64(pw) : first;
    const u32 s = pw_state(w);
    if (s == P_RESIDENT || s == P_ARRIVED) { slot = pw_slot(w); gen = pw_low(w); return LK_HIT; }
    st_u32(c.wrec + g, s == P_ABSENT ? kNil : pw_low(w));
    __threadfence();
    if (s == P_ABSENT) {
      const u64 wanted = mk_pw(P_WANTED, 0, g);
      if (atomicCAS((unsigned long long *)pw, w, wanted) != w) continue;
      st.missed++;
      // First requester: find the page a slot -- but never ahead of pages that already wait for
      // one.  Requests leave in the order in which their pages were first wanted, so each has
      // gathered as many waiters as it can by the time it is posted; letting new pages jump the
      // queue whenever the backlog had room cost 16 % more fetches on config 3.
      const bool room = may_post(c);
      const bool queued = (int)ld_u32((const u32 *)c.want.count) > 0;
      u32 prev_gen = 0;
      const u32 sl = (room && !queued) ? alloc_slot(c, kNil, st, prev_gen) : kNil;
      if (sl != kNil) {
        assign_and_post(c, page, sl, prev_gen, wanted, st);
      } else {
        q_push(c, c.want, page);
        if (room) serve_want(c, kNil, st);      // the oldest waiting page takes the opening
      }
      return LK_WAIT;
    }
    if (atomicCAS((unsigned long long *)pw, w, (w & 0xFFFFFFFF00000000ull) | g) != w) continue;
    st.missed++; st.joins++;
    return LK_WAIT;
  }
  raise(c, 8, 0x42, page, g);
  return LK_WAIT;
}

// ------------------------------------------------------------------------------------------
// distances (warp cooperative)
// ------------------------------------------------------------------------------------------
// Squared L2 between query qid and the vector at `rec` (a node record inside a cache slot).
// uint8: per-lane 4-byte words, |a-b| per byte then a 4-way dot product into u32 (exact).
// fp32 : per-lane strided elements, fused multiply-add, butterfly reduction (fixed order).
__device__ __forceinline__ u32 warp_dist(const Ctx &c, const u8 *rec, u32 qid, u32 lane) {
  const u8 *q = (const u8 *)c.queries + (u64)qid * c.vec_bytes;
  if (c.dtype == 0) {
    const u32 words = c.dim >> 2;
    u32 acc = 0;
    for (u32 w = lane; w < words; w += 32) {
      u32 a = __ldcg((const u32 *)rec + w), b = __ldg((const u32 *)q + w);
      u32 d = __vabsdiffu4(a, b);
      acc = __dp4a(d, d, acc);
    }
    return __reduce_add_sync(0xffffffffu, acc);
  } else {
    float acc = 0.f;
    for (u32 i = lane; i < c.dim; i += 32) {
      float diff = __ldg((const float *)q + i) - __ldcg((const float *)rec + i);
      acc = fmaf(diff, diff, acc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    return __float_as_uint(acc);
  }
}
__device__ __forceinline__ u64 mk_key(u32 dist, u32 id) { return ((u64)dist << 32) | ((u64)id << 1); }
__device__ __forceinline__ u32 key_id(u64 k) { return (u32)(k & 0xFFFFFFFFull) >> 1; }
__device__ __forceinline__ u32 key_dist(u64 k) { return (u32)(k >> 32); }

constexpr u32 kStashBusy = 0xFFFFFFFEu;
__device__ __forceinline__ u32 hash32(u32 v) { v *= 0x9E3779B1u; v ^= v >> 15; return v * 0x85EBCA77u; }

// Consume item j of query slot qs from the page in `slot` (warp cooperative).
//   PH_EVAL   : score the node, write its key into the candidate buffer.
//   PH_EXPAND : copy the node's adjacency list into the query's buffer (PQ mode: also the
//               node's exact distance into the rerank pool's staging entries).
__device__ void consume_item(const Ctx &c, u32 qs, u32 j, u32 slot, u32 lane) {
  const QHdr *h = c.hdr + qs;
  const u32 phase = ld_u32(&h->phase), qid = ld_u32(&h->qid);
  const u32 node = ld_u32(c.items + (u64)qs * c.WR + j);
  const u8 *rec = rec_ptr(c, slot, node);
  if (phase == PH_EVAL) {
    u32 d = warp_dist(c, rec, qid, lane);
    const u64 key = mk_key(d, node);
    if (lane == 0) st_u64(c.cand + (u64)qs * c.WR + j, key);
    // The node's page is in hand now.  If the node can still enter the list (its key beats
    // the list's worst as of the last merge; the worst only improves, so this errs on the
    // safe side), keep its adjacency list in the query's stash: expanding it later then
    // needs no page.  The stash is a direct-mapped table; a busy or overwritten entry only
    // means that the expansion goes through the page cache as usual.
    if (c.stash_cap && key < ld_u64((const u64 *)&h->worst_lo)) {
      const u32 e = hash32(node) & (c.stash_cap - 1);
      u32 *tag = c.stash_tag + (u64)qs * c.stash_cap + e;
      u32 busy = 0;
      if (lane == 0) busy = atomicExch(tag, kStashBusy) == kStashBusy ? 1u : 0u;
      if (!__shfl_sync(0xffffffffu, busy, 0)) {
        const u32 *adj = (const u32 *)(rec + c.vec_bytes);
        u32 *dst = c.stash + ((u64)qs * c.stash_cap + e) * (c.R + 1u);
        for (u32 i = lane; i < c.R + 1u; i += 32) st_u32(dst + i, __ldcg(adj + i));   // degree, then ids
        __syncwarp();
        if (lane == 0) { __threadfence(); st_u32(tag, node); }
      }
    }
  } else {
    const u32 *adj = (const u32 *)(rec + c.vec_bytes);
    u32 deg = __ldcg(adj);
    u32 *dst = c.adj + ((u64)qs * c.W + j) * c.R;
    for (u32 i = lane; i < c.R; i += 32) st_u32(dst + i, __ldcg(adj + 1 + i));
    if (lane == 0) st_u32(c.adjdeg + (u64)qs * c.W + j, deg);
    if (c.pq_m) {
      u32 d = warp_dist(c, rec, qid, lane);
      if (lane == 0) st_u64(c.pool + (u64)qs * (c.K + c.W) + c.K + j, mk_key(d, node));
    }
  }
}

// n items of query slot qs are done; the one that brings `awaiting` to zero resumes it.
__device__ __forceinline__ void complete_items(const Ctx &c, u32 qs, u32 n) {
  __threadfence();
  u32 old = atomicSub(&c.hdr[qs].awaiting, n);
  if (old == n) { if (!c.blocking) q_push(c, c.run, qs, false); stat_add(c, S_RESUMES, 1); }
  else if (old < n) raise(c, 8, 0x61, qs, old, n);
}

// Score the nodes of `eval_mask` (lane i holds node i's query id, node id and cache slot) with
// 128-bit loads: the warp works as four 8-lane groups, each group scores one node per round,
// lane t of a group handling the 16-byte chunks t, t+8, t+16 of the vector.  Records are only
// 4-byte aligned inside a page (388- or 644-byte nodes), so a chunk is assembled from the two
// 16-byte-aligned pieces that cover it by word selection; query rows are 16-byte aligned.
// ROUNDS nodes per group are loaded before any is reduced.  Returns the distance (u32 bits) to
// the lanes of eval_mask.
__device__ __forceinline__ u32 pick_word(const uint4 &a, const uint4 &b, u32 i) {
  // word i (0..6) of the 8-word sequence a.x a.y a.z a.w b.x b.y b.z b.w
  const u32 lo = (i & 2u) ? ((i & 1u) ? a.w : a.z) : ((i & 1u) ? a.y : a.x);
  const u32 hi = (i & 2u) ? ((i & 1u) ? b.w : b.z) : ((i & 1u) ? b.y : b.x);
  return (i & 4u) ? hi : lo;
}

template <int CH, int ROUNDS>
__device__ __forceinline__ u32 score_group128(const Ctx &c, u32 eval_mask, u32 qid, u32 node, u32 slot, u32 lane) {
  const u32 grp = lane >> 3, t = lane & 7u;
  const u32 nchunk = c.vec_bytes >> 4;
  u32 dist = 0;
  for (u32 m = eval_mask; m;) {
    uint4 A[ROUNDS][CH], B[ROUNDS][CH], Q[ROUNDS][CH];
    u32 src[ROUNDS], sw[ROUNDS];
    bool valid[ROUNDS];
#pragma unroll
    for (int r = 0; r < ROUNDS; ++r) {
      const u32 sel = __fns(m, 0, (int)(r * 4 + grp) + 1);      // this group's node of this round
      valid[r] = sel < 32u;
      src[r] = valid[r] ? sel : 0u;
      const u32 s_qid = __shfl_sync(0xffffffffu, qid, src[r]), s_node = __shfl_sync(0xffffffffu, node, src[r]);
      const u32 s_slot = __shfl_sync(0xffffffffu, slot, src[r]);
      const u32 off = rec_off(c, s_node);
      sw[r] = (off & 15u) >> 2;
      const u8 *base = c.slot_data + (u64)s_slot * c.slot_bytes + (off & ~15u);
      const u8 *q = (const u8 *)c.queries + (u64)s_qid * c.vec_bytes;
#pragma unroll
      for (int k = 0; k < CH; ++k) {
        const u32 ch = t + 8u * (u32)k;
        const bool in = valid[r] && ch < nchunk;
        A[r][k] = in ? __ldcg((const uint4 *)(base + 16u * ch)) : make_uint4(0, 0, 0, 0);
        B[r][k] = (in && sw[r]) ? __ldcg((const uint4 *)(base + 16u * ch + 16u)) : make_uint4(0, 0, 0, 0);
        Q[r][k] = in ? __ldg((const uint4 *)(q + 16u * ch)) : make_uint4(0, 0, 0, 0);
      }
    }
#pragma unroll
    for (int r = 0; r < ROUNDS; ++r) {
      u32 d;
      if (c.dtype == 0) {
        u32 acc = 0;
#pragma unroll
        for (int k = 0; k < CH; ++k) {
          const u32 qq[4] = {Q[r][k].x, Q[r][k].y, Q[r][k].z, Q[r][k].w};
#pragma unroll
          for (int i = 0; i < 4; ++i) { const u32 x = __vabsdiffu4(pick_word(A[r][k], B[r][k], sw[r] + i), qq[i]); acc = __dp4a(x, x, acc); }
        }
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        d = acc;
      } else {
        float acc = 0.f;
#pragma unroll
        for (int k = 0; k < CH; ++k) {
          const u32 qq[4] = {Q[r][k].x, Q[r][k].y, Q[r][k].z, Q[r][k].w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float x = __uint_as_float(qq[i]) - __uint_as_float(pick_word(A[r][k], B[r][k], sw[r] + i));
            acc = fmaf(x, x, acc);
          }
        }
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        d = __float_as_uint(acc);
      }
      // hand each group's result to the lane that owns the node
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const u32 dg = __shfl_sync(0xffffffffu, d, g * 8);
        const u32 owner = __shfl_sync(0xffffffffu, valid[r] ? src[r] : 0xFFu, g * 8);
        if (lane == owner) dist = dg;
      }
    }
#pragma unroll
    for (int i = 0; i < 4 * ROUNDS; ++i) m &= m - 1;      // the nodes just scored
  }
  return dist;
}

// Consume up to 32 items at once: lane i holds item i = (query slot, item index, cache slot) if
// bit i of `mask` is set.  The items' metadata is fetched lane-parallel, and the vectors of
// scoring items are loaded four items at a time before any of them is reduced, so that the
// L2 round trips of different items overlap instead of adding up (the per-item version is
// latency bound).  Adjacency copies (expansion items) and vectors longer than 96 words take
// the one-at-a-time path.
//
// Lane i also holds its item's metadata: the query's phase and id, the node, and (exact
// navigation with a stash) the list's worst key as of the last merge.
template <bool PQ>
__device__ __noinline__ void consume_group(const Ctx &c, u32 mask, u32 qs, u32 j, u32 slot, u32 phase, u32 qid,
                                           u32 node, u64 worst, u32 lane) {
  const bool mine = (mask >> lane) & 1u;
  if (!mine) { phase = 0; qid = 0; node = 0; worst = 0; }
  const u32 words = c.vec_bytes >> 2;
  const u32 eval_mask = words <= 96u ? __ballot_sync(0xffffffffu, mine && phase == PH_EVAL) : 0u;
  u32 dist = 0;
  if (c.vec128 && eval_mask) {
    if (c.vec_bytes <= 128u) dist = score_group128<1, 2>(c, eval_mask, qid, node, slot, lane);
    else dist = score_group128<3, 1>(c, eval_mask, qid, node, slot, lane);
  }
  for (u32 m = c.vec128 ? 0u : eval_mask; m;) {
    u32 src[4], a[4][3], b[4][3];
    int ng = 0;
#pragma unroll
    for (int g = 0; g < 4; ++g) { src[g] = 0; if (m) { src[g] = __ffs(m) - 1; m &= m - 1; ng = g + 1; } }
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      if (g < ng) {
        const u32 s_qid = __shfl_sync(0xffffffffu, qid, src[g]), s_node = __shfl_sync(0xffffffffu, node, src[g]);
        const u32 s_slot = __shfl_sync(0xffffffffu, slot, src[g]);
        const u32 *rec = (const u32 *)rec_ptr(c, s_slot, s_node);
        const u32 *q = (const u32 *)((const u8 *)c.queries + (u64)s_qid * c.vec_bytes);
#pragma unroll
        for (int w = 0; w < 3; ++w) {
          const u32 idx = (u32)w * 32u + lane;
          const bool in = idx < words;
          a[g][w] = in ? __ldcg(rec + idx) : 0u;
          b[g][w] = in ? __ldg(q + idx) : 0u;
        }
      }
    }
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      if (g < ng) {
        u32 d;
        if (c.dtype == 0) {
          u32 acc = 0;
#pragma unroll
          for (int w = 0; w < 3; ++w) { const u32 x = __vabsdiffu4(a[g][w], b[g][w]); acc = __dp4a(x, x, acc); }
          d = __reduce_add_sync(0xffffffffu, acc);
        } else {
          float acc = 0.f;
#pragma unroll
          for (int w = 0; w < 3; ++w) { const float x = __uint_as_float(b[g][w]) - __uint_as_float(a[g][w]); acc = fmaf(x, x, acc); }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
          d = __float_as_uint(acc);
        }
        if (lane == src[g]) dist = d;
      }
    }
  }
  const bool scored = (eval_mask >> lane) & 1u;
  const u64 key = mk_key(dist, node);
  if (scored) st_u64(c.cand + (u64)qs * c.WR + j, key);
  // Adjacency stash for candidates that can still enter the list (see consume_item).  Every
  // owner lane claims its own entry (all claims in flight together), the warp copies the
  // claimed lists two at a time with their loads in flight, and the tags are published last.
  {
    u32 e = 0;
    bool own = false;
    if (scored && c.stash_cap && key < worst) {
      e = hash32(node) & (c.stash_cap - 1);
      own = atomicExch(c.stash_tag + (u64)qs * c.stash_cap + e, kStashBusy) != kStashBusy;
    }
    const u32 owners = __ballot_sync(0xffffffffu, own);
    const bool narrow = c.R + 1u <= 96u;
    for (u32 m = owners; m;) {
      u32 src[2], a[2][3];
      int ng = 0;
#pragma unroll
      for (int g = 0; g < 2; ++g) { src[g] = 0; if (m && (g == 0 || narrow)) { src[g] = __ffs(m) - 1; m &= m - 1; ng = g + 1; } }
#pragma unroll
      for (int g = 0; g < 2; ++g) {
        if (g < ng) {
          const u32 s_node = __shfl_sync(0xffffffffu, node, src[g]), s_slot = __shfl_sync(0xffffffffu, slot, src[g]);
          const u32 *adj = (const u32 *)(rec_ptr(c, s_slot, s_node) + c.vec_bytes);
          if (narrow) {
#pragma unroll
            for (int k = 0; k < 3; ++k) { const u32 i = (u32)k * 32u + lane; a[g][k] = i <= c.R ? __ldcg(adj + i) : 0u; }
          }
        }
      }
#pragma unroll
      for (int g = 0; g < 2; ++g) {
        if (g < ng) {
          const u32 s_qs = __shfl_sync(0xffffffffu, qs, src[g]), s_e = __shfl_sync(0xffffffffu, e, src[g]);
          u32 *dst = c.stash + ((u64)s_qs * c.stash_cap + s_e) * (c.R + 1u);
          if (narrow) {
#pragma unroll
            for (int k = 0; k < 3; ++k) { const u32 i = (u32)k * 32u + lane; if (i <= c.R) st_u32(dst + i, a[g][k]); }
          } else {
            const u32 s_node = __shfl_sync(0xffffffffu, node, src[g]), s_slot = __shfl_sync(0xffffffffu, slot, src[g]);
            const u32 *adj = (const u32 *)(rec_ptr(c, s_slot, s_node) + c.vec_bytes);
            for (u32 i = lane; i < c.R + 1u; i += 32) st_u32(dst + i, __ldcg(adj + i));
          }
        }
      }
    }
    if (owners) {
      __syncwarp();
      if (own) { __threadfence(); st_u32(c.stash_tag + (u64)qs * c.stash_cap + e, node); }
    }
  }
  // Expansion items: copy the node's adjacency list into the query's buffer (PQ navigation: also
  // its exact distance into the rerank pool's staging entries), two items' loads in flight.
  const u32 rest = mask & ~eval_mask;
  const bool paired = words <= 96u && c.R + 1u <= 96u;
  for (u32 m = paired ? rest : 0u; m;) {
    u32 src[2], a[2][3], v[2][3], qw[2][3];
    int ng = 0;
#pragma unroll
    for (int g = 0; g < 2; ++g) { src[g] = 0; if (m) { src[g] = __ffs(m) - 1; m &= m - 1; ng = g + 1; } }
#pragma unroll
    for (int g = 0; g < 2; ++g) {
      if (g < ng) {
        const u32 s_node = __shfl_sync(0xffffffffu, node, src[g]), s_slot = __shfl_sync(0xffffffffu, slot, src[g]);
        const u32 s_qid = __shfl_sync(0xffffffffu, qid, src[g]);
        const u32 *rec = (const u32 *)rec_ptr(c, s_slot, s_node);
        const u32 *adj = rec + words;                       // degree, then R ids
        const u32 *q = (const u32 *)((const u8 *)c.queries + (u64)s_qid * c.vec_bytes);
#pragma unroll
        for (int k = 0; k < 3; ++k) {
          const u32 idx = (u32)k * 32u + lane;
          a[g][k] = idx <= c.R ? __ldcg(adj + idx) : 0u;
          const bool in = PQ && idx < words;
          v[g][k] = in ? __ldcg(rec + idx) : 0u;
          qw[g][k] = in ? __ldg(q + idx) : 0u;
        }
      }
    }
#pragma unroll
    for (int g = 0; g < 2; ++g) {
      if (g < ng) {
        const u32 s_qs = __shfl_sync(0xffffffffu, qs, src[g]), s_j = __shfl_sync(0xffffffffu, j, src[g]);
        const u32 s_node = __shfl_sync(0xffffffffu, node, src[g]);
        u32 *dst = c.adj + ((u64)s_qs * c.W + s_j) * c.R;
#pragma unroll
        for (int k = 0; k < 3; ++k) {
          const u32 idx = (u32)k * 32u + lane;
          if (idx >= 1u && idx <= c.R) st_u32(dst + idx - 1u, a[g][k]);
        }
        if (lane == 0) st_u32(c.adjdeg + (u64)s_qs * c.W + s_j, a[g][0]);
        if (PQ) {
          u32 d;
          if (c.dtype == 0) {
            u32 acc = 0;
#pragma unroll
            for (int k = 0; k < 3; ++k) { const u32 x = __vabsdiffu4(v[g][k], qw[g][k]); acc = __dp4a(x, x, acc); }
            d = __reduce_add_sync(0xffffffffu, acc);
          } else {                                          // same order as warp_dist
            float acc = 0.f;
#pragma unroll
            for (int k = 0; k < 3; ++k) { const float x = __uint_as_float(qw[g][k]) - __uint_as_float(v[g][k]); acc = fmaf(x, x, acc); }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            d = __float_as_uint(acc);
          }
          if (lane == 0) st_u64(c.pool + (u64)s_qs * (c.K + c.W) + c.K + s_j, mk_key(d, s_node));
        }
      }
    }
  }
  // everything else one at a time
  for (u32 m = paired ? 0u : rest; m; m &= m - 1) {
    const u32 src = __ffs(m) - 1;
    consume_item(c, __shfl_sync(0xffffffffu, qs, src), __shfl_sync(0xffffffffu, j, src),
                 __shfl_sync(0xffffffffu, slot, src), lane);
  }
  __syncwarp();
}

// Waiter lists can be long (every query waits on the entry page at the start), so a warp
// consumes at most kChainSegment records and hands the rest of the chain to another warp
// through the arrival queue; `parts` counts the segments still being served for the slot.
constexpr u32 kChainSegment = 32;
constexpr u32 kContFlag = 0x80000000u;

__device__ void finish_arrival(const Ctx &c, u32 slot, u32 page, u32 gen, u32 lane) {
  // last segment done: the page becomes evictable, and the slot's turn-over feeds the
  // pages that are waiting for a slot
  if (lane == 0) {
    __threadfence();
    st_u64(c.ptab + page, mk_pw(P_RESIDENT, slot, gen));
    LaneStats st = {0, 0, 0, 0, 0, 0};
    serve_want(c, slot, st);
    stat_add(c, S_EVICT, st.evict); stat_add(c, S_POSTED, st.posted);
  }
  __syncwarp();
}

// Consume the waiter chain starting at record g for the page held in `slot`.
template <bool PQ>
__device__ void consume_chain(const Ctx &c, u32 slot, u32 page, u32 gen, u32 g, u32 lane, u64 tp = 0) {
  const u32 limit = c.n_qslots * c.WR;
  if (c.prof && tp == 0) tp = globaltimer();
  phase_mark(c, tp, S_A_HEAD, lane);
  // chase up to a segment of next pointers first so that the remainder is handed off early
  u32 mine = kNil, n = 0, cur = g;
  while (cur != kNil && n < kChainSegment) {
    if (cur >= limit) { if (lane == 0) raise(c, 8, 0x73, slot, cur, n); return; }
    if (lane == n) mine = cur;
    cur = uld(c.wrec + cur);
    ++n;
  }
  if (cur != kNil && lane == 0) {
    atomicAdd(c.parts + slot, 1u);
    q_push(c, c.arr, kContFlag | cur);
  }
  phase_mark(c, tp, S_A_WALK, lane);
  {
    const bool have = lane < n;
    const u32 qs = have ? mine / c.WR : 0u, j = have ? mine % c.WR : 0u;
    u32 phase = 0, qid = 0, node = 0;
    u64 worst = 0;
    if (have) {
      const QHdr *h = c.hdr + qs;
      phase = ld_u32(&h->phase); qid = ld_u32(&h->qid);
      node = ld_u32(c.items + mine);
      if (c.stash_cap) worst = ld_u64((const u64 *)&h->worst_lo);
    }
    consume_group<PQ>(c, n >= 32 ? 0xffffffffu : ((1u << n) - 1u), qs, j, slot, phase, qid, node, worst, lane);
    phase_mark(c, tp, S_A_GROUP, lane);
    // consume_group ends with a warp barrier: every lane's result stores happen before the
    // owner lane's fence + decrement below
    if (have) complete_items(c, qs, 1);
    __syncwarp();
    phase_mark(c, tp, S_A_COMPLETE, lane);
  }
  u32 last = 0;
  if (lane == 0) last = atomicSub(c.parts + slot, 1u) == 1u ? 1u : 0u;
  if (__shfl_sync(0xffffffffu, last, 0)) finish_arrival(c, slot, page, gen, lane);
  phase_mark(c, tp, S_A_FINISH, lane);
}

// A page has arrived in `slot` (Section 3.2: the per-slot ready entry): take its waiter
// list, serve it, then make the page evictable.  v is a slot id, or a continuation
// (kContFlag | record) of a chain another warp handed off.
template <bool PQ>
__device__ void consume_arrival(const Ctx &c, u32 v, u32 lane) {
  if (v & kContFlag) {
    const u32 g = v & ~kContFlag;
    if (g >= c.n_qslots * c.WR) { if (lane == 0) raise(c, 8, 0x74, g); return; }
    const u32 node = uld(c.items + g);
    const u32 page = unit_of(c, node);
    u64 w = ld_u64(c.ptab + page);
    w = __shfl_sync(0xffffffffu, w, 0);
    if (pw_state(w) != P_ARRIVED) { if (lane == 0) raise(c, 8, 0x75, g, page, (u32)(w >> 32)); return; }
    consume_chain<PQ>(c, pw_slot(w), page, pw_low(w), g, lane);
    return;
  }
  const u32 slot = v;
  if (slot >= c.n_slots) { if (lane == 0) raise(c, 8, 0x71, slot); return; }
  const u64 tp = c.prof ? globaltimer() : 0;
  u64 m = ld_u64(c.smeta + slot);
  m = __shfl_sync(0xffffffffu, m, 0);
  const u32 page = sm_page(m), gen = sm_gen(m);
  if (page >= c.n_units) { if (lane == 0) raise(c, 8, 0x76, slot, page); return; }
  u32 head = 0, bad = 0;
  if (lane == 0) {
    // acquire the copier's stores into the slot (normally long done: the completion was
    // published at least the remote latency after the bytes arrived)
    u32 spins = 0;
    while (ld_u32(c.filled + slot) != gen) {
      __nanosleep(100);
      if (++spins > (1u << 20)) { raise(c, 5, 0x77, slot, gen); bad = 1; break; }
    }
    __threadfence();
  }
  if (__shfl_sync(0xffffffffu, bad, 0)) return;
  if (lane == 0) {
    st_u32(c.parts + slot, 1u);
    atomicSub(&c.cs->in_flight, 1);
    st_u64(c.smeta + slot, m | 1ull);                      // a fresh page gets its second chance
    const u64 old = atomicExch((unsigned long long *)(c.ptab + page), mk_pw(P_ARRIVED, slot, gen));
    if (pw_state(old) != P_FILLING || pw_slot(old) != slot) { raise(c, 8, 0x72, slot, page, (u32)(old >> 32)); bad = 1; }
    head = pw_low(old);
    __threadfence();
  }
  if (__shfl_sync(0xffffffffu, bad, 0)) return;
  head = __shfl_sync(0xffffffffu, head, 0);
  consume_chain<PQ>(c, slot, page, gen, head, lane, tp);
}

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
      w_first = ld_u64(c.ptab + page);    // in flight while the page set is probed
      if (count_pages) {                  // distinct index pages, whatever the cache's unit
        const u32 ipage = node / c.npp;
        u32 r = set_insert(pset, c.pset_cap, ipage);
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
      if (pending) code = page_lookup(c, page, qs * c.WR + j, round ? ld_u64(c.ptab + page) : w_first, slot, gen, st);
      __syncwarp();
      phase_mark(c, tq, S_I_LOOKUP, lane);
      if (code == LK_WAIT) pending = false;
      const u32 hits = __ballot_sync(0xffffffffu, code == LK_HIT);
      if (hits) consume_group<PQ>(c, hits, qs, j, slot, phase, qid, node, worst, lane);
      if (hits) {
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
      if (round > 1024) { if (lane == 0) raise(c, 8, 0x84, qs, base); break; }
      if (warp_stopped(c)) break;
    }
    if (warp_stopped(c)) break;
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

// ------------------------------------------------------------------------------------------
// warp-sorted candidate list
// ------------------------------------------------------------------------------------------
// Bitonic sort of 32*NPL u64 keys held NPL per lane, element e at lane e%32, register e/32.
// k_first = 2 sorts; k_first = 32*NPL runs only the last pass, which merges an array whose
// lower half ascends and whose upper half descends.  desc sorts into descending order.
template <int NPL>
__device__ __forceinline__ void bitonic_sort(u64 (&x)[NPL], u32 lane, u32 k_first = 2, bool desc = false) {
  // Stages whose stride is below 32 exchange between lanes and do the same thing to every
  // register, so they run as a runtime loop over one stage body; stages with a stride of 32 or
  // more pair registers and need static indices.  (Fully unrolled, the 512-key network is
  // several thousand instructions, and warps in different phases evict each other's code.)
#pragma unroll 1
  for (u32 k = k_first; k <= 32u * NPL; k <<= 1) {
#pragma unroll
    for (int kk = 64; kk <= 32 * NPL; kk <<= 1) {
      if (k == (u32)kk) {
#pragma unroll
        for (int jr = kk >> 6; jr > 0; jr >>= 1) {
#pragma unroll
          for (int r = 0; r < NPL; ++r) {
            const int pr = r ^ jr;
            if (pr > r) {
              const bool asc = (((r << 5) & kk) == 0) != desc;
              const u64 a = x[r], b = x[pr];
              const bool sw = asc ? (a > b) : (a < b);
              x[r] = sw ? b : a;
              x[pr] = sw ? a : b;
            }
          }
        }
      }
    }
#pragma unroll 1
    for (u32 j = (k >> 1) < 16u ? (k >> 1) : 16u; j > 0; j >>= 1) {
      const bool lower = (lane & j) == 0;
#pragma unroll
      for (int r = 0; r < NPL; ++r) {
        const u64 a = x[r];
        const u64 b = __shfl_xor_sync(0xffffffffu, a, j);
        const bool asc = (((((u32)r << 5) | lane) & k) == 0) != desc;
        const u64 mn = a < b ? a : b, mx = a < b ? b : a;
        x[r] = (asc == lower) ? mn : mx;
      }
    }
  }
}

__device__ __forceinline__ void write_result(const Ctx &c, u32 qid, u32 k, u64 key, bool valid) {
  const u64 o = (u64)qid * c.K + k;
  c.out_ids[o] = valid ? key_id(key) : kInvalidId;
  u32 d = valid ? key_dist(key) : (c.dtype == 0 ? kInvalidId : 0x7F800000u);
  ((u32 *)c.out_dists)[o] = d;
}

// Merge the scored candidates of the finished PH_EVAL batch into the list (top-L by key),
// then choose and mark the frontier: the first W unexpanded entries in key order.  The
// frontier's node ids become the items of the next (PH_EXPAND) batch.  Returns |frontier|;
// 0 means the search of this query is over (exact mode: the results are written here).
template <int NPL>
__device__ __noinline__ u32 merge_select(const Ctx &c, u32 qs, u32 lane) {
  QHdr *h = c.hdr + qs;
  u32 len = uld(&h->list_len);
  const u32 nc = uld(&h->n_items);
  u64 *list = c.list + (u64)qs * c.L;
  const u64 *cand = c.cand + (u64)qs * c.WR;
  // The list (sorted, at most L <= 16*NPL keys) lives in the lower half of the registers.  A
  // chunk of up to 16*NPL new candidates is sorted on its own, descending, in the upper half,
  // which makes the whole array bitonic; one merge pass then orders it, and everything beyond
  // L is dropped.  (Sorting list and candidates together cost 2-4x the compare-exchanges.)
  constexpr int H = NPL / 2;
  constexpr u32 HALF = 16u * NPL;
  u64 x[NPL];
#pragma unroll
  for (int r = 0; r < NPL; ++r) {
    const u32 e = (u32)r * 32u + lane;
    x[r] = e < len ? ld_u64(list + e) : kPadKey;
  }
  u32 done = 0;
  while (done < nc) {
    const u32 take = min(HALF, nc - done);
    u64 y[H];
#pragma unroll
    for (int r = 0; r < H; ++r) {
      const u32 e = (u32)r * 32u + lane;
      y[r] = e < take ? ld_u64(cand + done + e) : kPadKey;
    }
    bitonic_sort<H>(y, lane, 2, true);
#pragma unroll
    for (int r = 0; r < H; ++r) x[H + r] = y[r];
    bitonic_sort<NPL>(x, lane, 32u * NPL);
    len = min(c.L, len + take);
    done += take;
#pragma unroll
    for (int r = 0; r < NPL; ++r) {
      const u32 e = (u32)r * 32u + lane;
      if (e >= len) x[r] = kPadKey;
    }
  }
  // frontier
  u32 taken = 0;
  u32 *items = c.items + (u64)qs * c.WR;
#pragma unroll
  for (int r = 0; r < NPL; ++r) {
    const u32 e = (u32)r * 32u + lane;
    const bool un = e < len && !(x[r] & 1ull);
    const u32 b = __ballot_sync(0xffffffffu, un);
    if (taken < c.W && b) {
      const u32 rank = taken + __popc(b & ((1u << lane) - 1u));
      if (un && rank < c.W) { x[r] |= 1ull; st_u32(items + rank, key_id(x[r])); }
      taken = min(c.W, taken + (u32)__popc(b));
    }
  }
#pragma unroll
  for (int r = 0; r < NPL; ++r) {
    const u32 e = (u32)r * 32u + lane;
    if (e < len) st_u64(list + e, x[r]);
  }
  if (lane == 0) st_u32(&h->list_len, len);
  {   // the L-th key once the list is full: what a new candidate has to beat
    const u32 wi = c.L - 1u;
    u64 worst = kPadKey;
#pragma unroll
    for (int r = 0; r < NPL; ++r)
      if ((u32)r == wi / 32u) worst = __shfl_sync(0xffffffffu, x[r], wi % 32u);
    if (lane == 0) st_u64((u64 *)&h->worst_lo, len == c.L ? (worst | 1ull) : kPadKey);
  }
  if (taken == 0 && c.pq_m == 0) {
    const u32 qid = uld(&h->qid);
#pragma unroll
    for (int r = 0; r < NPL; ++r) {
      const u32 e = (u32)r * 32u + lane;
      if (e < c.K) write_result(c, qid, e, x[r], e < len);
    }
  }
  return taken;
}

__device__ u32 merge_select_dispatch(const Ctx &c, u32 qs, u32 lane) {
  if (c.L <= 32) return merge_select<2>(c, qs, lane);        // the list fits half of 32*NPL keys
  if (c.L <= 64) return merge_select<4>(c, qs, lane);
  if (c.L <= 128) return merge_select<8>(c, qs, lane);
  return merge_select<16>(c, qs, lane);
}

// PQ mode: fold the exact distances of the nodes just expanded into the rerank pool
// (sorted, the best K kept).  Entries K..K+nf-1 of the pool array are the staging area.
template <int NPL>
__device__ __noinline__ void pool_merge(const Ctx &c, u32 qs, u32 nf, bool final_out, u32 lane) {
  QHdr *h = c.hdr + qs;
  u64 *pool = c.pool + (u64)qs * (c.K + c.W);
  u32 len = uld(&h->pool_len);
  u64 x[NPL];
#pragma unroll
  for (int r = 0; r < NPL; ++r) {
    const u32 e = (u32)r * 32u + lane;
    x[r] = e < len ? ld_u64(pool + e) : (e - len < nf ? ld_u64(pool + c.K + (e - len)) : kPadKey);
  }
  if (nf) bitonic_sort<NPL>(x, lane);
  len = min(c.K, len + nf);
#pragma unroll
  for (int r = 0; r < NPL; ++r) {
    const u32 e = (u32)r * 32u + lane;
    if (e < len) st_u64(pool + e, x[r]);
  }
  if (lane == 0) st_u32(&h->pool_len, len);
  if (final_out) {
    const u32 qid = uld(&h->qid);
#pragma unroll
    for (int r = 0; r < NPL; ++r) {
      const u32 e = (u32)r * 32u + lane;
      if (e < c.K) write_result(c, qid, e, x[r], e < len);
    }
  }
}
__device__ void pool_merge_dispatch(const Ctx &c, u32 qs, u32 nf, bool final_out, u32 lane) {
  const u32 need = c.K + c.W;
  if (need <= 32) pool_merge<1>(c, qs, nf, final_out, lane);
  else if (need <= 64) pool_merge<2>(c, qs, nf, final_out, lane);
  else if (need <= 128) pool_merge<4>(c, qs, nf, final_out, lane);
  else if (need <= 256) pool_merge<8>(c, qs, nf, final_out, lane);
  else pool_merge<16>(c, qs, nf, final_out, lane);
}

// Read the adjacency lists delivered by the finished PH_EXPAND batch, drop every neighbour
// already in the exact visited set, and store the survivors as the next batch's items.
__device__ u32 collect_neighbors(const Ctx &c, u32 qs, u32 lane) {
  QHdr *h = c.hdr + qs;
  const u32 nf = uld(&h->n_items);
  const u32 *adj = c.adj + (u64)qs * c.W * c.R;
  const u32 *adjdeg = c.adjdeg + (u64)qs * c.W;
  u32 *items = c.items + (u64)qs * c.WR;
  u32 *seen = c.seen + (u64)qs * c.seen_cap;
  u32 sum_deg = 0;
  for (u32 f = 0; f < nf; ++f) {
    u32 d = ld_u32(adjdeg + f);
    if (d > c.R) { if (lane == 0) raise(c, 7, 0x91, qs, f, d); return 0; }
    sum_deg += d;
  }
  u32 out = 0;
  const u32 total = nf * c.R;
  for (u32 base = 0; base < total; base += 32) {
    const u32 p = base + lane;
    bool isnew = false;
    u32 v = 0;
    if (p < total) {
      const u32 f = p / c.R, i = p % c.R;
      if (i < ld_u32(adjdeg + f)) {
        v = ld_u32(adj + p);
        if (v >= c.n_nodes) raise(c, 7, 0x92, qs, v);
        else {
          u32 r = set_insert(seen, c.seen_cap, v);
          if (r == 2) raise(c, 6, 0x93, qs, v);
          isnew = r == 1;
        }
      }
    }
    const u32 b = __ballot_sync(0xffffffffu, isnew);
    if (isnew) st_u32(items + out + __popc(b & ((1u << lane) - 1u)), v);
    out += __popc(b);
  }
  __syncwarp();
  if (lane == 0) {
    st_u32(&h->sum_deg, ld_u32(&h->sum_deg) + sum_deg);
    st_u32(&h->n_eval, ld_u32(&h->n_eval) + out);
  }
  return out;
}

// ------------------------------------------------------------------------------------------
// PQ asymmetric distance: per-query lookup table in shared memory
// ------------------------------------------------------------------------------------------
// LUT[m][c] = sum_j (q[m*dsub+j] - cent[m][c][j])^2 (exact, < 2^20 for dsub <= 16);
// adc(v) = sum_m LUT[m][code[v][m]].
// The table is stored losslessly in 20 bits per entry -- a u16 array of low halves followed by
// the high nibbles packed eight to a word -- 640 bytes per subspace instead of 1024, so that
// ten warps per SM can each keep a table instead of six.
__device__ __forceinline__ const u32 *lut_hi(const Ctx &c, const u32 *lut) { return lut + c.pq_m * (kPqKsub / 2); }
__device__ __forceinline__ u32 lut_get(const u16 *lo, const u32 *hi, u32 e) {
  return (u32)lo[e] | (((hi[e >> 3] >> ((e & 7u) * 4u)) & 15u) << 16);
}

// Building the table reads the whole codebook (pq_m x 256 centroids, L2 resident).  A query that
// is resumed on another warp rebuilds it, so the loads are issued in batches before any result
// is needed: one load at a time costs an L2 round trip per entry (86 us per table measured).
//
// dsub == 4 (one word per centroid) with a 16-byte-aligned codebook: a lane takes four
// consecutive entries per 16-byte load, eight loads in flight.
__device__ void build_lut_w1(const Ctx &c, const u8 *q, u32 *lut, u32 lane) {
  const u32 quads = c.pq_m * (kPqKsub / 4);
  const uint4 *cent = (const uint4 *)c.pq_cent;
  uint2 *lo2 = (uint2 *)lut;
  u32 *hi = lut + c.pq_m * (kPqKsub / 2);
  for (u32 g0 = lane; g0 < quads; g0 += 32u * 8u) {
    uint4 cw[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const u32 g = g0 + 32u * (u32)k;
      cw[k] = g < quads ? __ldg(cent + g) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const u32 g = g0 + 32u * (u32)k;
      const bool in = g < quads;                         // the same for a lane and its partner: quads is even
      const u32 qw = in ? __ldg((const u32 *)q + (g >> 6)) : 0u;     // 64 groups of four per subspace
      u32 d, s0, s1, s2, s3;
      d = __vabsdiffu4(cw[k].x, qw); s0 = __dp4a(d, d, 0u);
      d = __vabsdiffu4(cw[k].y, qw); s1 = __dp4a(d, d, 0u);
      d = __vabsdiffu4(cw[k].z, qw); s2 = __dp4a(d, d, 0u);
      d = __vabsdiffu4(cw[k].w, qw); s3 = __dp4a(d, d, 0u);
      if (in) lo2[g] = make_uint2((s0 & 0xFFFFu) | (s1 << 16), (s2 & 0xFFFFu) | (s3 << 16));
      // entries 4g..4g+3 are half of the high-nibble word g >> 1; the neighbouring lane holds the other half
      const u32 nib = ((s0 >> 16) & 15u) | (((s1 >> 16) & 15u) << 4) | (((s2 >> 16) & 15u) << 8) | (((s3 >> 16) & 15u) << 12);
      const u32 other = __shfl_xor_sync(0xffffffffu, nib, 1);
      if (in && (lane & 1u) == 0u) hi[g >> 1] = nib | (other << 16);
    }
  }
  __syncwarp();
}

template <int WSUB>
__device__ void build_lut_gen(const Ctx &c, const u8 *q, u32 *lut, u32 lane) {
  const u32 total = c.pq_m * kPqKsub;                  // a multiple of 256: no lane ever idles
  u16 *lo = (u16 *)lut;
  u32 *hi = lut + c.pq_m * (kPqKsub / 2);
  for (u32 e0 = lane; e0 < total; e0 += 32u * 4u) {
    u32 cw[4][WSUB];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const u32 *p = (const u32 *)(c.pq_cent + (u64)(e0 + 32u * (u32)u) * c.pq_dsub);
#pragma unroll
      for (int w = 0; w < WSUB; ++w) cw[u][w] = __ldg(p + w);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const u32 e = e0 + 32u * (u32)u;
      const u32 *qw = (const u32 *)(q + (e >> 8) * c.pq_dsub);
      u32 s = 0;
#pragma unroll
      for (int w = 0; w < WSUB; ++w) { const u32 d = __vabsdiffu4(cw[u][w], __ldg(qw + w)); s = __dp4a(d, d, s); }
      lo[e] = (u16)s;
      // eight consecutive entries (lanes 8k..8k+7) share one word of high nibbles
      u32 nib = ((s >> 16) & 15u) << ((lane & 7u) * 4u);
      nib |= __shfl_xor_sync(0xffffffffu, nib, 1);
      nib |= __shfl_xor_sync(0xffffffffu, nib, 2);
      nib |= __shfl_xor_sync(0xffffffffu, nib, 4);
      if ((lane & 7u) == 0) hi[e >> 3] = nib;
    }
  }
  __syncwarp();
}

__device__ __noinline__ void build_lut(const Ctx &c, u32 qid, u32 *lut, u32 lane) {
  const u8 *q = (const u8 *)c.queries + (u64)qid * c.vec_bytes;
  switch (c.pq_dsub >> 2) {
    case 1:
      if (((uintptr_t)c.pq_cent & 15u) == 0) build_lut_w1(c, q, lut, lane);
      else build_lut_gen<1>(c, q, lut, lane);
      break;
    case 2: build_lut_gen<2>(c, q, lut, lane); break;
    case 3: build_lut_gen<3>(c, q, lut, lane); break;
    default: build_lut_gen<4>(c, q, lut, lane); break;
  }
}
// One node per lane: the lane reads the node's code (pq_m bytes, 4 at a time) and sums pq_m
// independent table entries from shared memory -- no cross-lane reduction, 32 nodes per pass.
__device__ __forceinline__ u32 lane_adc(const Ctx &c, const u32 *lut, u32 v) {
  const u32 *code = (const u32 *)(c.pq_codes + (u64)v * c.pq_m);
  const u16 *lo = (const u16 *)lut;
  const u32 *hi = lut_hi(c, lut);
  u32 acc = 0;
  for (u32 w = 0; w < (c.pq_m >> 2); ++w) {
    const u32 cw = __ldg(code + w);
    acc += lut_get(lo, hi, ((4u * w + 0u) << 8) + (cw & 255u)) + lut_get(lo, hi, ((4u * w + 1u) << 8) + ((cw >> 8) & 255u)) +
           lut_get(lo, hi, ((4u * w + 2u) << 8) + ((cw >> 16) & 255u)) + lut_get(lo, hi, ((4u * w + 3u) << 8) + (cw >> 24));
  }
  return acc;
}

// ------------------------------------------------------------------------------------------
// query life cycle
// ------------------------------------------------------------------------------------------
__device__ void finish_query(const Ctx &c, u32 qs, u32 lane) {
  QHdr *h = c.hdr + qs;
  if (c.pq_m) pool_merge_dispatch(c, qs, 0, true, lane);
  __threadfence();
  __syncwarp();
  if (lane == 0) {
    const u32 qid = ld_u32(&h->qid);
    const u32 pd = ld_u32(&h->pages_distinct), ni = ld_u32(&h->n_iter), nx = ld_u32(&h->n_expand),
              ne = ld_u32(&h->n_eval), sd = ld_u32(&h->sum_deg);
    if (c.out_pages) c.out_pages[qid] = pd;
    if (c.out_counters) {
      u32 *o = c.out_counters + (u64)qid * 5;
      o[0] = pd; o[1] = ni; o[2] = nx; o[3] = ne; o[4] = sd;
    }
    stat_add(c, S_NEVAL, ne); stat_add(c, S_NEXPAND, nx); stat_add(c, S_SUMDEG, sd);
    stat_add(c, S_NITER, ni); stat_add(c, S_DONE, 1);
    __threadfence();
    u32 d = atomicAdd(&c.ctl->done, 1u) + 1u;
    if (d == c.nq) st_u32(&c.ctl->stop, 1u);
  }
}

__device__ __forceinline__ void reset_hdr(QHdr *h, u32 qid) {
  st_u32(&h->qid, qid); st_u32(&h->phase, PH_NEW); st_u32(&h->awaiting, 0); st_u32(&h->n_items, 0);
  st_u32(&h->reserved0, 0); st_u32(&h->list_len, 0); st_u32(&h->n_iter, 0); st_u32(&h->n_expand, 0);
  st_u32(&h->n_eval, 0); st_u32(&h->sum_deg, 0); st_u32(&h->pages_distinct, 0); st_u32(&h->pool_len, 0);
  st_u32(&h->worst_lo, 0xFFFFFFFFu); st_u32(&h->worst_hi, 0xFFFFFFFFu);
}

// The slot's query is done: admit the next unstarted query into the same slot, if any.
__device__ bool recycle_slot(const Ctx &c, u32 qs, u32 lane) {
  u32 nxt = 0;
  if (lane == 0) nxt = atomicAdd(&c.ctl->next_query, 1u);
  nxt = __shfl_sync(0xffffffffu, nxt, 0);
  if (nxt >= c.nq) return false;
  uint4 ff = make_uint4(kInvalidId, kInvalidId, kInvalidId, kInvalidId);
  uint4 *s4 = (uint4 *)(c.seen + (u64)qs * c.seen_cap);
  for (u32 i = lane; i < c.seen_cap / 4; i += 32) __stcg(s4 + i, ff);
  uint4 *p4 = (uint4 *)(c.pset + (u64)qs * c.pset_cap);
  for (u32 i = lane; i < c.pset_cap / 4; i += 32) __stcg(p4 + i, ff);
  uint4 *t4 = (uint4 *)(c.stash_tag + (u64)qs * c.stash_cap);
  for (u32 i = lane; i < c.stash_cap / 4; i += 32) __stcg(t4 + i, ff);
  if (lane == 0) reset_hdr(c.hdr + qs, nxt);
  __threadfence();
  __syncwarp();
  return true;
}

__device__ void copy_page(const Ctx &c, u32 idx, u32 lane);
__device__ bool warp_ticket(int *count, u32 *head, u32 &idx, u32 lane);

// One unit of the work that keeps pages moving, in priority order: execute a copy the proxy
// has admitted, consume a page the proxy has published (or a handed-off waiter chain), give
// a waiting page a slot.  Returns 0 if there was nothing to do, 1 for a copy, 2 for an arrival.
template <bool PQ>
__device__ __noinline__ u32 service_step(const Ctx &c, u32 lane) {
  u32 v;
  if (warp_ticket(&c.ctl->counts[0], &c.cs->copy_head, v, lane)) {    // the outstanding window waits on these
    copy_page(c, v, lane);
    return 1;
  }
  if (warp_ticket(&c.ctl->counts[1], &c.cs->comp_head, v, lane)) {    // completion v: its page has arrived
    const u64 e = __shfl_sync(0xffffffffu, ld_u64(c.ring_dev + (v & c.ring_mask)), 0);
    consume_arrival<PQ>(c, (u32)(e >> 8) & 0xFFFFFFu, lane);
    return 2;
  }
  if (warp_pop(c, c.arr, v, lane)) {                                  // handed-off waiter chains
    consume_arrival<PQ>(c, v, lane);
    return 2;
  }
  return 0;
}
__device__ void idle_step(const Ctx &c, u32 lane) {
  // nothing else to do: see whether a page waiting for a slot can be given one
  if (lane == 0 && (int)ld_u32((const u32 *)c.want.count) > 0) {
    LaneStats st = {0, 0, 0, 0, 0, 0};
    serve_want(c, kNil, st);
    stat_add(c, S_EVICT, st.evict); stat_add(c, S_POSTED, st.posted);
  }
  __syncwarp();
}

// Blocking mode (the demand-paging baseline the paper compares against, Section 5.1: misses
// "issue remote reads and wait for page readiness"): the warp keeps its query and waits in
// place until the batch it issued is complete.  It still moves pages while it waits -- someone
// has to -- but it never picks up another query, so at most one query per warp is in flight.
template <bool PQ>
__device__ __noinline__ bool wait_in_place(const Ctx &c, u32 qs, u32 lane) {
  const u64 t0 = globaltimer();
  for (u32 it = 0;; ++it) {
    if (uld(&c.hdr[qs].awaiting) == 0u) { __threadfence(); return true; }
    if (warp_stopped(c)) return false;
    if (service_step<PQ>(c, lane) == 0) { idle_step(c, lane); __nanosleep(200); }
    u32 late = ((it & 255u) == 255u && globaltimer() - t0 > c.timeout_ns) ? 1u : 0u;
    if (__shfl_sync(0xffffffffu, late, 0)) { if (lane == 0) raise(c, 5, 0xB5, qs); return false; }
  }
}

// lut_qid: the query whose table currently sits in this warp's shared memory (kept across calls,
// so a query that runs several phases in a row on one warp builds its table once).
template <bool PQ>
__device__ void run_query(const Ctx &c, u32 qs, u32 lane, u32 *lut, u32 &lut_qid) {
  QHdr *h = c.hdr + qs;
  u64 tp = c.prof ? globaltimer() : 0;
  for (u32 guard = 0; guard < 4u * c.max_iters + 64u; ++guard) {
    if (warp_stopped(c)) return;
    const u32 phase = uld(&h->phase);
    if (phase == PH_NEW) {
      const u32 qid = uld(&h->qid);
      if (lane == 0) {
        set_insert(c.seen + (u64)qs * c.seen_cap, c.seen_cap, c.entry);
        st_u32(c.items + (u64)qs * c.WR, c.entry);
        st_u32(&h->n_items, 1); st_u32(&h->n_eval, 1); st_u32(&h->phase, PH_EVAL);
      }
      __syncwarp();
      if (PQ) {
        if (lut_qid != qid) { build_lut(c, qid, lut, lane); lut_qid = qid; }
        phase_mark(c, tp, S_P_LUT, lane);
        if (lane == 0) st_u64(c.cand + (u64)qs * c.WR, mk_key(lane_adc(c, lut, c.entry), c.entry));
        __syncwarp();
      } else {
        const bool go = issue_batch<PQ>(c, qs, lane);
        phase_mark(c, tp, S_P_ISSUE_EVAL, lane);
        if (!go && !(c.blocking && wait_in_place<PQ>(c, qs, lane))) return;
      }
    } else if (phase == PH_EVAL) {
      const u32 nf = merge_select_dispatch(c, qs, lane);
      phase_mark(c, tp, S_P_MERGE, lane);
      if (nf == 0) {
        finish_query(c, qs, lane);
        phase_mark(c, tp, S_P_FINISH, lane);
        const bool more = recycle_slot(c, qs, lane);
        phase_mark(c, tp, S_P_RECYCLE, lane);
        if (!more) return;
        guard = 0;
        continue;
      }
      if (lane == 0) {
        const u32 it = ld_u32(&h->n_iter) + 1u;
        st_u32(&h->n_iter, it); st_u32(&h->n_expand, ld_u32(&h->n_expand) + nf);
        st_u32(&h->n_items, nf); st_u32(&h->phase, PH_EXPAND);
        if (it > c.max_iters) raise(c, 6, 0xA1, qs, it);
      }
      __syncwarp();
      {
        const bool go = issue_batch<PQ>(c, qs, lane);
        phase_mark(c, tp, S_P_ISSUE_EXP, lane);
        if (!go && !(c.blocking && wait_in_place<PQ>(c, qs, lane))) return;
      }
    } else {  // PH_EXPAND complete
      const u32 nf = uld(&h->n_items);
      const u32 nn = collect_neighbors(c, qs, lane);
      phase_mark(c, tp, S_P_COLLECT, lane);
      if (PQ) {
        pool_merge_dispatch(c, qs, nf, false, lane);
        phase_mark(c, tp, S_P_POOL, lane);
        const u32 qid = uld(&h->qid);
        if (lut_qid != qid) { build_lut(c, qid, lut, lane); lut_qid = qid; }
        phase_mark(c, tp, S_P_LUT, lane);
        const u32 *items = c.items + (u64)qs * c.WR;
        for (u32 base = 0; base < nn; base += 32) {
          const u32 i = base + lane;
          if (i < nn) {
            const u32 v = ld_u32(items + i);
            st_u64(c.cand + (u64)qs * c.WR + i, mk_key(lane_adc(c, lut, v), v));
          }
        }
        __syncwarp();
        phase_mark(c, tp, S_P_ADC, lane);
      }
      if (lane == 0) { st_u32(&h->n_items, nn); st_u32(&h->phase, PH_EVAL); }
      __syncwarp();
      if (!PQ && nn > 0) {
        const bool go = issue_batch<PQ>(c, qs, lane);
        phase_mark(c, tp, S_P_ISSUE_EVAL, lane);
        if (!go && !(c.blocking && wait_in_place<PQ>(c, qs, lane))) return;
      }
    }
  }
  if (lane == 0) raise(c, 6, 0xA2, qs);
}

// Execute the copy of admitted request idx (the proxy admits requests in ring order and
// publishes how many; the request itself is read from the device copy of the ring): pull
// the 4 KB page from the pinned store into its cache slot.  Any worker warp does this, ahead
// of all other work; only the page bytes cross the host link on this path.  The host is told
// as soon as the page's bytes have arrived on the GPU (they are in registers), so that no
// fence sits inside the proxy's outstanding window; the stores into the slot are then
// released to the consumers of the arrival through the slot's `filled` generation.
__device__ void copy_page(const Ctx &c, u32 idx, u32 lane) {
  const u64 cmd = __shfl_sync(0xffffffffu, ld_u64(c.ring_dev + (idx & c.ring_mask)), 0);
  const u32 page = (u32)(cmd >> 32), slot = (u32)(cmd >> 8) & 0xFFFFFFu;
  if (page >= c.n_units || slot >= c.n_slots) { if (lane == 0) raise(c, 8, 0xC1, idx, page, slot); return; }
  // what to pull: the whole page, or (selective materialisation, Section 7.2) only the
  // 16-byte-aligned span of its page that covers the wanted record
  const uint4 *src;
  u32 chunks = kPageBytes / 16u;      // page granularity moves the whole 4 KB block, as a block device would
  if (c.record_mode) {
    const u32 off = (page % c.npp) * c.node_bytes;
    src = (const uint4 *)(c.host_pages + (u64)(page / c.npp) * kPageBytes + (off & ~15u));
    chunks = ((off & 15u) + c.node_bytes + 15u) >> 4;
  } else {
    src = (const uint4 *)(c.host_pages + (u64)page * kPageBytes);
  }
  uint4 *dst = (uint4 *)(c.slot_data + (u64)slot * c.slot_bytes);
  uint4 v[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = (u32)i * 32u + lane < chunks ? __ldcs(src + i * 32 + lane) : make_uint4(0, 0, 0, 0);
  // The acknowledgement carries a checksum of the page above the lap tag (the host looks at the
  // tag only): a value that really depends on every loaded word, so the store cannot issue
  // before the page's bytes have arrived.
  u32 sum = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) sum ^= v[i].x ^ v[i].y ^ v[i].z ^ v[i].w;
  sum = __reduce_xor_sync(0xffffffffu, sum);
  if (lane == 0) st_sys_u32(c.fdone + (idx & c.ring_mask), ((u32)cmd & 0xFFu) | (sum << 8));
#pragma unroll
  for (int i = 0; i < 8; ++i) if ((u32)i * 32u + lane < chunks) __stcg(dst + i * 32 + lane, v[i]);
  __syncwarp();          // orders every lane's stores before lane 0's release below
  if (lane == 0) {
    const u32 gen = sm_gen(ld_u64(c.smeta + slot));
    __threadfence();
    st_u32(c.filled + slot, gen);
  }
}

// Debug aid: one snapshot of where slots, pages and queries are, taken by the poller warp.
__device__ void census(const Ctx &c, u32 lane) {
  u32 cnt[12] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
  for (u32 s = lane; s < c.n_slots; s += 32) {
    const u64 m = ld_u64(c.smeta + s);
    const u32 pg = sm_page(m);
    if (pg >= c.n_units) { cnt[0]++; continue; }
    const u64 w = ld_u64(c.ptab + pg);
    if (pw_slot(w) != s || pw_state(w) < P_FILLING) { cnt[1]++; continue; }   // slot between owners
    if (pw_state(w) == P_FILLING) cnt[2]++;
    else if (pw_state(w) == P_ARRIVED) cnt[3]++;
    else if (m & 1ull) cnt[4]++; else cnt[5]++;
  }
  for (u32 p = lane; p < c.n_units; p += 32) {
    const u32 st = pw_state(ld_u64(c.ptab + p));
    if (st == P_WANTED) cnt[6]++;
  }
  for (u32 q = lane; q < c.n_qslots; q += 32) {
    const u32 aw = ld_u32(&c.hdr[q].awaiting);
    if (aw > 0) { cnt[7]++; cnt[8] += aw; }
  }
  for (int i = 0; i < 12; ++i) cnt[i] = __reduce_add_sync(0xffffffffu, cnt[i]);
  if (lane == 0) {
    for (int i = 0; i < 9; ++i) c.ctl->census[i] = cnt[i];
    c.ctl->census[9] = (u32)*c.want.count; c.ctl->census[10] = (u32)c.ctl->counts[1]; c.ctl->census[11] = (u32)*c.run.count;
    c.ctl->census[12] = ld_u32(&c.ctl->done); c.ctl->census[13] = ld_u32(&c.ctl->ring_head);
  }
}

// Warp 0 of block 0 is the only warp that reads control words from host memory.  The proxy
// admits requests and publishes completions in ring order, and the GPU keeps its own copy of
// every descriptor, so all the host has to say is two counters: how many requests are
// admitted (their pages may be copied now) and how many completions are published (their
// pages have "arrived").  One 16-byte read per iteration fetches both and the abort word;
// the poller turns the deltas into tickets that worker warps take with fetch-and-add.
//
// A control read is a PCIe read like any other: its completion queues behind the page data
// already requested, so under load it takes about 6 us instead of 1.4 (46,000 reads in a 287 ms
// search).  One read in flight at a time is nevertheless the best found: with four in flight
// (each re-issued as soon as its result was used) every read took ~19 us, the proxy saw a
// service time of 33 us instead of 22, and config 3 fell from 34.8 k to 24.5 k QPS.
__device__ void poller(const Ctx &c, u32 lane) {
  u32 seen_pub = 0, seen_adm = 0, it = 0;
  const u64 t0 = globaltimer();
  bool census_done = c.census_ns == 0;
  for (;;) {
    if (warp_stopped(c)) break;
    if (!census_done && globaltimer() - t0 > c.census_ns) { census(c, lane); census_done = true; }
    u32 pub = 0, abort_req = 0, adm = 0;
    if (lane == 0) {
      const uint4 h = ld_sys_v4(c.host_ctl);
      pub = h.x; abort_req = h.y; adm = h.z;
      if (adm != seen_adm) atomicAdd(&c.ctl->counts[0], (int)(adm - seen_adm));
      if (pub != seen_pub) atomicAdd(&c.ctl->counts[1], (int)(pub - seen_pub));
      if (adm == seen_adm && pub == seen_pub) __nanosleep(100);
      seen_adm = adm; seen_pub = pub;
    }
    abort_req = __shfl_sync(0xffffffffu, abort_req, 0);
    if (abort_req) { if (lane == 0) raise(c, 5, 0xB1); break; }
    u32 late = ((++it & 63u) == 0 && globaltimer() - t0 > c.timeout_ns) ? 1u : 0u;
    if (__shfl_sync(0xffffffffu, late, 0)) { if (lane == 0) raise(c, 5, 0xB2); break; }
  }
  if (lane == 0) c.ctl->stats[S_POLLS] = it;
}

// Take one ticket from a (count, head) pair released by the poller; lane 0 only.
__device__ __forceinline__ bool take_ticket(int *count, u32 *head, u32 &idx) {
  if ((int)ld_u32((const u32 *)count) <= 0) return false;
  if (atomicSub(count, 1) <= 0) { atomicAdd(count, 1); return false; }
  idx = atomicAdd(head, 1u);
  return true;
}
__device__ bool warp_ticket(int *count, u32 *head, u32 &idx, u32 lane) {
  u32 ok = 0, v = 0;
  if (lane == 0) ok = take_ticket(count, head, v) ? 1u : 0u;
  idx = __shfl_sync(0xffffffffu, v, 0);
  return __shfl_sync(0xffffffffu, ok, 0) != 0u;
}

// Register budget: at most 80 per thread, so that 24 warps (61,440 registers) fit on an SM.  With
// PQ navigation the per-warp table in shared memory allows 12 warps at most, so that variant is
// built for 384 threads and may use twice the registers (no spills).
template <bool PQ>
__global__ void __launch_bounds__(PQ ? 384 : 768, 1) search_kernel(const Ctx c) {
  extern __shared__ u32 smem_lut[];
  const u32 lane = lane_id(), warp = threadIdx.x >> 5;
  if (blockIdx.x == 0 && warp == 0) { poller(c, lane); return; }
  u32 *lut = PQ ? smem_lut + (u64)warp * c.pq_m * kPqLutWords : nullptr;
  const u64 t0 = globaltimer();
  u32 idle = 0;
  // where the worker warps' time goes (ns, summed over warps): arrivals, query phases, idle
  u64 t_arr = 0, t_run = 0, t_idle = 0, t_cpy = 0, n_arr = 0, n_run = 0;
  u32 lut_qid = kInvalidId;
  u64 tp = t0;
  for (;;) {
    if (warp_stopped(c)) break;
    u32 v;
    if (idle) {
      // idle warps look at all five work counters with one 32-byte read (they sit together in
      // the control block) and back off exponentially: thousands of warps polling five hot
      // words would otherwise delay the very ticket atomics that hand out the work
      u32 any = 0;
      if (lane == 0) {
        const uint4 a = ld_v4((const u32 *)&c.ctl->counts[0]);
        const int w5 = (int)ld_u32((const u32 *)&c.ctl->counts[4]);
        any = ((int)a.x > 0 || (int)a.y > 0 || (int)a.z > 0 || (int)a.w > 0 || w5 > 0) ? 1u : 0u;
      }
      if (!__shfl_sync(0xffffffffu, any, 0)) {
        ++idle;
        __nanosleep(idle < 7 ? (64u << idle) : c.idle_ns);
        u32 late = ((idle & 127u) == 0 && globaltimer() - t0 > c.timeout_ns) ? 1u : 0u;
        if (__shfl_sync(0xffffffffu, late, 0)) { if (lane == 0) raise(c, 5, 0xB3); break; }
        { const u64 t = globaltimer(); t_idle += t - tp; tp = t; }
        continue;
      }
    }
    if (const u32 what = service_step<PQ>(c, lane)) {
      idle = 0;
      const u64 t = globaltimer();
      if (what == 1) t_cpy += t - tp; else { t_arr += t - tp; ++n_arr; }
      tp = t;
      continue;
    }
    if (warp_pop(c, c.run, v, lane)) {
      run_query<PQ>(c, v, lane, lut, lut_qid); idle = 0;
      const u64 t = globaltimer(); t_run += t - tp; tp = t; ++n_run;
      continue;
    }
    idle_step(c, lane);
    ++idle;
    { const u64 t = globaltimer(); t_idle += t - tp; tp = t; }
  }
  if (lane == 0) {
    atomicAdd((unsigned long long *)&c.ctl->stats[S_T_ARR], t_arr);
    atomicAdd((unsigned long long *)&c.ctl->stats[S_T_RUN], t_run);
    atomicAdd((unsigned long long *)&c.ctl->stats[S_T_IDLE], t_idle);
    atomicAdd((unsigned long long *)&c.ctl->stats[S_N_ARR], n_arr);
    atomicAdd((unsigned long long *)&c.ctl->stats[S_T_CPY], t_cpy);
  }
}

// ------------------------------------------------------------------------------------------
// set-up kernels
// ------------------------------------------------------------------------------------------
__global__ void init_kernel(const Ctx c) {
  const u32 tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
  for (u32 i = tid; i < c.n_qslots; i += nth) reset_hdr(c.hdr + i, i);
  // runnable queue starts with every slot; the others start empty
  u64 *run = (u64 *)c.run.buf, *arr = (u64 *)c.arr.buf, *want = (u64 *)c.want.buf;
  for (u32 i = tid; i <= c.run.mask; i += nth) run[i] = i < c.n_qslots ? (((u64)(i + 1u) << 32) | i) : ((u64)i << 32);
  for (u32 i = tid; i <= c.arr.mask; i += nth) arr[i] = (u64)i << 32;
  for (u32 i = tid; i <= c.want.mask; i += nth) want[i] = (u64)i << 32;
  if (tid == 0) {
    Ctl *ctl = c.ctl;
    ctl->stop = 0; ctl->status = 0; ctl->next_query = c.n_qslots; ctl->done = 0; ctl->ring_head = 0;
    for (int i = 0; i < 16; ++i) ctl->q_heads[i] = 0;
    for (int i = 0; i < 8; ++i) ctl->counts[i] = 0;
    for (int i = 0; i < 8; ++i) ctl->dbg[i] = 0;
    *c.run.tail = c.n_qslots;
    *c.run.count = (int)c.n_qslots;
    ctl->counts[0] = 0; ctl->counts[1] = 0; c.cs->copy_head = 0; c.cs->comp_head = 0; c.cs->in_flight = 0;
  }
}

// Empty the cache; slots 0..preloaded-1 hold pages 0..preloaded-1 (their bytes were copied
// there by the host before this kernel) and are RESIDENT.
__global__ void cache_reset_kernel(const Ctx c, u32 preloaded) {
  const u32 tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
  for (u32 p = tid; p < c.n_units; p += nth) c.ptab[p] = p < preloaded ? mk_pw(P_RESIDENT, p, 1) : kAbsentWord;
  for (u32 s = tid; s < c.n_slots; s += nth) {
    c.smeta[s] = s < preloaded ? mk_sm(s, 1, 1) : mk_sm(kInvalidId, 0, 0);
    c.parts[s] = 0;
    c.filled[s] = s < preloaded ? 1u : 0u;
  }
  if (tid == 0) { c.cs->bump = preloaded; c.cs->hand = 0; }
}

// ------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------
// With lazy module loading the first launch of a kernel may need a context-wide
// synchronisation; querying the attributes loads all code at open time instead, so that no
// launch ever has to wait behind a resident persistent kernel.
cudaError_t preload_kernels() {
  cudaFuncAttributes a;
  cudaError_t e;
  if ((e = cudaFuncGetAttributes(&a, search_kernel<false>)) != cudaSuccess) return e;
  if ((e = cudaFuncGetAttributes(&a, search_kernel<true>)) != cudaSuccess) return e;
  if ((e = cudaFuncGetAttributes(&a, init_kernel)) != cudaSuccess) return e;
  return cudaFuncGetAttributes(&a, cache_reset_kernel);
}

cudaError_t launch_init(const Ctx &c, cudaStream_t s) {
  init_kernel<<<148, 256, 0, s>>>(c);
  return cudaGetLastError();
}

cudaError_t launch_cache_reset(const Ctx &c, u32 preloaded, cudaStream_t s) {
  cache_reset_kernel<<<148, 256, 0, s>>>(c, preloaded);
  return cudaGetLastError();
}

static size_t search_smem(const Ctx &c, u32 warps) { return c.pq_m ? (size_t)warps * c.pq_m * kPqLutWords * 4 : 0; }

cudaError_t search_occupancy(u32 pq_m, u32 warps_per_block, int *blocks_per_sm) {
  if (pq_m) {
    const size_t smem = (size_t)warps_per_block * pq_m * kPqLutWords * 4;
    cudaError_t e = cudaFuncSetAttribute(search_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, search_kernel<true>, warps_per_block * 32, smem);
  }
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, search_kernel<false>, warps_per_block * 32, 0);
}

cudaError_t launch_search(const Ctx &c, u32 blocks, u32 warps_per_block, cudaStream_t s) {
  const size_t smem = search_smem(c, warps_per_block);
  if (c.pq_m) {
    cudaError_t e = cudaFuncSetAttribute(search_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    search_kernel<true><<<blocks, warps_per_block * 32, smem, s>>>(c);
  } else {
    search_kernel<false><<<blocks, warps_per_block * 32, 0, s>>>(c);
  }
  return cudaGetLastError();
}

}  // namespace gorio
