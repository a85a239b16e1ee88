// The HBM page cache and miss tracker: per-page state words, slot allocation by clock, request
// descriptors, lookup / miss registration.
// Part of the persistent search kernel; included by search_kernels.cu in this order.
#pragma once
#include "../gorio_internal.h"

namespace gorio {

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

// Post a request descriptor: one 64-bit word [page:32][slot:24][lap:8].  The ring holds at least
// twice as many entries as there are slots, and every pending request owns a distinct FILLING
// slot, so an entry is never overwritten before it has been consumed.  (Section 3.2: reserve a
// descriptor slot atomically, record page id and target cache slot, publish through a ready flag
// -- here the lap tag inside the word.)
// The worker writes the descriptor into the DEVICE copy of the ring only; the poster warp forwards
// it to the host-visible ring (see poster()).  Worker warps therefore never have a store to host
// memory in flight behind a post: every later fence of such a warp would have to wait for it, and
// with the host link saturated by page reads that wait was ~5 us per fence and 18 us for the
// system-scope fence that used to stand here.  A posted request waits in the ring for its turn
// in the proxy's window anyway (the backlog is several windows deep), so the microsecond the
// forwarding adds costs nothing.
__device__ __forceinline__ void post_request(const Ctx &c, u32 page, u32 slot) {
  const u32 idx = atomicAdd(&c.ctl->ring_head, 1u);
  atomicAdd(&c.cs->in_flight, 1);
  const u32 lap = ((idx >> c.ring_shift) % 255u) + 1u;
  const u64 e = ((u64)page << 32) | ((u64)slot << 8) | lap;
  __threadfence();             // page word and slot label before the descriptor can be seen
  st_u64(c.ring_dev + (idx & c.ring_mask), e);   // also what copy and arrival tickets refer to
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
//
// Joining a waiter list is a compare-and-swap on the page word, and a batch starts with every
// query joining the entry node's page at once: thousands of lanes retry against one word, and
// every success makes all other attempts in flight fail.  The loop is lock-free (some lane
// always gets through), so the retry bound is generous; a failed attempt continues from the
// word the compare-and-swap returned instead of re-reading it, and backs off for a short,
// per-lane pseudo-random time once it has failed a few times.  (A bound of 4,096 attempts
// without back-off was exceeded once in some two hundred full-size searches.)
constexpr u32 kLookupTries = 1u << 20;
__device__ u32 page_lookup(const Ctx &c, u32 page, u32 g, u64 first, u32 &slot, u32 &gen, LaneStats &st) {
  u64 *pw = c.ptab + page;
  u64 w = first;
  for (u32 tries = 0; tries < kLookupTries; ++tries) {
    const u32 s = pw_state(w);
    if (s == P_RESIDENT || s == P_ARRIVED) { slot = pw_slot(w); gen = pw_low(w); return LK_HIT; }
    st_u32(c.wrec + g, s == P_ABSENT ? kNil : pw_low(w));
    __threadfence();
    const u64 mine = s == P_ABSENT ? mk_pw(P_WANTED, 0, g) : ((w & 0xFFFFFFFF00000000ull) | g);
    const u64 old = atomicCAS((unsigned long long *)pw, w, mine);
    if (old != w) {                                   // lost the race: `old` is the word as it is now
      w = old;
      if (tries >= 4) __nanosleep(32u * (tries < 32u ? tries : 32u) + (hash32(g + tries) & 1023u));
      continue;
    }
    st.missed++;
    if (s != P_ABSENT) { st.joins++; return LK_WAIT; }
    // First requester: find the page a slot -- but never ahead of pages that already wait for
    // one.  Requests leave in the order in which their pages were first wanted, so each has
    // gathered as many waiters as it can by the time it is posted; letting new pages jump the
    // queue whenever the backlog had room cost 16 % more fetches on config 3.
    const bool room = may_post(c);
    const bool queued = (int)ld_u32((const u32 *)c.want.count) > 0;
    u32 prev_gen = 0;
    const u32 sl = (room && !queued) ? alloc_slot(c, kNil, st, prev_gen) : kNil;
    if (sl != kNil) {
      assign_and_post(c, page, sl, prev_gen, mine, st);
    } else {
      q_push(c, c.want, page);
      if (room) serve_want(c, kNil, st);      // the oldest waiting page takes the opening
    }
    return LK_WAIT;
  }
  raise(c, 8, 0x42, page, g);
  return LK_WAIT;
}

}  // namespace gorio
