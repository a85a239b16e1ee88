// What happens when a page arrives: its waiter chain is consumed by whichever warp picks the
// arrival up, in segments, and the page then becomes evictable.
// Part of the persistent search kernel; included by search_kernels.cu in this order.
#pragma once
#include "../gorio_internal.h"

namespace gorio {

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
  if (lane == 0 && !c.dma_fill) {
    // acquire the copier's stores into the slot (normally long done: the completion was
    // published at least the remote latency after the bytes arrived).  With copy-engine
    // fills the proxy publishes only after the copy has completed, so there is nothing to wait for.
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

}  // namespace gorio
