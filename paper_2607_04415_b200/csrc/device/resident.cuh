// The whole-index-resident fast path: when every page sits in the slot of its own number for the
// life of the call, nothing can miss, so a query never parks and no other warp ever touches its
// state.  The warp that takes a query then runs it from admission to output in one go: the sorted
// list stays in registers, the frontier and the iteration's candidates go through a small
// per-warp area of shared memory, adjacency lists are read straight from the pages, and nothing
// but the exact visited / page sets (too large for anything but HBM/L2) is kept in global memory.
// Same algorithm, same keys, same counters as the general path -- only where the state lives differs.
// Part of the persistent search kernel; included by search_kernels.cu in this order.
#pragma once
#include "../gorio_internal.h"

namespace gorio {

// shared memory of one warp on this path: WR candidate words (node id, then the node's key) and
// up to 16 frontier ids
__host__ __device__ inline u32 resident_warp_words(u32 WR) { return 2u * WR + 16u; }

// Insert into a per-query exact set (bitmap or hash set): 1 = new, 0 = present, 2 = full.
__device__ __forceinline__ u32 qset_insert(u32 *tab, u32 cap, bool bitmap, u32 v) {
  return bitmap ? bit_insert(tab, v) : set_insert(tab, cap, v);
}

// Distance of one node per active lane on this path (exact navigation or rerank distances).
__device__ __forceinline__ u32 resident_exact(const Ctx &c, bool active, u32 qid, u32 node, u32 lane) {
  if (c.vec128) return lane_score128(c, active, qid, node, unit_of(c, node));
  // vectors that are not whole 16-byte chunks: one node at a time, the warp strides over its words
  u32 dist = 0;
  for (u32 m = __ballot_sync(0xffffffffu, active); m; m &= m - 1) {
    const u32 src = __ffs(m) - 1;
    const u32 v = __shfl_sync(0xffffffffu, node, src);
    const u32 d = warp_dist(c, rec_ptr(c, unit_of(c, v), v), qid, lane);
    if (lane == src) dist = d;
  }
  return dist;
}

// H: list keys per lane (L <= 32*H).
template <bool PQ, int H>
__device__ __noinline__ void resident_query(const Ctx &c, u32 qs, u32 qid, u32 lane, u32 *lut, u32 &lut_qid, u32 *ws) {
  u64 *wk = (u64 *)ws;                     // [WR] candidate: node id, later its key
  u32 *fr = ws + 2u * c.WR;                // [16] frontier node ids
  u32 *seen = c.seen + (u64)qs * c.seen_cap;
  u32 *pset = c.pset + (u64)qs * c.pset_cap;
  const bool seen_bm = c.seen_bitmap != 0, pset_bm = c.pset_bitmap != 0;
  const u32 lt = (1u << lane) - 1u;
  u64 xl[H];                               // the sorted list, in registers from admission to output
#pragma unroll
  for (int r = 0; r < H; ++r) xl[r] = kPadKey;
  u32 len = 0, n_iter = 0, n_expand = 0, n_eval = 1, my_deg = 0, my_pages = 0, pool_len = 0;
  u64 pool = kPadKey;                      // PQ: rerank pool, one key per lane (K + W <= 32 on this path)
  u64 tp = c.prof ? globaltimer() : 0;     // debug profile: warp time per step

  if (PQ && lut_qid != qid) { build_lut(c, qid, lut, lane); lut_qid = qid; }
  phase_mark(c, tp, S_P_LUT, lane);
  // admission: the entry node is the first iteration's only candidate
  if (lane == 0) { qset_insert(seen, c.seen_cap, seen_bm, c.entry); wk[0] = (u64)c.entry; }
  u32 out = 1;
  __syncwarp();

  for (;;) {
    // score the new nodes, one per lane: exact navigation from their own records (their pages are
    // the ones touched), PQ navigation from resident codes.  Only keys that beat the list's worst
    // are kept (the others cannot enter it), compacted in place.
    const u64 worst = list_worst<H>(xl, len, c.L, lane);
    u32 kept = 0;
    for (u32 base = 0; base < out; base += 32u) {
      const u32 i = base + lane;
      const bool act = i < out;
      const u32 v = act ? (u32)wk[i] : 0u;
      u32 d, r = 0;
      if (PQ) {
        d = act ? lane_adc(c, lut, v) : 0u;
      } else {
        if (act) r = qset_insert(pset, c.pset_cap, pset_bm, v / c.npp);      // in flight with the vector loads
        d = resident_exact(c, act, qid, v, lane);
        if (r == 1u) ++my_pages; else if (r == 2u) raise(c, 6, 0x81, qs, v / c.npp);
      }
      const u64 key = mk_key(d, v);
      const bool keep = act && key < worst;
      const u32 b = __ballot_sync(0xffffffffu, keep);       // (every lane has read its entry by now)
      if (keep) wk[kept + __popc(b & lt)] = key;
      kept += __popc(b);
    }
    __syncwarp();
    phase_mark(c, tp, PQ ? S_P_ADC : S_P_ISSUE_EVAL, lane);

    list_insert<H, false>(xl, len, wk, kept, c.L, lane);
    __syncwarp();                          // the candidate area is rewritten below
    phase_mark(c, tp, S_P_MERGE, lane);

    // frontier: the first W unexpanded entries in key order, marked before anything is inserted
    u32 taken = 0;
#pragma unroll
    for (int r = 0; r < H; ++r) {
      const u32 e = (u32)r * 32u + lane;
      const bool un = e < len && !(xl[r] & 1ull);
      const u32 b = __ballot_sync(0xffffffffu, un);
      if (taken < c.W && b) {
        const u32 rank = taken + __popc(b & lt);
        if (un && rank < c.W) { xl[r] |= 1ull; fr[rank] = key_id(xl[r]); }
        taken = min(c.W, taken + (u32)__popc(b));
      }
    }
    if (taken == 0) break;
    __syncwarp();
    const u32 stop_seen = ld_u32(&c.ctl->stop);      // consumed after the adjacency round trips below
    ++n_iter; n_expand += taken;
    if (n_iter > c.max_iters) { if (lane == 0) raise(c, 6, 0xA1, qs, n_iter); return; }

    // PQ navigation: the expanded nodes' pages are the ones touched, and their exact distances go
    // into the rerank pool
    if (PQ) {
      const bool mine = lane < taken;
      const u32 u = mine ? fr[lane] : 0u;
      u32 r = 0;
      if (mine) r = qset_insert(pset, c.pset_cap, pset_bm, u / c.npp);
      const u32 d = resident_exact(c, mine, qid, u, lane);
      if (r == 1u) ++my_pages; else if (r == 2u) raise(c, 6, 0x81, qs, u / c.npp);
      const u64 key = mk_key(d, u);
      // new keys go to lanes pool_len .. pool_len+taken-1, then one 32-key sort; the best K stay
      const u64 moved = __shfl_sync(0xffffffffu, key, (lane - pool_len) & 31u);
      if (lane >= pool_len && lane < pool_len + taken) pool = moved;
      u64 p1[1] = {pool};
      bitonic_sort<1>(p1, lane);
      pool_len = min(c.K, pool_len + taken);
      pool = lane < pool_len ? p1[0] : kPadKey;
      phase_mark(c, tp, S_P_POOL, lane);
    }

    // adjacency lists straight from the pages, through the exact visited set, survivors compacted
    // into shared memory; eight neighbour positions per lane in flight
    out = 0;
    const u32 total = taken * c.R;
    for (u32 base = 0; base < total; base += 256u) {
      u32 v[8], dg[8], pos[8];
      bool ok[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const u32 p = base + 32u * (u32)k + lane;
        ok[k] = p < total;
        const u32 f = ok[k] ? p / c.R : 0u;
        pos[k] = p - f * c.R;
        const u32 u = fr[f];
        const u32 *adj = (const u32 *)(rec_ptr(c, unit_of(c, u), u) + c.vec_bytes);
        dg[k] = ok[k] ? __ldcg(adj) : 0u;
        v[k] = ok[k] ? __ldcg(adj + 1 + pos[k]) : kInvalidId;
      }
      // all eight insertions in flight before any result is looked at
      u32 r[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        r[k] = 3u;                                           // not a neighbour position
        if (ok[k] && dg[k] <= c.R && pos[k] < dg[k]) r[k] = v[k] < c.n_nodes ? qset_insert(seen, c.seen_cap, seen_bm, v[k]) : 4u;
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (ok[k] && pos[k] == 0u) {                         // one lane per expanded node
          if (dg[k] > c.R) raise(c, 7, 0x91, qs, dg[k]); else my_deg += dg[k];
        }
        if (r[k] == 4u) raise(c, 7, 0x92, qs, v[k]);
        else if (r[k] == 2u) raise(c, 6, 0x93, qs, v[k]);
        const u32 b = __ballot_sync(0xffffffffu, r[k] == 1u);
        if (r[k] == 1u) wk[out + __popc(b & lt)] = (u64)v[k];
        out += __popc(b);
      }
    }
    n_eval += out;
    __syncwarp();
    phase_mark(c, tp, S_P_COLLECT, lane);
    // a corrupt page or a full set met earlier (by any lane), or an abort from outside
    if (__any_sync(0xffffffffu, stop_seen != 0u)) return;
  }

  // output and counters
  if (PQ) {
    if (lane < c.K) write_result(c, qid, lane, pool, lane < pool_len);
  } else {
#pragma unroll
    for (int r = 0; r < H; ++r) {
      const u32 e = (u32)r * 32u + lane;
      if (e < c.K) write_result(c, qid, e, xl[r], e < len);
    }
  }
  const u32 pd = __reduce_add_sync(0xffffffffu, my_pages);
  const u32 sum_deg = __reduce_add_sync(0xffffffffu, my_deg);
  __threadfence();
  __syncwarp();
  if (lane == 0) {
    if (c.out_pages) c.out_pages[qid] = pd;
    if (c.out_counters) {
      u32 *o = c.out_counters + (u64)qid * 5;
      o[0] = pd; o[1] = n_iter; o[2] = n_expand; o[3] = n_eval; o[4] = sum_deg;
    }
    stat_add(c, S_NEVAL, n_eval); stat_add(c, S_NEXPAND, n_expand); stat_add(c, S_SUMDEG, sum_deg);
    stat_add(c, S_NITER, n_iter); stat_add(c, S_DONE, 1);
    stat_add(c, S_HIT, PQ ? n_expand : n_eval + n_expand);     // every page lookup was served from a resident slot
    __threadfence();
    const u32 d = atomicAdd(&c.ctl->done, 1u) + 1u;
    if (d == c.nq) st_u32(&c.ctl->stop, 1u);
  }
  phase_mark(c, tp, S_P_FINISH, lane);
}

template <bool PQ>
__device__ void resident_dispatch(const Ctx &c, u32 qs, u32 qid, u32 lane, u32 *lut, u32 &lut_qid, u32 *ws) {
  if (c.L <= 32) resident_query<PQ, 1>(c, qs, qid, lane, lut, lut_qid, ws);
  else if (c.L <= 64) resident_query<PQ, 2>(c, qs, qid, lane, lut, lut_qid, ws);
  else if (c.L <= 128) resident_query<PQ, 4>(c, qs, qid, lane, lut, lut_qid, ws);
  else resident_query<PQ, 8>(c, qs, qid, lane, lut, lut_qid, ws);
}

// Worker loop of the resident fast path: take a query slot, run its query to the end, admit the
// next unstarted query into the same slot, until none is left.
template <bool PQ>
__device__ void resident_worker(const Ctx &c, u32 lane, u32 *lut, u32 *ws) {
  u32 lut_qid = kInvalidId, qs = 0;
  bool have = false;
  const u64 t0 = globaltimer();
  for (;;) {
    if (warp_stopped(c)) break;
    if (!have && !warp_pop(c, c.run, qs, lane)) break;      // no slot left to take: done
    const u32 qid = uld(&c.hdr[qs].qid);
    resident_dispatch<PQ>(c, qs, qid, lane, lut, lut_qid, ws);
    u64 tr = c.prof ? globaltimer() : 0;
    have = recycle_slot(c, qs, lane);                        // the next unstarted query, in the same slot
    phase_mark(c, tr, S_P_RECYCLE, lane);
  }
  if (lane == 0) atomicAdd((unsigned long long *)&c.ctl->stats[S_T_RUN], globaltimer() - t0);
}

}  // namespace gorio
