// Query life cycle and the persistent kernel: page copies, the host poller, the poster, the puller
// warps, ticket hand-out, the worker loop.
// Part of the persistent search kernel; included by search_kernels.cu in this order.
#pragma once
#include "../gorio_internal.h"

namespace gorio {

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
  const uint4 sclear = c.seen_bitmap ? make_uint4(0, 0, 0, 0) : ff;
  for (u32 i = lane; i < c.seen_cap / 4; i += 32) __stcg(s4 + i, sclear);
  uint4 *p4 = (uint4 *)(c.pset + (u64)qs * c.pset_cap);
  const uint4 pclear = c.pset_bitmap ? make_uint4(0, 0, 0, 0) : ff;
  for (u32 i = lane; i < c.pset_cap / 4; i += 32) __stcg(p4 + i, pclear);
  uint4 *t4 = (uint4 *)(c.stash_tag + (u64)qs * c.stash_cap);
  for (u32 i = lane; i < c.stash_cap / 4; i += 32) __stcg(t4 + i, ff);
  if (lane == 0) reset_hdr(c.hdr + qs, nxt);
  __threadfence();
  __syncwarp();
  return true;
}

__device__ void copy_page(const Ctx &c, u32 idx, u32 lane);
template <bool PQ> __device__ void resident_worker(const Ctx &c, u32 lane, u32 *lut, u32 *ws);
__host__ __device__ inline u32 resident_warp_words(u32 WR);
__device__ bool warp_ticket(int *count, u32 *head, u32 &idx, u32 lane);
__device__ void puller(const Ctx &c, u32 lane);

// One unit of the work that keeps pages moving, in priority order: execute a copy the proxy
// has admitted, consume a page the proxy has published (or a handed-off waiter chain), give
// a waiting page a slot.  Returns 0 if there was nothing to do, 1 for a copy, 2 for an arrival.
template <bool PQ>
__device__ __noinline__ u32 service_step(const Ctx &c, u32 lane) {
  u32 v;
  if (!c.pullers && warp_ticket(&c.ctl->counts[0], &c.cs->copy_head, v, lane)) {    // the outstanding window waits on these
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

// Blocking mode (the demand-paging baseline the paper compares against, Section 5.1, in which
// a miss starts the remote read and the requester stays put until the page is there): the warp keeps its query and waits in
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
__device__ void run_query(const Ctx &c, u32 qs, u32 lane, u32 *lut, u32 &lut_qid, u32 *ws) {
  QHdr *h = c.hdr + qs;
  u64 tp = c.prof ? globaltimer() : 0;
  for (u32 guard = 0; guard < 4u * c.max_iters + 64u; ++guard) {
    if (warp_stopped(c)) return;
    const u32 phase = uld(&h->phase);
    if (phase == PH_NEW) {
      const u32 qid = uld(&h->qid);
      if (lane == 0) {
        if (c.seen_bitmap) bit_insert(c.seen + (u64)qs * c.seen_cap, c.entry);
        else set_insert(c.seen + (u64)qs * c.seen_cap, c.seen_cap, c.entry);
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
      const u32 nf = merge_select_dispatch(c, qs, lane, (u64 *)ws);
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
// the 4 KB page from the pinned store into its cache slot.  A puller warp does this (or, in the
// shared scheme, any worker warp, ahead of all other work); only the page bytes cross the host link
// on this path.  The host is told
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
  const u64 t_issue = c.prof ? globaltimer() : 0;
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
  if (c.prof && lane == 0) atomicAdd((unsigned long long *)&c.ctl->stats[S_C_DATA], globaltimer() - t_issue);
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
// the poller passes the admitted count on to the puller warps (a word they wait on) and turns
// new completions into tickets that worker warps take with fetch-and-add (in the shared scheme
// admissions become tickets too).
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
    if (!census_done && globaltimer() - t0 > c.census_ns) { census(c, lane); census_done = true; }
    u32 pub = 0, abort_req = 0, adm = 0, stop = 0;
    if (lane == 0) {
      const uint4 h = ld_sys_v4(c.host_ctl);       // ~6 us under load; the stop flag's load rides along
      stop = ld_u32(&c.ctl->stop);
      pub = h.x; abort_req = h.y; adm = h.z;
      if (adm != seen_adm) {
        if (c.pullers) st_u32(&c.ctl->adm_seen, adm);        // the puller warps wait on this word
        else atomicAdd(&c.ctl->counts[0], (int)(adm - seen_adm));
      }
      if (pub != seen_pub) atomicAdd(&c.ctl->counts[1], (int)(pub - seen_pub));
      if (adm == seen_adm && pub == seen_pub) __nanosleep(100);
      seen_adm = adm; seen_pub = pub;
    }
    if (__shfl_sync(0xffffffffu, stop, 0)) break;
    abort_req = __shfl_sync(0xffffffffu, abort_req, 0);
    if (abort_req) { if (lane == 0) raise(c, 5, 0xB1); break; }
    u32 late = ((++it & 63u) == 0 && globaltimer() - t0 > c.timeout_ns) ? 1u : 0u;
    if (__shfl_sync(0xffffffffu, late, 0)) { if (lane == 0) raise(c, 5, 0xB2); break; }
  }
  if (lane == 0) c.ctl->stats[S_POLLS] = it;
}

// Warp 1 of block 0 forwards request descriptors from the device copy of the ring to the
// host-visible ring, in ring order, up to 32 per look (lane i looks at entry next + i; the ready
// ones form a prefix as far as this look is concerned).  It is the only warp that writes
// descriptors to host memory.
__device__ void poster(const Ctx &c, u32 lane) {
  u32 next = 0, it = 0;
  const u64 t0 = globaltimer();
  for (;;) {
    const u32 idx = next + lane;
    const u64 e = ld_u64(c.ring_dev + (idx & c.ring_mask));
    const bool ready = (u32)(e & 0xFFu) == ((idx >> c.ring_shift) % 255u) + 1u;
    const u32 n = (u32)__ffs((int)~__ballot_sync(0xffffffffu, ready)) - 1u;      // leading ready entries (32 if all)
    const u32 cnt = n > 32u ? 32u : n;
    if (lane < cnt) st_sys_u64(c.ring + (idx & c.ring_mask), e);
    next += cnt;
    if (cnt == 0) {
      if (warp_stopped(c)) break;
      __nanosleep(200);
      u32 late = ((++it & 1023u) == 0 && globaltimer() - t0 > c.timeout_ns) ? 1u : 0u;
      if (__shfl_sync(0xffffffffu, late, 0)) { if (lane == 0) raise(c, 5, 0xB4); break; }
    }
  }
}

// Puller warps (the last warp of every block when pages are pulled by the SMs): each claims the
// next request index in ring order ahead of time, waits until the poller has seen that request
// admitted, and pulls its page.  Pulls are thus issued in admission order, by warps that are
// doing nothing else, the moment the admission is known on the GPU -- the proxy publishes
// completions in that same order, so a pull that starts late holds up every request behind it.
__device__ void puller(const Ctx &c, u32 lane) {
  const u64 t0 = globaltimer();
  u64 t_cpy = 0;
  for (;;) {
    u32 idx = 0;
    if (lane == 0) idx = atomicAdd(&c.cs->copy_head, 1u);
    idx = __shfl_sync(0xffffffffu, idx, 0);
    bool go = false;
    for (u32 it = 0;; ++it) {
      u32 st = 0;
      if (lane == 0) {
        if ((int)(ld_u32(&c.ctl->adm_seen) - idx) > 0) st = 1u;
        else if (ld_u32(&c.ctl->stop)) st = 2u;
        else if ((it & 1023u) == 1023u && globaltimer() - t0 > c.timeout_ns) st = 3u;
      }
      st = __shfl_sync(0xffffffffu, st, 0);
      if (st == 1u) { go = true; break; }
      if (st == 3u && lane == 0) raise(c, 5, 0xB6, idx);
      if (st) break;
      __nanosleep(it < 16u ? 50u : 400u);
    }
    if (!go) break;
    const u64 t1 = globaltimer();
    copy_page(c, idx, lane);
    t_cpy += globaltimer() - t1;
  }
  if (lane == 0) atomicAdd((unsigned long long *)&c.ctl->stats[S_T_CPY], t_cpy);
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

// Register budget: MAXT threads per block, one block per SM.  768 threads (24 warps, used when
// the whole index is resident and there are many queries per SM) leave 80 registers per thread;
// 512 threads (the default 16 warps whenever pages can be missed) leave 128 and need no spills.
// With PQ navigation the per-warp table in shared memory allows 12 warps at most, so that
// variant is built for 384 threads (168 registers).
template <bool PQ, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) search_kernel(const Ctx c) {
  extern __shared__ u32 smem_lut[];
  const u32 lane = lane_id(), warp = threadIdx.x >> 5;
  if (blockIdx.x == 0 && warp == 0) { poller(c, lane); return; }
  if (blockIdx.x == 0 && warp == 1 && !c.identity) { poster(c, lane); return; }     // (nothing is ever posted when the whole index is resident)
  if (blockIdx.x < c.pullers && warp == (blockDim.x >> 5) - 1u) { puller(c, lane); return; }
  u32 *lut = PQ ? smem_lut + (u64)warp * c.pq_m * kPqLutWords : nullptr;
  // this warp's candidate area (WR keys and 16 frontier ids), behind the PQ tables
  u32 *ws = smem_lut + (PQ ? (u64)(blockDim.x >> 5) * c.pq_m * kPqLutWords : 0) + (u64)warp * resident_warp_words(c.WR);
  if (c.resident_fast) {                   // whole index resident: queries run start to end on one warp
    resident_worker<PQ>(c, lane, lut, ws);
    return;
  }
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
      run_query<PQ>(c, v, lane, lut, lut_qid, ws); idle = 0;
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

}  // namespace gorio
