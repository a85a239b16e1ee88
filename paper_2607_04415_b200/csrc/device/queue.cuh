// Bounded multi-producer multi-consumer queues in HBM (runnable queries, handed-off waiter
// chains, pages waiting for a slot).
// Part of the persistent search kernel; included by search_kernels.cu in this order.
#pragma once
#include "../gorio_internal.h"

namespace gorio {

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

}  // namespace gorio
