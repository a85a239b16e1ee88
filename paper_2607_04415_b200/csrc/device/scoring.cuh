// Distances and the consumption of page items: scoring nodes against their queries, adjacency
// copies, the adjacency stash.
// Part of the persistent search kernel; included by search_kernels.cu in this order.
#pragma once
#include "../gorio_internal.h"

namespace gorio {

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

// Lane-per-node scoring with 128-bit loads: every active lane scores its OWN node against its own
// query, so up to 32 nodes are in flight per pass and no lane waits on another's data.  A vector
// is handled in blocks of eight 16-byte chunks: the lane loads the nine aligned chunks that cover
// the block (records are only 4-byte aligned in a page), shifts them down by its own misalignment
// (0..3 words, two conditional-move levels, no dynamic register indexing) and reduces against the
// query's chunks, which are 16-byte aligned.  uint8: |a-b| per byte and a 4-way dot product into
// one exact u32.  fp32: eight accumulators, accumulator t taking the chunks t, t+8, t+16 in that
// order, combined as ((a0+a4)+(a2+a6))+((a1+a5)+(a3+a7)) -- the summation order of an 8-lane
// butterfly, so the value does not depend on which path scored the node.
__device__ __forceinline__ u32 lane_score128(const Ctx &c, bool active, u32 qid, u32 node, u32 slot) {
  const u32 nchunk = c.vec_bytes >> 4;                       // <= 24 (checked on the host: vec128)
  const u32 off = rec_off(c, node);
  const u32 sw = (off & 15u) >> 2;
  const uint4 *base = (const uint4 *)(c.slot_data + (u64)slot * c.slot_bytes + (off & ~15u));
  const uint4 *q4 = (const uint4 *)((const u8 *)c.queries + (u64)qid * c.vec_bytes);
  const u32 ncha = nchunk + (sw ? 1u : 0u);                  // aligned chunks that hold the vector
  const bool s2 = (sw & 2u) != 0u, s1 = (sw & 1u) != 0u;
  u32 acc_u = 0;
  float acc_f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  uint4 carry = make_uint4(0, 0, 0, 0);
  for (u32 b0 = 0; b0 < nchunk; b0 += 8) {
    u32 w[36];
    {
      uint4 A[9];
      A[0] = carry;
#pragma unroll
      for (int k = 0; k < 9; ++k) {
        if (k == 0 && b0 != 0) continue;                     // carried over from the previous block
        const u32 a = b0 + (u32)k;
        A[k] = (active && a < ncha) ? __ldcg(base + a) : make_uint4(0, 0, 0, 0);
      }
      carry = A[8];
#pragma unroll
      for (int k = 0; k < 9; ++k) { w[4 * k] = A[k].x; w[4 * k + 1] = A[k].y; w[4 * k + 2] = A[k].z; w[4 * k + 3] = A[k].w; }
    }
#pragma unroll
    for (int i = 0; i < 34; ++i) w[i] = s2 ? w[i + 2] : w[i];
#pragma unroll
    for (int i = 0; i < 32; ++i) w[i] = s1 ? w[i + 1] : w[i];
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      if (b0 + (u32)t < nchunk) {                            // warp-uniform
        const uint4 qv = active ? __ldg(q4 + b0 + t) : make_uint4(0, 0, 0, 0);
        const u32 qq[4] = {qv.x, qv.y, qv.z, qv.w};
        if (c.dtype == 0) {
#pragma unroll
          for (int i = 0; i < 4; ++i) { const u32 x = __vabsdiffu4(w[4 * t + i], qq[i]); acc_u = __dp4a(x, x, acc_u); }
        } else {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float x = __uint_as_float(qq[i]) - __uint_as_float(w[4 * t + i]);
            acc_f[t] = fmaf(x, x, acc_f[t]);
          }
        }
      }
    }
  }
  if (c.dtype == 0) return acc_u;
  return __float_as_uint(((acc_f[0] + acc_f[4]) + (acc_f[2] + acc_f[6])) + ((acc_f[1] + acc_f[5]) + (acc_f[3] + acc_f[7])));
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
  if (c.vec128 && eval_mask) dist = lane_score128(c, (eval_mask >> lane) & 1u, qid, node, slot);
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

}  // namespace gorio
