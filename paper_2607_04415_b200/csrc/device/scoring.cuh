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

}  // namespace gorio
