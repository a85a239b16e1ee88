// The warp-sorted candidate list: bitonic network, list update and frontier selection, the PQ
// rerank pool, neighbour collection.
// Part of the persistent search kernel; included by search_kernels.cu in this order.
#pragma once
#include "../gorio_internal.h"

namespace gorio {

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

// Fold n new keys into the sorted list xl (H keys per lane, ascending, padded beyond len; the list
// never holds more than L <= 32*H keys).  A chunk of new keys is sorted on its own, descending, so
// that list ++ chunk is bitonic; one compare-exchange stage then leaves the 32*H smallest of both
// in xl (everything else could not stay in the list anyway and is dropped on the spot), and one
// merge pass over H registers re-sorts them.  The chunk's sorting network is picked by its size
// (32, 64 or 32*H keys): after the first few iterations only a handful of new keys beat the
// list's worst, and callers pass only those.  GLOBAL: the keys are read with L2 loads from
// global memory instead of plain loads (shared memory).
template <int H, bool GLOBAL>
__device__ __forceinline__ void list_insert(u64 (&xl)[H], u32 &len, const u64 *keys, u32 n, u32 L, u32 lane) {
  for (u32 done = 0; done < n;) {
    const u32 take = min(32u * (u32)H, n - done);
    const u64 *src = keys + done;
    u64 y[H];
    if (H > 1 && take <= 32u) {
      u64 t[1];
      t[0] = lane < take ? (GLOBAL ? ld_u64(src + lane) : src[lane]) : kPadKey;
      bitonic_sort<1>(t, lane, 2, true);
#pragma unroll
      for (int r = 0; r < H; ++r) y[r] = r == H - 1 ? t[0] : kPadKey;
    } else if (H > 2 && take <= 64u) {
      u64 t[2];
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const u32 e = (u32)r * 32u + lane;
        t[r] = e < take ? (GLOBAL ? ld_u64(src + e) : src[e]) : kPadKey;
      }
      bitonic_sort<2>(t, lane, 2, true);
#pragma unroll
      for (int r = 0; r < H; ++r) y[r] = r == H - 2 ? t[0] : (r == H - 1 ? t[1] : kPadKey);
    } else {
#pragma unroll
      for (int r = 0; r < H; ++r) {
        const u32 e = (u32)r * 32u + lane;
        y[r] = e < take ? (GLOBAL ? ld_u64(src + e) : src[e]) : kPadKey;
      }
      bitonic_sort<H>(y, lane, 2, true);
    }
#pragma unroll
    for (int r = 0; r < H; ++r) xl[r] = xl[r] < y[r] ? xl[r] : y[r];
    bitonic_sort<H>(xl, lane, 32u * (u32)H);
    len = min(L, len + take);
    done += take;
#pragma unroll
    for (int r = 0; r < H; ++r) {
      const u32 e = (u32)r * 32u + lane;
      if (e >= len) xl[r] = kPadKey;
    }
  }
}

// The list's L-th key once it is full (what a new key has to beat, with the expanded bit set so
// that the comparison ignores that bit), all ones before.
template <int H>
__device__ __forceinline__ u64 list_worst(const u64 (&xl)[H], u32 len, u32 L, u32 lane) {
  const u32 wi = L - 1u;
  u64 worst = kPadKey;
#pragma unroll
  for (int r = 0; r < H; ++r)
    if ((u32)r == wi / 32u) worst = __shfl_sync(0xffffffffu, xl[r], wi % 32u);
  return len == L ? (worst | 1ull) : kPadKey;
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
// H: list keys per lane (L <= 32*H).  wk: this warp's candidate area in shared memory (WR keys):
// only candidates that beat the list's worst key are gathered there and sorted.
template <int H>
__device__ __noinline__ u32 merge_select(const Ctx &c, u32 qs, u32 lane, u64 *wk) {
  QHdr *h = c.hdr + qs;
  u32 len = uld(&h->list_len);
  const u32 nc = uld(&h->n_items);
  u64 *list = c.list + (u64)qs * c.L;
  const u64 *cand = c.cand + (u64)qs * c.WR;
  const u32 lt = (1u << lane) - 1u;
  u64 xl[H];
#pragma unroll
  for (int r = 0; r < H; ++r) {
    const u32 e = (u32)r * 32u + lane;
    xl[r] = e < len ? ld_u64(list + e) : kPadKey;
  }
  const u64 worst = list_worst<H>(xl, len, c.L, lane);
  u32 kept = 0;
  for (u32 base = 0; base < nc; base += 128u) {          // four loads per lane in flight
    u64 key[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const u32 i = base + 32u * (u32)k + lane;
      key[k] = i < nc ? ld_u64(cand + i) : kPadKey;
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const bool keep = key[k] < worst;
      const u32 b = __ballot_sync(0xffffffffu, keep);
      if (keep) wk[kept + __popc(b & lt)] = key[k];
      kept += __popc(b);
    }
  }
  __syncwarp();
  list_insert<H, false>(xl, len, wk, kept, c.L, lane);
  __syncwarp();
  // frontier
  u32 taken = 0;
  u32 *items = c.items + (u64)qs * c.WR;
#pragma unroll
  for (int r = 0; r < H; ++r) {
    const u32 e = (u32)r * 32u + lane;
    const bool un = e < len && !(xl[r] & 1ull);
    const u32 b = __ballot_sync(0xffffffffu, un);
    if (taken < c.W && b) {
      const u32 rank = taken + __popc(b & lt);
      if (un && rank < c.W) { xl[r] |= 1ull; st_u32(items + rank, key_id(xl[r])); }
      taken = min(c.W, taken + (u32)__popc(b));
    }
  }
#pragma unroll
  for (int r = 0; r < H; ++r) {
    const u32 e = (u32)r * 32u + lane;
    if (e < len) st_u64(list + e, xl[r]);
  }
  if (lane == 0) st_u32(&h->list_len, len);
  {   // the L-th key once the list is full: what a new candidate has to beat
    const u64 w2 = list_worst<H>(xl, len, c.L, lane);
    if (lane == 0) st_u64((u64 *)&h->worst_lo, w2);
  }
  if (taken == 0 && c.pq_m == 0) {
    const u32 qid = uld(&h->qid);
#pragma unroll
    for (int r = 0; r < H; ++r) {
      const u32 e = (u32)r * 32u + lane;
      if (e < c.K) write_result(c, qid, e, xl[r], e < len);
    }
  }
  return taken;
}

__device__ u32 merge_select_dispatch(const Ctx &c, u32 qs, u32 lane, u64 *wk) {
  if (c.L <= 32) return merge_select<1>(c, qs, lane, wk);
  if (c.L <= 64) return merge_select<2>(c, qs, lane, wk);
  if (c.L <= 128) return merge_select<4>(c, qs, lane, wk);
  return merge_select<8>(c, qs, lane, wk);
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
          u32 r = c.seen_bitmap ? bit_insert(seen, v) : set_insert(seen, c.seen_cap, v);
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

}  // namespace gorio
