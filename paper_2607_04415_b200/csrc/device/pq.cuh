// PQ navigation: the per-query distance table in shared memory and asymmetric distances.
// Part of the persistent search kernel; included by search_kernels.cu in this order.
#pragma once
#include "../gorio_internal.h"

namespace gorio {

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
// One node per lane: the lane reads the node's code (pq_m bytes) and sums pq_m independent table
// entries from shared memory -- no cross-lane reduction, 32 nodes per pass.  The code is read in
// 16-byte chunks, the next chunk's load issued before the current one is looked up, so a 32-byte
// code costs one round trip to L2/HBM, not one per word; the loop body (16 lookups) is kept
// rolled to stay small in the instruction cache.
__device__ __forceinline__ u32 adc_word(const u16 *lo, const u32 *hi, u32 sub0, u32 cw) {
  return lut_get(lo, hi, ((sub0 + 0u) << 8) + (cw & 255u)) + lut_get(lo, hi, ((sub0 + 1u) << 8) + ((cw >> 8) & 255u)) +
         lut_get(lo, hi, ((sub0 + 2u) << 8) + ((cw >> 16) & 255u)) + lut_get(lo, hi, ((sub0 + 3u) << 8) + (cw >> 24));
}
__device__ __forceinline__ u32 lane_adc(const Ctx &c, const u32 *lut, u32 v) {
  const u8 *code = c.pq_codes + (u64)v * c.pq_m;
  const u16 *lo = (const u16 *)lut;
  const u32 *hi = lut_hi(c, lut);
  u32 acc = 0;
  if ((c.pq_m & 15u) == 0u && ((uintptr_t)c.pq_codes & 15u) == 0u) {
    const uint4 *c4 = (const uint4 *)code;
    const u32 nch = c.pq_m >> 4;
    uint4 cur = __ldg(c4);
#pragma unroll 1
    for (u32 ch = 0; ch < nch; ++ch) {
      uint4 nxt = cur;
      if (ch + 1u < nch) nxt = __ldg(c4 + ch + 1u);
      acc += adc_word(lo, hi, 16u * ch, cur.x) + adc_word(lo, hi, 16u * ch + 4u, cur.y) +
             adc_word(lo, hi, 16u * ch + 8u, cur.z) + adc_word(lo, hi, 16u * ch + 12u, cur.w);
      cur = nxt;
    }
  } else {
    for (u32 w = 0; w < (c.pq_m >> 2); ++w) acc += adc_word(lo, hi, 4u * w, __ldg((const u32 *)code + w));
  }
  return acc;
}

}  // namespace gorio
