// Device side of the GPU-owned paged beam search (sm_100a).
//
// One persistent kernel runs every query of a batch.  Warps are the execution slots: a
// warp pops a runnable query slot from a queue in HBM, advances it by one or more phases,
// and parks it when it has to wait for pages (paper Section 3.3: a search block takes a
// query, runs its traversal, and ends by either completing it or leaving it pending on a page).
//
// Data flow of one query iteration:
//   PH_EVAL  complete -> merge the scored candidates into the sorted L-entry list, pick the
//                        first W unexpanded entries (the frontier), issue their pages
//   PH_EXPAND complete -> read the frontier's adjacency lists, filter through the exact
//                        visited set, issue the pages of the new neighbours (exact mode) or
//                        score them from resident PQ codes (PQ mode)
// "Issuing" a batch of page items means, per item: look the page up in the cache; on a hit
// consume it now; if the page is in flight register as a waiter; if it is absent claim a
// slot (clock eviction), post a request descriptor (the poster warp forwards it to the
// host-visible ring) and register.
// Requests the host proxy has admitted are pulled from the pinned store by the puller warps (the
// last warp of every block), in ring order; the proxy publishes each completion once the page's
// bytes are on the GPU and the injected latency has passed.
// A page that arrives is consumed for every registered waiter by whichever warp picks the
// arrival up, using only the waiter's query vector, so no page stays pinned for a query.
// The last item consumed of a batch pushes the query back onto the runnable queue.
#include "gorio_internal.h"

#include "device/mem.cuh"
#include "device/queue.cuh"
#include "device/page_cache.cuh"
#include "device/scoring.cuh"
#include "device/arrival.cuh"
#include "device/batch.cuh"
#include "device/list.cuh"
#include "device/pq.cuh"
#include "device/scheduler.cuh"
#include "device/resident.cuh"

namespace gorio {

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
    ctl->counts[0] = 0; ctl->counts[1] = 0; c.cs->copy_head = 0; c.cs->comp_head = 0; c.cs->in_flight = 0; ctl->adm_seen = 0;
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
// Link probe: what the host link delivers to the access pattern of copy_page and nothing else.
// Every warp pulls whole 4 KB pages of the pinned store into a 4 KB area of its own in HBM, one
// page at a time with all of the page's loads in flight (exactly copy_page's loads), pull i going
// to page hash(i) mod n_pages (or page i mod n_pages when `sequential`).  The number of warps is
// the number of pages in flight.  No cache, no proxy, no queries.
__global__ void __launch_bounds__(128) link_probe_kernel(const u8 *host_pages, u32 n_pages, u32 n_pulls, u32 sequential,
                                                         u8 *scratch, u32 *next, u32 *sink) {
  const u32 lane = threadIdx.x & 31u;
  const u32 warp = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  uint4 *dst = (uint4 *)(scratch + (u64)warp * kPageBytes);
  u32 acc = 0;
  for (;;) {
    u32 i = 0;
    if (lane == 0) i = atomicAdd(next, 1u);
    i = __shfl_sync(0xffffffffu, i, 0);
    if (i >= n_pulls) break;
    const u32 page = (sequential ? i : hash32(i)) % n_pages;
    const uint4 *src = (const uint4 *)(host_pages + (u64)page * kPageBytes);
    uint4 v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = __ldcs(src + k * 32 + lane);
#pragma unroll
    for (int k = 0; k < 8; ++k) acc ^= v[k].x ^ v[k].y ^ v[k].z ^ v[k].w;
#pragma unroll
    for (int k = 0; k < 8; ++k) __stcg(dst + k * 32 + lane, v[k]);
  }
  acc = __reduce_xor_sync(0xffffffffu, acc);
  if (lane == 0) atomicXor(sink, acc);
}

cudaError_t launch_link_probe(const u8 *host_pages, u32 n_pages, u32 n_pulls, u32 warps, u32 sequential, u8 *scratch,
                              u32 *next, u32 *sink, cudaStream_t s) {
  link_probe_kernel<<<(warps + 3) / 4, 128, 0, s>>>(host_pages, n_pages, n_pulls, sequential, scratch, next, sink);
  return cudaGetLastError();
}

// With lazy module loading the first launch of a kernel may need a context-wide
// synchronisation; querying the attributes loads all code at open time instead, so that no
// launch ever has to wait behind a resident persistent kernel.
cudaError_t preload_kernels() {
  cudaFuncAttributes a;
  cudaError_t e;
  if ((e = cudaFuncGetAttributes(&a, search_kernel<false, 512>)) != cudaSuccess) return e;
  if ((e = cudaFuncGetAttributes(&a, search_kernel<false, 768>)) != cudaSuccess) return e;
  if ((e = cudaFuncGetAttributes(&a, search_kernel<true, 384>)) != cudaSuccess) return e;
  if ((e = cudaFuncGetAttributes(&a, init_kernel)) != cudaSuccess) return e;
  if ((e = cudaFuncGetAttributes(&a, link_probe_kernel)) != cudaSuccess) return e;
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

// Dynamic shared memory per warp: the PQ distance table and the warp's candidate area.
size_t search_smem_per_warp(const Ctx &c) {
  return (c.pq_m ? (size_t)c.pq_m * kPqLutWords * 4 : 0) + (size_t)resident_warp_words(c.WR) * 4;
}

template <typename K>
static cudaError_t occupancy_of(K kernel, u32 threads, size_t smem, int *blocks_per_sm) {
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, kernel, threads, smem);
}

cudaError_t search_occupancy(const Ctx &c, u32 warps_per_block, int *blocks_per_sm) {
  const size_t smem = search_smem_per_warp(c) * warps_per_block;
  if (c.pq_m) return occupancy_of(search_kernel<true, 384>, warps_per_block * 32, smem, blocks_per_sm);
  if (warps_per_block <= 16) return occupancy_of(search_kernel<false, 512>, warps_per_block * 32, smem, blocks_per_sm);
  return occupancy_of(search_kernel<false, 768>, warps_per_block * 32, smem, blocks_per_sm);
}

cudaError_t launch_search(const Ctx &c, u32 blocks, u32 warps_per_block, cudaStream_t s) {
  const size_t smem = search_smem_per_warp(c) * warps_per_block;
  cudaError_t e;
  if (c.pq_m) {
    if ((e = cudaFuncSetAttribute(search_kernel<true, 384>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    search_kernel<true, 384><<<blocks, warps_per_block * 32, smem, s>>>(c);
  } else if (warps_per_block <= 16) {
    if ((e = cudaFuncSetAttribute(search_kernel<false, 512>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    search_kernel<false, 512><<<blocks, warps_per_block * 32, smem, s>>>(c);
  } else {
    if ((e = cudaFuncSetAttribute(search_kernel<false, 768>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    search_kernel<false, 768><<<blocks, warps_per_block * 32, smem, s>>>(c);
  }
  return cudaGetLastError();
}

}  // namespace gorio
