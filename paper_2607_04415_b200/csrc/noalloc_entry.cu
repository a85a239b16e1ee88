// gorio_search_resident_noalloc: the beam search for callers that must not allocate.
//
// Some callers cannot call cudaMalloc at the point where they need a search: code running
// inside a memory-pool-managed service where every byte is accounted to a pre-sized arena,
// real-time loops where the allocator's implicit device synchronisation is unacceptable, or
// plugins loaded into a host process that forbids allocations after start-up.  For them this
// entry point runs the same persistent search kernel over an index that is already resident
// in device memory, with all of its working state (query slots, visited sets, queues, page
// table) carved out of one fixed file-scope device array instead of cudaMalloc'd buffers.
//
// The array lives in every CUDA context that loads this library, for the life of the
// process (kNoallocScratchBytes per GPU).  Calls share it and it keeps the previous call's
// contents, so everything that must start clean is re-initialised at the top of each call,
// and two calls whose kernels overlap on the same GPU would corrupt each other: the caller
// must serialise them (the call itself blocks until its kernel has finished).
#include <cstdio>
#include <cstring>
#include <mutex>

#include "../../include/gorio.h"
#include "gorio_internal.h"

using namespace gorio;

namespace gorio { void set_global_error(const char *msg); }

namespace {

constexpr size_t kNoallocScratchBytes = 12u << 20;      // 12 MiB per GPU
constexpr u32 kNaMaxPages = 32768;                      // 128 MiB of index pages
constexpr u32 kNaSlots = 64;                            // queries in flight (slots are recycled)
constexpr u32 kNaMaxWR = 256;                           // W * max_degree
constexpr u32 kNaMaxL = 256;
constexpr u32 kNaMaxW = 16;
constexpr u32 kNaVisited = 16384;                       // per-query visited / page set entries
constexpr u32 kNaRing = 256;                            // dummy proxy rings (never written)

// In host code this name is only a handle for cudaGetSymbolAddress; it is not an address the
// device can use.  Device code may name it directly.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoallocScratchBytes];

constexpr int kMaxDevices = 64;
unsigned char *g_scratch_dev[kMaxDevices] = {};         // device address of the array, per GPU
int g_sm_count[kMaxDevices] = {};
std::mutex g_setup_mu;

struct Carver {
  unsigned char *base;
  size_t off = 0;
  template <typename T>
  T *take(size_t count) {
    off = (off + 255) & ~(size_t)255;
    T *p = (T *)(base + off);
    off += count * sizeof(T);
    return p;
  }
};

int na_fail(int status, const char *msg) {
  gorio::set_global_error(msg);
  return status;
}

}  // namespace

extern "C" int gorio_search_resident_noalloc(const gorio_index_desc *d, const void *pages_dev,
                                             const void *queries_dev, uint32_t nq, uint32_t K, uint32_t L,
                                             uint32_t W, uint32_t *out_ids_dev, void *out_dists_dev,
                                             uint32_t *out_pages_distinct_dev, void *cuda_stream) {
  if (!d || !pages_dev || !queries_dev || !out_ids_dev || !out_dists_dev || nq < 1)
    return na_fail(GORIO_ERR_INVALID_ARG, "noalloc search: null argument or nq == 0");
  const u32 esz = d->dtype == GORIO_DTYPE_U8 ? 1u : 4u;
  const u64 nb = (u64)d->dim * esz + 4 + 4ull * d->max_degree;
  if (d->dtype > GORIO_DTYPE_F32 || d->page_bytes != kPageBytes || d->dim == 0 || d->dim % 4 != 0 ||
      d->max_degree == 0 || d->nodes_per_page == 0 || nb * d->nodes_per_page > kPageBytes || d->n_nodes == 0 ||
      d->n_nodes >= (1ull << 31) || d->entry_id >= d->n_nodes)
    return na_fail(GORIO_ERR_INVALID_ARG, "noalloc search: bad index description");
  // the kernels read and write 32-bit words through these pointers: a misaligned one would trap
  if ((((uintptr_t)pages_dev | (uintptr_t)queries_dev | (uintptr_t)out_ids_dev | (uintptr_t)out_dists_dev |
        (uintptr_t)out_pages_distinct_dev) & 3u) != 0)
    return na_fail(GORIO_ERR_INVALID_ARG, "noalloc search: pages, queries and outputs must be at least 4-byte aligned");
  if (d->pq_m != 0) return na_fail(GORIO_ERR_INVALID_ARG, "noalloc search: PQ navigation is not supported here");
  const u64 n_pages = (d->n_nodes + d->nodes_per_page - 1) / d->nodes_per_page;
  if (n_pages > kNaMaxPages)
    return na_fail(GORIO_ERR_INVALID_ARG, "noalloc search: index exceeds the fixed scratch (at most 32768 pages)");
  if (K < 1 || K > L || L > kNaMaxL || W < 1 || W > kNaMaxW || (u64)W * d->max_degree > kNaMaxWR)
    return na_fail(GORIO_ERR_INVALID_ARG, "noalloc search: need 1 <= K <= L <= 256, W <= 16, W*max_degree <= 256");

  // One-time set-up per device: resolve the device address of the scratch array.
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) return na_fail(GORIO_ERR_CUDA, "noalloc search: cudaGetDevice failed");
  {
    std::lock_guard<std::mutex> lk(g_setup_mu);
    if (!g_scratch_dev[dev]) {
      void *p = nullptr;
      e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
      if (e != cudaSuccess || !p) return na_fail(GORIO_ERR_CUDA, "noalloc search: cudaGetSymbolAddress failed");
      int sms = 0;
      e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess || sms < 1) return na_fail(GORIO_ERR_CUDA, "noalloc search: cannot read the SM count");
      if (preload_kernels() != cudaSuccess) return na_fail(GORIO_ERR_CUDA, "noalloc search: kernels failed to load");
      g_sm_count[dev] = sms;
      g_scratch_dev[dev] = (unsigned char *)p;
    }
  }
  cudaStream_t stream = (cudaStream_t)cuda_stream;

  // Carve the working state out of the scratch array.
  const u32 R = d->max_degree, WR = W * R;
  const u32 slots = nq < kNaSlots ? nq : kNaSlots;
  Carver cv{g_scratch_dev[dev]};
  Ctx c{};
  c.n_nodes = (u32)d->n_nodes; c.dim = d->dim; c.dtype = d->dtype; c.R = R; c.npp = d->nodes_per_page;
  c.node_bytes = (u32)nb; c.vec_bytes = d->dim * esz; c.entry = d->entry_id; c.n_pages = (u32)n_pages;
  c.slot_data = (u8 *)const_cast<void *>(pages_dev);      // every page is resident: slot p holds page p
  c.n_slots = (u32)n_pages; c.n_units = (u32)n_pages; c.slot_bytes = kPageBytes; c.record_mode = 0;
  c.ctl = cv.take<Ctl>(1);
  c.cs = cv.take<CacheShared>(1);
  c.ptab = cv.take<u64>(n_pages); c.smeta = cv.take<u64>(n_pages);
  c.parts = cv.take<u32>(n_pages); c.filled = cv.take<u32>(n_pages);
  // proxy words that nothing ever writes: the poller reads zeros (device memory) and idles
  u32 *dummy = cv.take<u32>(64);
  c.host_ctl = dummy;
  c.ring = cv.take<u64>(kNaRing); c.ring_mask = kNaRing - 1; c.ring_shift = 8;
  c.ring_dev = cv.take<u64>(kNaRing); c.fdone = cv.take<u32>(kNaRing);
  c.host_pages = (const u8 *)pages_dev;
  const u32 runq = 2 * kNaSlots, arrq = 1024, smallq = 256;
  u32 *qh = c.ctl->q_heads;
  int *cnt = c.ctl->counts;
  c.arr = Queue{(u32 *)cv.take<u64>(arrq), arrq - 1, qh + 0, qh + 1, cnt + 2};
  c.run = Queue{(u32 *)cv.take<u64>(runq), runq - 1, qh + 3, qh + 4, cnt + 3};
  c.want = Queue{(u32 *)cv.take<u64>(smallq), smallq - 1, qh + 6, qh + 7, cnt + 4};
  c.n_qslots = slots; c.nq = nq; c.K = K; c.L = L; c.W = W; c.WR = WR;
  c.hdr = cv.take<QHdr>(slots);
  c.list = cv.take<u64>((size_t)slots * L); c.cand = cv.take<u64>((size_t)slots * WR);
  c.items = cv.take<u32>((size_t)slots * WR); c.wrec = cv.take<u32>((size_t)slots * WR);
  c.adj = cv.take<u32>((size_t)slots * WR); c.adjdeg = cv.take<u32>((size_t)slots * W);
  c.pool = nullptr;
  c.seen_cap = kNaVisited; c.pset_cap = kNaVisited;
  c.stash = nullptr; c.stash_tag = nullptr; c.stash_cap = 0;    // everything is resident: no stash needed
  c.seen = cv.take<u32>((size_t)slots * kNaVisited); c.pset = cv.take<u32>((size_t)slots * kNaVisited);
  if (cv.off > kNoallocScratchBytes) return na_fail(GORIO_ERR_INTERNAL, "noalloc search: scratch layout exceeds the array");
  c.queries = queries_dev; c.out_ids = out_ids_dev; c.out_dists = out_dists_dev;
  c.out_pages = out_pages_distinct_dev; c.out_counters = nullptr;
  c.timeout_ns = 60ull * 1000000000ull;
  c.census_ns = 0;
  c.max_iters = 64u * L + 1024u;
  c.blocking = 0;
  c.identity = 1;           // every page is resident in the slot of its own number
  c.resident_fast = 1;      // ... so every query runs start to end on the warp that takes it
  c.max_in_flight = 1u << 30;
  c.idle_ns = 8000;
  c.pullers = 0;
  c.vec128 = (c.vec_bytes % 16 == 0 && c.vec_bytes <= 384 && ((uintptr_t)queries_dev & 15) == 0 &&
              ((uintptr_t)pages_dev & 15) == 0) ? 1u : 0u;

  // The array keeps the previous call's contents: reset everything that must start clean.
  const size_t ring_bytes = (size_t)((unsigned char *)(c.fdone + kNaRing) - (unsigned char *)dummy);
  if ((e = cudaMemsetAsync(c.ctl, 0, sizeof(Ctl), stream)) != cudaSuccess ||
      (e = cudaMemsetAsync(dummy, 0, ring_bytes, stream)) != cudaSuccess ||
      (e = cudaMemsetAsync(c.seen, 0xFF, (size_t)slots * kNaVisited * 4, stream)) != cudaSuccess ||
      (e = cudaMemsetAsync(c.pset, 0xFF, (size_t)slots * kNaVisited * 4, stream)) != cudaSuccess ||
      (e = launch_cache_reset(c, (u32)n_pages, stream)) != cudaSuccess ||     // every page RESIDENT in slot = page
      (e = launch_init(c, stream)) != cudaSuccess ||
      (e = launch_search(c, (u32)g_sm_count[dev], 16, stream)) != cudaSuccess)
    return na_fail(GORIO_ERR_CUDA, cudaGetErrorString(e));
  Ctl h;
  if ((e = cudaMemcpyAsync(&h, c.ctl, sizeof(Ctl), cudaMemcpyDeviceToHost, stream)) != cudaSuccess ||
      (e = cudaStreamSynchronize(stream)) != cudaSuccess)
    return na_fail(GORIO_ERR_CUDA, cudaGetErrorString(e));
  if (h.status != 0 || h.stop != 1) {
    char buf[160];
    const u32 s = h.status ? h.status : (u32)GORIO_ERR_INTERNAL;
    std::snprintf(buf, sizeof buf, "noalloc search: device status %u (site 0x%x, %u, %u); done %u/%u%s", s, h.dbg[0],
                  h.dbg[1], h.dbg[2], h.done, nq,
                  s == GORIO_ERR_CAPACITY ? "; a query visited more nodes than the fixed per-query set holds" : "");
    return na_fail((int)s, buf);
  }
  return GORIO_OK;
}
