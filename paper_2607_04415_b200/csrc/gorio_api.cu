// Host side of the C ABI declared in include/gorio.h: resource management, the blocking
// search call, and the CPU proxy thread that services page requests from the emulated
// remote tier (paper Section 3.3: the proxy groups submissions and completions, bounds the
// remote reads in flight and makes arrivals visible to the GPU; it never looks at search state).
#include <atomic>
#if defined(__x86_64__) || defined(__i386__)
#include <immintrin.h>
#endif
#include <chrono>
#include <condition_variable>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <deque>
#include <mutex>
#include <new>
#include <string>
#include <thread>
#include <vector>

#include "../../include/gorio.h"
#include "gorio_internal.h"

using namespace gorio;

namespace {

typedef std::chrono::steady_clock Clock;

inline u32 next_pow2(u64 v) { u32 p = 1; while (p < v) p <<= 1; return p; }
inline u32 ilog2(u32 v) { u32 s = 0; while ((1u << s) < v) ++s; return s; }

enum ProxyState : int { PX_IDLE = 0, PX_RUN = 1, PX_EXIT = 2 };
constexpr int kFillStreams = 4;
constexpr int kFillEvents = 256;
constexpr u32 kFillBatch = 32;      // most copies the proxy issues before it looks at completions again

}  // namespace

struct gorio_index {
  gorio_index_desc desc{};
  int dev = 0;
  int n_sms = 0;
  u32 n_pages = 0, node_bytes = 0, vec_bytes = 0;
  bool registered_pages = false;
  const u8 *pages_dev = nullptr;   // device view of the host page store

  // cache
  gorio_cache_cfg cfg{};
  bool cache_ready = false, cache_dirty = false;
  u32 n_slots = 0, preloaded = 0;
  u32 n_units = 0, slot_bytes = kPageBytes, record_mode = 0;   // cache unit: page, or node record
  u8 *slot_data = nullptr;
  u64 *ptab = nullptr, *smeta = nullptr;
  u32 *parts = nullptr, *filled = nullptr;
  CacheShared *cs = nullptr;
  u64 *want_buf = nullptr; u32 want_cap = 0;
  u64 *ring_copy = nullptr;
  // host-mapped communication areas
  u64 *ring_h = nullptr; u64 *ring_d = nullptr; u32 ring_cap = 0;
  u32 *hctl_h = nullptr; u32 *hctl_d = nullptr;     // [0] completions published, [1] abort, [2] requests admitted
  u32 *fdone_h = nullptr; u32 *fdone_d = nullptr;   // copy acknowledgements, GPU -> proxy
  u64 *arr_buf = nullptr; u32 arr_cap = 0;

  // query state
  gorio_tuning tune{};
  u32 qs_slots = 0, qs_L = 0, qs_W = 0, qs_WR = 0, qs_K = 0, qs_seen = 0, qs_pset = 0, qs_stash = 0, qs_nslots = 0, qs_units = 0;
  void *qs_block = nullptr;
  Ctx ctx{};
  Ctl *ctl = nullptr;
  u64 *run_buf = nullptr; u32 runq_cap = 0;

  // host-buffer search staging
  void *st_q = nullptr; size_t st_q_bytes = 0;
  void *st_out = nullptr; size_t st_out_bytes = 0;

  std::recursive_mutex api_mu;   // calls on one index are serialised (search_host calls search)

  // proxy
  std::thread proxy;
  std::mutex mu;
  std::condition_variable cv;
  std::atomic<int> px_state{PX_IDLE};
  std::atomic<int> px_stop{0};
  std::atomic<int> px_error{0};
  cudaStream_t own_stream = nullptr;
  cudaEvent_t done_ev = nullptr;
  // copy-engine mode of the proxy: streams the proxy issues its page copies on, and a ring of
  // events through which it learns that a batch of copies has landed
  cudaStream_t fill_streams[kFillStreams] = {};
  cudaEvent_t fill_events[kFillEvents] = {};

  // statistics
  u64 host_fetched_bytes = 0;
  u64 host_fetched = 0, host_max_out = 0, host_batches = 0, host_search_ns = 0;
  u64 host_service_ns = 0, host_ack_wait = 0, host_window_full = 0, host_ring_empty = 0, host_iters = 0, host_out_sum = 0;
  u32 px_dbg[8] = {};   // proxy progress at the end of its last service loop
  std::string err;
};

namespace {

int fail(gorio_index *ix, int status, const std::string &msg) {
  if (ix) ix->err = msg;
  return status;
}
int cuda_fail(gorio_index *ix, cudaError_t e, const char *what) {
  return fail(ix, e == cudaErrorMemoryAllocation ? GORIO_ERR_NOMEM : GORIO_ERR_CUDA,
              std::string(what) + ": " + cudaGetErrorString(e));
}
#define CK(call)                                                         \
  do {                                                                   \
    cudaError_t e__ = (call);                                            \
    if (e__ != cudaSuccess) return cuda_fail(ix, e__, #call);            \
  } while (0)

// Flush the CPU's write-combining buffers (the control block the GPU polls is write-combined
// memory: written by the proxy, never read by it, and read over PCIe without a cache snoop).
inline void flush_wc() {
#if defined(__x86_64__) || defined(__i386__)
  _mm_sfence();
#else
  std::atomic_thread_fence(std::memory_order_seq_cst);
#endif
}

template <typename T>
cudaError_t host_mapped(T **h, T **d, size_t count, unsigned extra_flags = 0) {
  void *p = nullptr;
  cudaError_t e = cudaHostAlloc(&p, count * sizeof(T), cudaHostAllocMapped | cudaHostAllocPortable | extra_flags);
  if (e != cudaSuccess) return e;
  std::memset(p, 0, count * sizeof(T));
  *h = (T *)p;
  void *dp = nullptr;
  e = cudaHostGetDevicePointer(&dp, p, 0);
  *d = (T *)dp;
  return e;
}

void free_cache(gorio_index *ix) {
  cudaFree(ix->slot_data); cudaFree(ix->ptab); cudaFree(ix->smeta); cudaFree(ix->parts); cudaFree(ix->filled); cudaFree(ix->cs);
  cudaFree(ix->want_buf); cudaFree(ix->ring_copy);
  ix->ring_copy = nullptr;
  if (ix->ring_h) cudaFreeHost(ix->ring_h);
  if (ix->fdone_h) cudaFreeHost(ix->fdone_h);
  ix->fdone_h = ix->fdone_d = nullptr;
  ix->slot_data = nullptr; ix->ptab = ix->smeta = nullptr; ix->parts = ix->filled = nullptr; ix->cs = nullptr;
  ix->want_buf = nullptr;
  ix->ring_h = ix->ring_d = nullptr;
  ix->cache_ready = false;
}

void free_qstate(gorio_index *ix) {
  cudaFree(ix->qs_block); cudaFree(ix->run_buf); cudaFree(ix->arr_buf);
  ix->qs_block = nullptr; ix->run_buf = ix->arr_buf = nullptr; ix->qs_slots = 0;
}

// ---------------------------------------------------------------------------------------
// the proxy: consumes request descriptors in order, bounds the number in service, commands
// the copy of each page from pinned host memory into its cache slot, and publishes the
// completion once the copy is acknowledged and no earlier than admission + latency.
// It issues no CUDA calls while a search runs: commands, acknowledgements and completions
// all travel through host-mapped memory.
// ---------------------------------------------------------------------------------------
struct InService { u32 slot; u32 idx; Clock::time_point admitted; u64 ev; };

void proxy_service(gorio_index *ix) {
  const u32 ring_mask = ix->ring_cap - 1, ring_shift = ilog2(ix->ring_cap);
  const u32 max_out = ix->cfg.max_outstanding;
  const auto latency = std::chrono::nanoseconds(ix->cfg.remote_latency_ns);
  volatile u64 *ring = ix->ring_h;
  volatile u32 *hctl = ix->hctl_h;
  volatile u32 *fdone = ix->fdone_h;
  u32 tail = 0, ct = 0, outstanding = 0;
  // copy-engine mode (gorio_cache_cfg.copy_mode): the proxy itself moves each page with one
  // cudaMemcpyAsync from the pinned store into the slot, on a few streams of its own, and learns
  // that a batch has landed by querying an event recorded behind it -- no kernel takes part in a
  // fill, so nothing needs a free block slot next to the persistent kernel.
  const bool dma = ix->cfg.copy_mode == GORIO_COPY_ENGINE;
  u64 ev_head = 0, ev_tail = 0;       // events recorded / events known complete (sequence numbers)
  int fill_k = 0;
  std::deque<InService> inflight;
  u64 fetched = 0, max_seen = 0, batches = 0;
  u64 service_ns = 0, ack_wait_iters = 0, window_full_iters = 0, ring_empty_iters = 0, iters = 0, out_sum = 0;
  // debug aid (with GORIO_CENSUS_MS): fetches published and mean outstanding per 10 ms interval
  const bool trace = std::getenv("GORIO_CENSUS_MS") != nullptr;
  std::vector<u64> tr_fetched, tr_out;
  Clock::time_point tr_next = Clock::now() + std::chrono::milliseconds(10);
  u64 tr_out_sum = 0, tr_iters = 0;

  while (!ix->px_stop.load(std::memory_order_acquire)) {
    ++iters;
    out_sum += outstanding;
    if (trace) {
      tr_out_sum += outstanding; ++tr_iters;
      if ((iters & 63) == 0 && Clock::now() >= tr_next) {
        tr_fetched.push_back(fetched); tr_out.push_back(tr_out_sum / (tr_iters ? tr_iters : 1));
        tr_out_sum = tr_iters = 0; tr_next += std::chrono::milliseconds(10);
      }
    }
    // 1. admit descriptors while the in-service window has room; each becomes a copy command
    u32 admitted = 0;
    const Clock::time_point now0 = Clock::now();
    const bool ev_room = !dma || ev_head - ev_tail < (u64)kFillEvents;
    while (outstanding < max_out && ev_room && (!dma || admitted < kFillBatch)) {
      const u64 e = ring[tail & ring_mask];
      const u32 lap = ((tail >> ring_shift) % 255u) + 1u;
      if ((u32)(e & 0xFFu) != lap) break;
      const u32 page = (u32)(e >> 32), slot = (u32)(e >> 8) & 0xFFFFFFu;
      if (page >= ix->n_units || slot >= ix->n_slots) {
        ix->px_error.store(1);   // a descriptor the GPU could not have produced
        return;
      }
      if (dma) {
        // the page, or at record granularity the 16-byte-aligned span that covers the record
        const u8 *src = (const u8 *)ix->desc.host_pages + (size_t)page * kPageBytes;
        size_t bytes = kPageBytes;
        if (ix->record_mode) {
          const u32 npp = ix->desc.nodes_per_page, off = (page % npp) * ix->node_bytes;
          src = (const u8 *)ix->desc.host_pages + (size_t)(page / npp) * kPageBytes + (off & ~15u);
          bytes = (size_t)(((off & 15u) + ix->node_bytes + 15u) >> 4) * 16u;
        }
        if (cudaMemcpyAsync(ix->slot_data + (size_t)slot * ix->slot_bytes, src, bytes, cudaMemcpyHostToDevice,
                            ix->fill_streams[fill_k]) != cudaSuccess) {
          ix->px_error.store(2);
          return;
        }
      }
      inflight.push_back({slot, tail, now0, ev_head});
      ++tail; ++outstanding; ++admitted;
    }
    if (admitted) {
      if (dma) {
        if (cudaEventRecord(ix->fill_events[ev_head % kFillEvents], ix->fill_streams[fill_k]) != cudaSuccess) {
          ix->px_error.store(2);
          return;
        }
        ++ev_head;
        fill_k = (fill_k + 1) % kFillStreams;
      } else {
        hctl[2] = tail;                           // requests [0, tail) may be copied now
        flush_wc();
      }
      ++batches;
      if (outstanding > max_seen) max_seen = outstanding;
    }
    if (dma) {                                    // which batches have landed (events complete in any order across streams)
      while (ev_tail < ev_head) {
        const cudaError_t qe = cudaEventQuery(ix->fill_events[ev_tail % kFillEvents]);
        if (qe == cudaErrorNotReady) break;
        if (qe != cudaSuccess) { ix->px_error.store(2); return; }
        ++ev_tail;
      }
    }
    if (outstanding >= max_out) {
      if ((u32)(ring[tail & ring_mask] & 0xFFu) == ((tail >> ring_shift) % 255u) + 1u) ++window_full_iters;
    } else {
      ++ring_empty_iters;
    }
    // 2. publish completions in admission order: copy acknowledged and latency elapsed
    if (!inflight.empty()) {
      const Clock::time_point now = Clock::now();
      u32 published = 0;
      while (!inflight.empty()) {
        const InService &r = inflight.front();
        if (now - r.admitted < latency) break;
        if (dma ? r.ev >= ev_tail
                : (fdone[r.idx & ring_mask] & 0xFFu) != ((r.idx >> ring_shift) % 255u) + 1u) { ++ack_wait_iters; break; }
        service_ns += (u64)std::chrono::duration_cast<std::chrono::nanoseconds>(now - r.admitted).count();
        ++ct; ++published;
        inflight.pop_front();
      }
      if (published) {
        hctl[0] = ct;                             // completions [0, ct) are published, in ring order
        flush_wc();
        outstanding -= published;
        fetched += published;
      }
    }
  }
  if (dma)       // nothing of this search may still be in flight when the caller frees or re-creates the cache
    for (int i = 0; i < kFillStreams; ++i) cudaStreamSynchronize(ix->fill_streams[i]);
  if (trace) {
    std::fprintf(stderr, "[gorio proxy] per 10 ms: fetched(k)/mean outstanding:");
    u64 prev = 0;
    for (size_t i = 0; i < tr_fetched.size(); ++i) { std::fprintf(stderr, " %llu/%llu", (unsigned long long)((tr_fetched[i] - prev) / 1000), (unsigned long long)tr_out[i]); prev = tr_fetched[i]; }
    std::fprintf(stderr, "\n");
  }
  ix->px_dbg[0] = tail; ix->px_dbg[1] = ct; ix->px_dbg[2] = outstanding; ix->px_dbg[3] = (u32)inflight.size();
  if (!inflight.empty()) {
    ix->px_dbg[4] = inflight.front().idx;
    ix->px_dbg[5] = fdone[inflight.front().idx & ring_mask];
  }
  ix->host_service_ns += service_ns; ix->host_ack_wait += ack_wait_iters; ix->host_window_full += window_full_iters;
  ix->host_ring_empty += ring_empty_iters; ix->host_iters += iters; ix->host_out_sum += out_sum;
  ix->host_fetched += fetched;
  ix->host_fetched_bytes += fetched * ix->slot_bytes;
  ix->host_batches += batches;
  if (max_seen > ix->host_max_out) ix->host_max_out = max_seen;
}

void proxy_main(gorio_index *ix) {
  cudaSetDevice(ix->dev);
  for (;;) {
    {
      std::unique_lock<std::mutex> lk(ix->mu);
      ix->cv.wait(lk, [&] { return ix->px_state.load() != PX_IDLE; });
    }
    if (ix->px_state.load() == PX_EXIT) return;
    proxy_service(ix);
    {
      std::lock_guard<std::mutex> lk(ix->mu);
      if (ix->px_state.load() != PX_EXIT) ix->px_state.store(PX_IDLE);
    }
    ix->cv.notify_all();
  }
}

void proxy_start(gorio_index *ix) {
  ix->px_stop.store(0);
  ix->px_error.store(0);
  {
    std::lock_guard<std::mutex> lk(ix->mu);
    ix->px_state.store(PX_RUN);
  }
  ix->cv.notify_all();
}

void proxy_stop(gorio_index *ix) {
  ix->px_stop.store(1, std::memory_order_release);
  std::unique_lock<std::mutex> lk(ix->mu);
  ix->cv.wait(lk, [&] { return ix->px_state.load() == PX_IDLE || ix->px_state.load() == PX_EXIT; });
}

// ---------------------------------------------------------------------------------------
int setup_cache(gorio_index *ix) {
  const gorio_cache_cfg &cfg = ix->cfg;
  free_cache(ix);
  u64 cap = cfg.capacity_pages;
  ix->record_mode = cfg.granularity == GORIO_GRAN_RECORD ? 1u : 0u;
  if (ix->record_mode) {
    // selective materialisation: the same bytes of HBM, divided into record-sized slots
    ix->n_units = (u32)ix->desc.n_nodes;
    ix->slot_bytes = (ix->node_bytes + 12u + 15u) & ~15u;
    cap = cap * kPageBytes / ix->slot_bytes;
  } else {
    ix->n_units = ix->n_pages;
    ix->slot_bytes = kPageBytes;
  }
  ix->n_slots = cap >= ix->n_units ? ix->n_units : (u32)cap;
  ix->ring_cap = next_pow2(2ull * ix->n_slots < 1024 ? 1024 : 2ull * ix->n_slots);
  ix->want_cap = next_pow2(ix->n_units < 64 ? 64 : ix->n_units);
  CK(cudaMalloc(&ix->slot_data, (size_t)ix->n_slots * ix->slot_bytes));
  CK(cudaMalloc(&ix->ptab, (size_t)ix->n_units * 8));
  CK(cudaMalloc(&ix->smeta, (size_t)ix->n_slots * 8));
  CK(cudaMalloc(&ix->parts, (size_t)ix->n_slots * 4));
  CK(cudaMalloc(&ix->filled, (size_t)ix->n_slots * 4));
  CK(cudaMalloc(&ix->cs, sizeof(CacheShared)));
  CK(cudaMalloc(&ix->want_buf, (size_t)ix->want_cap * 8));
  CK(cudaMalloc(&ix->ring_copy, (size_t)ix->ring_cap * 8));
  CK(host_mapped(&ix->ring_h, &ix->ring_d, ix->ring_cap));
  CK(host_mapped(&ix->fdone_h, &ix->fdone_d, ix->ring_cap));
  ix->preloaded = 0;
  if (cfg.preload) {
    ix->preloaded = cap >= ix->n_pages ? ix->n_pages : ix->n_slots;
    CK(cudaMemcpy(ix->slot_data, ix->desc.host_pages, (size_t)ix->preloaded * kPageBytes, cudaMemcpyHostToDevice));
  }
  Ctx c{};
  c.ptab = ix->ptab; c.smeta = ix->smeta; c.parts = ix->parts; c.filled = ix->filled; c.cs = ix->cs;
  c.n_slots = ix->n_slots; c.n_pages = ix->n_pages; c.n_units = ix->n_units;
  CK(launch_cache_reset(c, ix->preloaded, ix->own_stream));
  CK(cudaStreamSynchronize(ix->own_stream));
  ix->cache_ready = true;
  ix->cache_dirty = false;
  return GORIO_OK;
}

// slot_cap: most query slots this search can use at once (the worker warps of the resident fast
// path, which run one query each; otherwise no limit beyond max_inflight)
int ensure_qstate(gorio_index *ix, u32 nq, u32 K, u32 L, u32 W, u32 slot_cap) {
  const u32 R = ix->desc.max_degree, WR = W * R;
  u32 max_inflight = ix->tune.max_inflight ? ix->tune.max_inflight : 16384u;
  if (slot_cap && slot_cap < max_inflight) max_inflight = slot_cap;
  const u32 slots = nq < max_inflight ? nq : max_inflight;
  // exact visited set per query: a bitmap over the nodes when that is no larger than the hash set
  // (one atomicOr, no probing, never full), else the hash set (config 5: 10M nodes)
  u32 seen_cap = ix->tune.visited_capacity ? ix->tune.visited_capacity : 32768u;
  const u32 hash_cap = seen_cap;
  const u32 node_words = (u32)(((ix->desc.n_nodes + 31u) / 32u + 3u) & ~(u64)3u);
  const bool seen_bitmap = node_words <= seen_cap;
  if (seen_bitmap) seen_cap = node_words;
  // distinct-page set per query: a bitmap over the index's pages when that is smaller than the
  // hash set (config 3: 100,000 pages = 12.5 KB instead of 128 KB per query), else the hash set
  u32 pset_cap = ix->desc.pq_m ? 4096u : hash_cap;
  const u32 bitmap_words = ((ix->n_pages + 31u) / 32u + 3u) & ~3u;
  const bool pset_bitmap = bitmap_words <= pset_cap;
  if (pset_bitmap) pset_cap = bitmap_words;
  if (ix->qs_block && ix->qs_slots >= slots && ix->qs_L == L && ix->qs_W == W && ix->qs_K == K &&
      ix->qs_seen == seen_cap && ix->qs_pset == pset_cap && ix->qs_stash == (ix->tune.stash_entries + 1u) &&
      ix->qs_nslots == ix->n_slots && ix->qs_units == ix->n_units) {      // (the arrival queue and the stash default depend on the slot count)
    ix->ctx.n_qslots = slots;
    return GORIO_OK;
  }
  free_qstate(ix);
  auto al = [](size_t v) { return (v + 255) & ~(size_t)255; };
  size_t off = 0;
  const size_t o_hdr = off;  off += al((size_t)slots * sizeof(QHdr));
  const size_t o_list = off; off += al((size_t)slots * L * 8);
  const size_t o_cand = off; off += al((size_t)slots * WR * 8);
  const size_t o_items = off; off += al((size_t)slots * WR * 4);
  const size_t o_wrec = off; off += al((size_t)slots * WR * 4);
  const size_t o_adj = off;  off += al((size_t)slots * WR * 4);
  const size_t o_adeg = off; off += al((size_t)slots * W * 4);
  const size_t o_pool = off; off += al((size_t)slots * (K + W) * 8);
  const size_t o_seen = off; off += al((size_t)slots * seen_cap * 4);
  const size_t o_pset = off; off += al((size_t)slots * pset_cap * 4);
  // adjacency stash: exact navigation only; by default on (1024 entries) unless every page has
  // a slot of its own, in which case expansions seldom wait for a page and the copies are waste
  u32 stash_cap = ix->tune.stash_entries > 1 ? ix->tune.stash_entries
                  : (ix->tune.stash_entries == 1 || ix->n_slots >= ix->n_units ? 0u : 1024u);
  if (ix->desc.pq_m) stash_cap = 0;
  const size_t o_stag = off; off += al((size_t)slots * stash_cap * 4);
  const size_t o_stash = off; off += al((size_t)slots * stash_cap * (R + 1) * 4);
  CK(cudaMalloc(&ix->qs_block, off));
  ix->runq_cap = next_pow2(2ull * slots < 64 ? 64 : 2ull * slots);
  CK(cudaMalloc(&ix->run_buf, (size_t)ix->runq_cap * 8));
  ix->arr_cap = next_pow2(2ull * ix->n_slots + (u64)slots * WR / 32 + 1024);
  CK(cudaMalloc(&ix->arr_buf, (size_t)ix->arr_cap * 8));
  u8 *b = (u8 *)ix->qs_block;
  Ctx &c = ix->ctx;
  c.hdr = (QHdr *)(b + o_hdr); c.list = (u64 *)(b + o_list); c.cand = (u64 *)(b + o_cand);
  c.items = (u32 *)(b + o_items); c.wrec = (u32 *)(b + o_wrec); c.adj = (u32 *)(b + o_adj);
  c.adjdeg = (u32 *)(b + o_adeg); c.pool = (u64 *)(b + o_pool);
  c.seen = (u32 *)(b + o_seen); c.pset = (u32 *)(b + o_pset);
  c.stash_tag = (u32 *)(b + o_stag); c.stash = (u32 *)(b + o_stash); c.stash_cap = stash_cap;
  c.seen_cap = seen_cap; c.pset_cap = pset_cap; c.pset_bitmap = pset_bitmap ? 1u : 0u; c.seen_bitmap = seen_bitmap ? 1u : 0u; c.n_qslots = slots;
  ix->qs_slots = slots; ix->qs_L = L; ix->qs_W = W; ix->qs_WR = WR; ix->qs_K = K;
  ix->qs_seen = seen_cap; ix->qs_pset = pset_cap; ix->qs_stash = ix->tune.stash_entries + 1u; ix->qs_nslots = ix->n_slots;
  ix->qs_units = ix->n_units;
  return GORIO_OK;
}

thread_local char g_global_error[256] = "";

const char *kDeviceErr[] = {"", "", "", "", "", "device wait expired", "per-query capacity exhausted",
                            "corrupt index page", "internal state-machine check failed"};

// whole index preloaded page by page: slot p holds page p and no request can ever be posted
bool whole_index_resident(const gorio_index *ix) {
  return !ix->record_mode && ix->preloaded == ix->n_units && ix->n_slots == ix->n_units;
}
// ... and the search fits the fast path's fixed shapes (PQ: the rerank pool is one key per lane)
bool resident_fast_path(const gorio_index *ix, u32 K, u32 W) {
  return whole_index_resident(ix) && !ix->tune.no_fast_path && W <= 16u && (ix->desc.pq_m == 0 || K + W <= 32u);
}

// Everything the kernels need for this search, gathered into the by-value context.
void fill_ctx(gorio_index *ix, const void *queries_dev, u32 nq, u32 K, u32 L, u32 W, u32 *out_ids_dev, void *out_dists_dev,
              u32 *out_pages_distinct_dev, u32 *out_counters_dev) {
  const gorio_index_desc &d = ix->desc;
  Ctx &c = ix->ctx;
  c.n_nodes = (u32)d.n_nodes; c.dim = d.dim; c.dtype = d.dtype; c.R = d.max_degree; c.npp = d.nodes_per_page;
  c.node_bytes = ix->node_bytes; c.vec_bytes = ix->vec_bytes; c.entry = d.entry_id; c.n_pages = ix->n_pages;
  c.pq_m = d.pq_m; c.pq_dsub = d.pq_m ? d.dim / d.pq_m : 0; c.pq_cent = d.pq_centroids_dev; c.pq_codes = d.pq_codes_dev;
  c.slot_data = ix->slot_data; c.ptab = ix->ptab; c.smeta = ix->smeta; c.parts = ix->parts; c.filled = ix->filled; c.cs = ix->cs;
  c.n_slots = ix->n_slots; c.n_units = ix->n_units; c.slot_bytes = ix->slot_bytes; c.record_mode = ix->record_mode;
  c.ring = ix->ring_d; c.ring_mask = ix->ring_cap - 1; c.ring_shift = ilog2(ix->ring_cap);
  c.ring_dev = ix->ring_copy; c.host_ctl = ix->hctl_d;
  c.fdone = ix->fdone_d; c.host_pages = ix->pages_dev;
  c.ctl = ix->ctl;
  u32 *qh = ix->ctl->q_heads;
  int *cnt = ix->ctl->counts;
  c.arr = Queue{(u32 *)ix->arr_buf, ix->arr_cap - 1, qh + 0, qh + 1, cnt + 2};
  c.run = Queue{(u32 *)ix->run_buf, ix->runq_cap - 1, qh + 3, qh + 4, cnt + 3};
  c.want = Queue{(u32 *)ix->want_buf, ix->want_cap - 1, qh + 6, qh + 7, cnt + 4};
  c.nq = nq; c.K = K; c.L = L; c.W = W; c.WR = ix->qs_WR;
  c.queries = queries_dev; c.out_ids = out_ids_dev; c.out_dists = out_dists_dev;
  c.out_pages = out_pages_distinct_dev; c.out_counters = out_counters_dev;
  c.timeout_ns = (u64)ix->cfg.timeout_ms * 1000000ull;
  c.max_iters = 64u * L + 1024u;
  c.blocking = ix->tune.blocking ? 1u : 0u;
  c.idle_ns = 8000u;
  { const char *e = std::getenv("GORIO_IDLE_NS"); if (e) c.idle_ns = (u32)std::atoi(e); }      // debug aid
  // default backlog: 4 x the proxy's window, but no more than 1024 (about what keeps the host
  // link busy) unless the window itself is larger
  c.max_in_flight = ix->tune.request_backlog ? ix->tune.request_backlog
                    : (4u * ix->cfg.max_outstanding < 1024u ? 4u * ix->cfg.max_outstanding : 1024u);
  if (c.max_in_flight < ix->cfg.max_outstanding) c.max_in_flight = ix->cfg.max_outstanding;
  c.vec128 = (ix->vec_bytes % 16 == 0 && ix->vec_bytes <= 384 && ((uintptr_t)queries_dev & 15) == 0) ? 1u : 0u;
  { const char *e = std::getenv("GORIO_CENSUS_MS"); c.census_ns = e ? (u64)std::atof(e) * 1000000ull : 0; }
  c.prof = std::getenv("GORIO_PROFILE") ? 1u : 0u;
  // whole index preloaded page by page: slot p holds page p and no request can ever be posted
  c.dma_fill = ix->cfg.copy_mode == GORIO_COPY_ENGINE ? 1u : 0u;
  c.identity = whole_index_resident(ix) ? 1u : 0u;
  c.resident_fast = resident_fast_path(ix, K, W) ? 1u : 0u;
  // who pulls pages (SM pull): one dedicated warp per block, in ring order -- unless nothing is ever
  // pulled (whole index resident, copy-engine fills), the unit is a record (request rates beyond
  // what one warp per SM carries), or the caller asks for the shared scheme
  c.pullers = (!c.dma_fill && !c.identity && !c.record_mode && !ix->tune.shared_pull) ? (u32)ix->n_sms : 0u;     // one per SM, also with two blocks per SM
}

// Launch geometry of the persistent kernel: blocks and warps per block.  Needs only the index, the
// cache and (K, W); runs before the query state is sized.
int launch_geometry(gorio_index *ix, u32 nq, u32 K, u32 W, u32 *blocks_out, u32 *warps_out) {
  const gorio_index_desc &d = ix->desc;
  // launch geometry: one block per SM by default
  const bool pq = d.pq_m != 0;
  Ctx g{};                        // the fields the shared-memory size depends on
  g.pq_m = d.pq_m; g.WR = W * d.max_degree; g.resident_fast = resident_fast_path(ix, K, W) ? 1u : 0u;
  // default warps per SM: 16 when pages will be missed (more warps lengthen every copy and arrival);
  // with every page resident one warp carries one query at a time, so no more than there are
  // queries per SM (fewer idle warps polling the queues), within 8..24
  u32 auto_warps = 16u;
  if (ix->n_slots >= ix->n_units) {
    auto_warps = (nq + (u32)ix->n_sms - 1) / (u32)ix->n_sms;
    auto_warps = auto_warps < 8u ? 8u : (auto_warps > 24u ? 24u : auto_warps);
    if (g.resident_fast && auto_warps > 16u) auto_warps = 16u;     // the fast path wants the 128-register build
  }
  u32 warps = ix->tune.warps_per_block ? ix->tune.warps_per_block : (pq ? 10u : auto_warps);
  const size_t per_warp = search_smem_per_warp(g);
  if (per_warp) {                 // per-warp tables / candidate areas in shared memory (227 KB per block at most)
    u32 lim = (u32)((227u * 1024u) / per_warp);
    if (pq && lim > 12u) lim = 12u;      // the PQ kernel is built for at most 12 warps
    if (warps > lim) warps = lim;
  }
  if (warps < 2) return fail(ix, GORIO_ERR_INVALID_ARG, "search: need at least 2 warps per block (block 0 gives two to the poller and the poster)");
  int occ = 0;
  CK(search_occupancy(g, warps, &occ));
  if (occ < 1) return fail(ix, GORIO_ERR_INVALID_ARG, "search: launch geometry does not fit an SM");
  u32 bps = ix->tune.blocks_per_sm ? ix->tune.blocks_per_sm : 1u;
  if ((int)bps > occ) bps = (u32)occ;
  *blocks_out = (u32)ix->n_sms * bps;
  *warps_out = warps;
  return GORIO_OK;
}

// Debug aids (GORIO_CENSUS_MS, GORIO_PROFILE): print what the kernel recorded.
void print_diagnostics(const Ctx &c, const Ctl &h) {
  if (c.census_ns)
    std::fprintf(stderr, "[gorio census] slots: unused %u, changing owner %u, FILLING %u, ARRIVED %u, RESIDENT ref %u, RESIDENT noref %u | "
                 "pages WANTED %u | queries awaiting %u (items %u) | queues want %d arr %d run %d | done %u posted %u\n",
                 h.census[0], h.census[1], h.census[2], h.census[3], h.census[4], h.census[5], h.census[6], h.census[7],
                 h.census[8], (int)h.census[9], (int)h.census[10], (int)h.census[11], h.census[12], h.census[13]);
  if (c.prof) {
    const char *names[] = {"merge", "issue_eval", "issue_expand", "collect", "pool", "lut", "adc", "finish", "recycle",
                           "(issue: setup", "lookup", "consume", "tail)"};
    std::fprintf(stderr, "[gorio profile] warp ms per query step (cumulative since stats_reset):");
    for (int i = 0; i < 13; ++i) std::fprintf(stderr, " %s %.1f", names[i], h.stats[S_P_MERGE + i] / 1e6);
    std::fprintf(stderr, " | control reads %llu | copies: loads issued -> bytes arrived %.1f",
                 (unsigned long long)h.stats[S_POLLS], h.stats[S_C_DATA] / 1e6);
    std::fprintf(stderr, " | arrival: head %.1f walk %.1f group %.1f complete %.1f finish %.1f", h.stats[S_A_HEAD] / 1e6,
                 h.stats[S_A_WALK] / 1e6, h.stats[S_A_GROUP] / 1e6, h.stats[S_A_COMPLETE] / 1e6, h.stats[S_A_FINISH] / 1e6);
    std::fprintf(stderr, " | arrivals %.1f copies %.1f queries %.1f idle %.1f\n", h.stats[S_T_ARR] / 1e6, h.stats[S_T_CPY] / 1e6,
                 h.stats[S_T_RUN] / 1e6, h.stats[S_T_IDLE] / 1e6);
  }
}

// The search did not end cleanly: status and a message with the site code and queue / proxy progress.
int device_failure(gorio_index *ix, const Ctl &h, u32 nq) {
  char buf[640];
  const u32 s = h.status ? h.status : (u32)GORIO_ERR_INTERNAL;
  std::snprintf(buf, sizeof buf,
                "device: %s (site 0x%x, %u, %u, %u; block %u thread %u; done %u/%u; posted %u; arrivals %u/%u; "
                "runnable %u/%u; want %u/%u; proxy consumed %u published %u outstanding %u queued %u "
                "[head command %u ack %u])",
                s < 9 ? kDeviceErr[s] : "?", h.dbg[0], h.dbg[1], h.dbg[2], h.dbg[3], h.dbg[4], h.dbg[5], h.done, nq,
                h.ring_head, h.q_heads[0], h.q_heads[1], h.q_heads[3], h.q_heads[4], h.q_heads[6], h.q_heads[7],
                ix->px_dbg[0], ix->px_dbg[1], ix->px_dbg[2], ix->px_dbg[3], ix->px_dbg[4], ix->px_dbg[5]);
  return fail(ix, (int)s, buf);
}


}  // namespace

namespace gorio {
// message of the last failed call that has no index handle (this thread)
void set_global_error(const char *msg) {
  std::snprintf(g_global_error, sizeof g_global_error, "%s", msg ? msg : "");
}
}  // namespace gorio

// =========================================================================================
extern "C" {

const char *gorio_status_str(int s) {
  switch (s) {
    case GORIO_OK: return "ok";
    case GORIO_ERR_INVALID_ARG: return "invalid argument";
    case GORIO_ERR_CUDA: return "CUDA error";
    case GORIO_ERR_NOMEM: return "out of memory";
    case GORIO_ERR_STATE: return "call out of order";
    case GORIO_ERR_TIMEOUT: return "timeout";
    case GORIO_ERR_CAPACITY: return "capacity exhausted";
    case GORIO_ERR_INDEX_CORRUPT: return "corrupt index";
    case GORIO_ERR_INTERNAL: return "internal error";
    default: return "unknown status";
  }
}

const char *gorio_last_error(gorio_index *ix) { return ix ? ix->err.c_str() : g_global_error; }

int gorio_index_open(const gorio_index_desc *d, int cuda_device, gorio_index **out) {
  if (!d || !out) return GORIO_ERR_INVALID_ARG;
  const u32 esz = d->dtype == GORIO_DTYPE_U8 ? 1u : 4u;
  const u64 nb = (u64)d->dim * esz + 4 + 4ull * d->max_degree;
  if (d->dtype > GORIO_DTYPE_F32 || d->page_bytes != kPageBytes || d->dim == 0 || d->dim % 4 != 0 ||
      d->max_degree == 0 || d->nodes_per_page == 0 || nb * d->nodes_per_page > kPageBytes ||
      d->n_nodes == 0 || d->n_nodes >= (1ull << 31) || d->entry_id >= d->n_nodes || !d->host_pages)
    return GORIO_ERR_INVALID_ARG;
  if (d->pq_m) {
    if (d->dtype != GORIO_DTYPE_U8 || d->dim % d->pq_m != 0 || (d->dim / d->pq_m) % 4 != 0 ||
        d->pq_m > 64 || d->dim / d->pq_m > 16 || !d->pq_centroids_dev || !d->pq_codes_dev)
      return GORIO_ERR_INVALID_ARG;
  }
  gorio_index *ix = new (std::nothrow) gorio_index();
  if (!ix) return GORIO_ERR_NOMEM;
  ix->desc = *d;
  ix->dev = cuda_device;
  ix->node_bytes = (u32)nb;
  ix->vec_bytes = d->dim * esz;
  ix->n_pages = (u32)((d->n_nodes + d->nodes_per_page - 1) / d->nodes_per_page);
  auto bail = [&](int st) { gorio_index_close(ix); return st; };
  cudaError_t e = cudaSetDevice(cuda_device);
  if (e != cudaSuccess) return bail(GORIO_ERR_CUDA);
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, cuda_device) != cudaSuccess) return bail(GORIO_ERR_CUDA);
  ix->n_sms = prop.multiProcessorCount;
  const size_t bytes = (size_t)ix->n_pages * kPageBytes;
  if (!(d->flags & GORIO_FLAG_PAGES_ALREADY_PINNED)) {
    e = cudaHostRegister((void *)d->host_pages, bytes, cudaHostRegisterMapped | cudaHostRegisterPortable);
    if (e != cudaSuccess) { cudaGetLastError(); return bail(GORIO_ERR_CUDA); }
    ix->registered_pages = true;
  }
  void *dp = nullptr;
  if (cudaHostGetDevicePointer(&dp, (void *)d->host_pages, 0) != cudaSuccess) return bail(GORIO_ERR_CUDA);
  ix->pages_dev = (const u8 *)dp;
  if (preload_kernels() != cudaSuccess) return bail(GORIO_ERR_CUDA);
  if (host_mapped(&ix->hctl_h, &ix->hctl_d, 64, cudaHostAllocWriteCombined) != cudaSuccess) return bail(GORIO_ERR_CUDA);
  if (cudaMalloc(&ix->ctl, sizeof(Ctl)) != cudaSuccess) return bail(GORIO_ERR_NOMEM);
  cudaMemset(ix->ctl, 0, sizeof(Ctl));
  if (cudaStreamCreateWithFlags(&ix->own_stream, cudaStreamNonBlocking) != cudaSuccess) return bail(GORIO_ERR_CUDA);
  if (cudaEventCreateWithFlags(&ix->done_ev, cudaEventDisableTiming) != cudaSuccess) return bail(GORIO_ERR_CUDA);
  for (int i = 0; i < kFillStreams; ++i)
    if (cudaStreamCreateWithFlags(&ix->fill_streams[i], cudaStreamNonBlocking) != cudaSuccess) return bail(GORIO_ERR_CUDA);
  for (int i = 0; i < kFillEvents; ++i)
    if (cudaEventCreateWithFlags(&ix->fill_events[i], cudaEventDisableTiming) != cudaSuccess) return bail(GORIO_ERR_CUDA);
  ix->proxy = std::thread(proxy_main, ix);
  *out = ix;
  return GORIO_OK;
}

int gorio_index_close(gorio_index *ix) {
  if (!ix) return GORIO_ERR_INVALID_ARG;
  cudaSetDevice(ix->dev);
  if (ix->proxy.joinable()) {
    ix->px_stop.store(1);
    {
      std::lock_guard<std::mutex> lk(ix->mu);
      ix->px_state.store(PX_EXIT);
    }
    ix->cv.notify_all();
    ix->proxy.join();
  }
  cudaDeviceSynchronize();
  free_cache(ix);
  free_qstate(ix);
  cudaFree(ix->ctl);
  cudaFree(ix->st_q); cudaFree(ix->st_out);
  if (ix->hctl_h) cudaFreeHost(ix->hctl_h);
  if (ix->own_stream) cudaStreamDestroy(ix->own_stream);
  if (ix->done_ev) cudaEventDestroy(ix->done_ev);
  for (int i = 0; i < kFillStreams; ++i) if (ix->fill_streams[i]) cudaStreamDestroy(ix->fill_streams[i]);
  for (int i = 0; i < kFillEvents; ++i) if (ix->fill_events[i]) cudaEventDestroy(ix->fill_events[i]);
  if (ix->registered_pages) cudaHostUnregister((void *)ix->desc.host_pages);
  delete ix;
  return GORIO_OK;
}

int gorio_cache_config(gorio_index *ix, const gorio_cache_cfg *cfg) {
  if (!ix || !cfg) return GORIO_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> api_lock(ix->api_mu);
  if (cfg->capacity_pages < 16 || cfg->max_outstanding < 1)
    return fail(ix, GORIO_ERR_INVALID_ARG, "cache_config: capacity >= 16, max_outstanding >= 1");
  if (cfg->granularity > GORIO_GRAN_RECORD) return fail(ix, GORIO_ERR_INVALID_ARG, "cache_config: unknown granularity");
  if (cfg->copy_mode > GORIO_COPY_ENGINE) return fail(ix, GORIO_ERR_INVALID_ARG, "cache_config: unknown copy_mode");
  if (cfg->granularity == GORIO_GRAN_RECORD && cfg->preload)
    return fail(ix, GORIO_ERR_INVALID_ARG, "cache_config: preload needs page granularity");
  u64 cap = cfg->capacity_pages < ix->n_pages ? cfg->capacity_pages : ix->n_pages;
  if (cfg->granularity == GORIO_GRAN_RECORD) {
    cap = cap * kPageBytes / ((ix->node_bytes + 12u + 15u) & ~15u);
    if (cap > ix->desc.n_nodes) cap = ix->desc.n_nodes;
  }
  if (cap >= (1ull << 24)) return fail(ix, GORIO_ERR_INVALID_ARG, "cache_config: at most 2^24 slots");
  CK(cudaSetDevice(ix->dev));
  ix->cfg = *cfg;
  if (ix->cfg.timeout_ms == 0) ix->cfg.timeout_ms = 60000;
  return setup_cache(ix);
}

int gorio_set_tuning(gorio_index *ix, const gorio_tuning *t) {
  if (!ix || !t) return GORIO_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> api_lock(ix->api_mu);
  if (t->visited_capacity && ((t->visited_capacity & (t->visited_capacity - 1)) || t->visited_capacity < 64))
    return fail(ix, GORIO_ERR_INVALID_ARG, "visited_capacity must be a power of two >= 64");
  if (t->warps_per_block > 24) return fail(ix, GORIO_ERR_INVALID_ARG, "warps_per_block <= 24");
  if (t->stash_entries > 1 && ((t->stash_entries & (t->stash_entries - 1)) || t->stash_entries < 64))
    return fail(ix, GORIO_ERR_INVALID_ARG, "stash_entries must be 0 (default), 1 (off) or a power of two >= 64");
  ix->tune = *t;
  return GORIO_OK;
}

int gorio_search(gorio_index *ix, const void *queries_dev, uint32_t nq, uint32_t K, uint32_t L, uint32_t W,
                 uint32_t *out_ids_dev, void *out_dists_dev, uint32_t *out_pages_distinct_dev,
                 uint32_t *out_counters_dev, void *cuda_stream) {
  if (!ix) return GORIO_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> api_lock(ix->api_mu);
  if (!queries_dev || !out_ids_dev || !out_dists_dev || nq < 1 || K < 1 || K > L || L > 256 || W < 1 ||
      W > 16 || (u64)W * ix->desc.max_degree > 1024)
    return fail(ix, GORIO_ERR_INVALID_ARG, "search: need 1 <= K <= L <= 256, 1 <= W <= 16, W*max_degree <= 1024");
  // the kernels read and write 32-bit words through these pointers: a misaligned one would trap
  if ((((uintptr_t)queries_dev | (uintptr_t)out_ids_dev | (uintptr_t)out_dists_dev | (uintptr_t)out_pages_distinct_dev |
        (uintptr_t)out_counters_dev) & 3u) != 0)
    return fail(ix, GORIO_ERR_INVALID_ARG, "search: queries and outputs must be at least 4-byte aligned");
  if (!ix->cache_ready) return fail(ix, GORIO_ERR_STATE, "search: call gorio_cache_config first");
  CK(cudaSetDevice(ix->dev));
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  const auto t_begin = Clock::now();
  if (ix->cache_dirty) {           // a failed search left requests in flight: start from a clean cache
    int st = setup_cache(ix);
    if (st != GORIO_OK) return st;
  }
  u32 blocks = 0, warps = 0;
  int st = launch_geometry(ix, nq, K, W, &blocks, &warps);
  if (st != GORIO_OK) return st;
  // on the resident fast path a warp carries one query from start to end, so no more query slots
  // than worker warps are ever in use (less state to clear per call)
  st = ensure_qstate(ix, nq, K, L, W, resident_fast_path(ix, K, W) ? blocks * warps : 0u);
  if (st != GORIO_OK) return st;

  fill_ctx(ix, queries_dev, nq, K, L, W, out_ids_dev, out_dists_dev, out_pages_distinct_dev, out_counters_dev);
  Ctx &c = ix->ctx;

  // reset the host-visible rings while the proxy is idle
  std::memset(ix->ring_h, 0, (size_t)ix->ring_cap * 8);
  std::memset(ix->fdone_h, 0, (size_t)ix->ring_cap * 4);
  std::memset(ix->hctl_h, 0, 64 * 4);
  flush_wc();
  std::atomic_thread_fence(std::memory_order_seq_cst);

  CK(cudaMemsetAsync(c.ring_dev, 0, (size_t)ix->ring_cap * 8, stream));      // no descriptor of an earlier search may look ready
  CK(cudaMemsetAsync(c.seen, c.seen_bitmap ? 0x00 : 0xFF, (size_t)c.n_qslots * c.seen_cap * 4, stream));
  CK(cudaMemsetAsync(c.pset, c.pset_bitmap ? 0x00 : 0xFF, (size_t)c.n_qslots * c.pset_cap * 4, stream));
  if (c.stash_cap) CK(cudaMemsetAsync(c.stash_tag, 0xFF, (size_t)c.n_qslots * c.stash_cap * 4, stream));
  CK(launch_init(c, stream));
  ix->cache_dirty = true;      // until this search ends cleanly
  proxy_start(ix);
  cudaError_t le = launch_search(c, blocks, warps, stream);
  if (le != cudaSuccess) { proxy_stop(ix); return cuda_fail(ix, le, "launch_search"); }
  cudaEventRecord(ix->done_ev, stream);

  // wait for the kernel; a host-side watchdog asks the device to abort if it overruns
  const auto deadline = Clock::now() + std::chrono::milliseconds(ix->cfg.timeout_ms);
  bool host_abort = false;
  cudaError_t qe;
  while ((qe = cudaEventQuery(ix->done_ev)) == cudaErrorNotReady) {
    if (ix->px_error.load() && !host_abort) { ((volatile u32 *)ix->hctl_h)[1] = 1; flush_wc(); host_abort = true; }
    if (!host_abort && Clock::now() > deadline) { ((volatile u32 *)ix->hctl_h)[1] = 1; flush_wc(); host_abort = true; }
    std::this_thread::sleep_for(std::chrono::microseconds(20));
  }
  proxy_stop(ix);
  if (qe != cudaSuccess) return cuda_fail(ix, qe, "search kernel");
  Ctl h{};
  CK(cudaMemcpyAsync(&h, ix->ctl, sizeof(Ctl), cudaMemcpyDeviceToHost, stream));
  CK(cudaStreamSynchronize(stream));
  ix->host_search_ns += (u64)std::chrono::duration_cast<std::chrono::nanoseconds>(Clock::now() - t_begin).count();
  print_diagnostics(c, h);
  if (ix->px_error.load() == 2) {
    for (int i = 0; i < kFillStreams; ++i) cudaStreamSynchronize(ix->fill_streams[i]);
    return fail(ix, GORIO_ERR_CUDA, "proxy: a page copy or its completion event failed");
  }
  if (ix->px_error.load()) return fail(ix, GORIO_ERR_INTERNAL, "proxy: descriptor out of range");
  if (h.status != 0 || h.stop != 1) return device_failure(ix, h, nq);
  ix->cache_dirty = false;
  return GORIO_OK;
}

int gorio_search_host(gorio_index *ix, const void *queries_host, uint32_t nq, uint32_t K, uint32_t L, uint32_t W,
                      uint32_t *out_ids_host, void *out_dists_host, uint32_t *out_pages_distinct_host,
                      uint32_t *out_counters_host) {
  if (!ix || !queries_host || !out_ids_host || !out_dists_host || nq < 1 || K < 1) return GORIO_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> api_lock(ix->api_mu);
  CK(cudaSetDevice(ix->dev));
  const size_t qb = (size_t)nq * ix->vec_bytes;
  const size_t ob = (size_t)nq * K * 8 + (size_t)nq * 4 + (size_t)nq * 20;
  if (qb > ix->st_q_bytes) { cudaFree(ix->st_q); ix->st_q = nullptr; CK(cudaMalloc(&ix->st_q, qb)); ix->st_q_bytes = qb; }
  if (ob > ix->st_out_bytes) { cudaFree(ix->st_out); ix->st_out = nullptr; CK(cudaMalloc(&ix->st_out, ob)); ix->st_out_bytes = ob; }
  u32 *ids = (u32 *)ix->st_out;
  u32 *dists = ids + (size_t)nq * K;
  u32 *pages = dists + (size_t)nq * K;
  u32 *counters = pages + nq;
  cudaStream_t s = ix->own_stream;
  CK(cudaMemcpyAsync(ix->st_q, queries_host, qb, cudaMemcpyHostToDevice, s));
  int st = gorio_search(ix, ix->st_q, nq, K, L, W, ids, dists, pages, counters, s);
  if (st != GORIO_OK) return st;
  CK(cudaMemcpyAsync(out_ids_host, ids, (size_t)nq * K * 4, cudaMemcpyDeviceToHost, s));
  CK(cudaMemcpyAsync(out_dists_host, dists, (size_t)nq * K * 4, cudaMemcpyDeviceToHost, s));
  if (out_pages_distinct_host) CK(cudaMemcpyAsync(out_pages_distinct_host, pages, (size_t)nq * 4, cudaMemcpyDeviceToHost, s));
  if (out_counters_host) CK(cudaMemcpyAsync(out_counters_host, counters, (size_t)nq * 20, cudaMemcpyDeviceToHost, s));
  CK(cudaStreamSynchronize(s));
  return GORIO_OK;
}

int gorio_stats(gorio_index *ix, gorio_stats_t *out) {
  if (!ix || !out) return GORIO_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> api_lock(ix->api_mu);
  CK(cudaSetDevice(ix->dev));
  Ctl h{};
  CK(cudaMemcpy(&h, ix->ctl, sizeof(Ctl), cudaMemcpyDeviceToHost));
  std::memset(out, 0, sizeof(*out));
  out->pages_hit = h.stats[S_HIT]; out->pages_missed = h.stats[S_MISSED]; out->pages_fetched = ix->host_fetched;
  out->dedupe_joins = h.stats[S_JOINS]; out->evictions = h.stats[S_EVICT]; out->retries = h.stats[S_RETRY];
  out->max_outstanding_seen = ix->host_max_out; out->queries_done = h.stats[S_DONE];
  out->n_eval = h.stats[S_NEVAL]; out->n_expand = h.stats[S_NEXPAND]; out->sum_degree = h.stats[S_SUMDEG];
  out->n_iter = h.stats[S_NITER]; out->resumes = h.stats[S_RESUMES]; out->search_ns = ix->host_search_ns;
  out->proxy_batches = ix->host_batches; out->posted = h.stats[S_POSTED];
  out->proxy_service_ns = ix->host_service_ns; out->proxy_ack_wait_iters = ix->host_ack_wait;
  out->proxy_window_full_iters = ix->host_window_full; out->proxy_ring_empty_iters = ix->host_ring_empty;
  out->proxy_iters = ix->host_iters; out->proxy_outstanding_sum = ix->host_out_sum;
  out->warp_ns_arrivals = h.stats[S_T_ARR]; out->warp_ns_queries = h.stats[S_T_RUN]; out->warp_ns_idle = h.stats[S_T_IDLE];
  out->arrivals_consumed = h.stats[S_N_ARR]; out->warp_ns_copies = h.stats[S_T_CPY]; out->stash_hits = h.stats[S_STASH];
  out->fetched_bytes = ix->host_fetched_bytes;
  return GORIO_OK;
}

int gorio_link_probe(gorio_index *ix, uint32_t n_pulls, uint32_t pages_in_flight, int sequential, void *cuda_stream,
                     double *gbs_out) {
  if (!ix || !gbs_out) return GORIO_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> api_lock(ix->api_mu);
  if (n_pulls == 0 || pages_in_flight == 0 || pages_in_flight > 16384u)
    return fail(ix, GORIO_ERR_INVALID_ARG, "link_probe: need n_pulls >= 1 and 1 <= pages_in_flight <= 16384");
  CK(cudaSetDevice(ix->dev));
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  const u32 warps = (pages_in_flight + 3u) / 4u * 4u;        // whole blocks of four warps
  u8 *scratch = nullptr;
  u32 *words = nullptr;                                      // [0] next pull, [1] checksum sink
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  float ms = 0.f;
  cudaError_t e = cudaMalloc(&scratch, (size_t)warps * kPageBytes);
  if (e == cudaSuccess) e = cudaMalloc(&words, 8);
  if (e == cudaSuccess) e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  if (e == cudaSuccess) e = cudaMemsetAsync(words, 0, 8, stream);
  if (e == cudaSuccess) e = cudaEventRecord(e0, stream);
  if (e == cudaSuccess) e = launch_link_probe(ix->pages_dev, ix->n_pages, n_pulls, warps, sequential ? 1u : 0u, scratch, words, words + 1, stream);
  if (e == cudaSuccess) e = cudaEventRecord(e1, stream);
  if (e == cudaSuccess) e = cudaEventSynchronize(e1);
  if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  cudaFree(scratch); cudaFree(words);
  if (e != cudaSuccess) return cuda_fail(ix, e, "link_probe");
  *gbs_out = ms > 0.f ? (double)n_pulls * kPageBytes / ((double)ms * 1e6) : 0.0;
  return GORIO_OK;
}

int gorio_stats_reset(gorio_index *ix) {
  if (!ix) return GORIO_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> api_lock(ix->api_mu);
  CK(cudaSetDevice(ix->dev));
  CK(cudaMemset((u8 *)ix->ctl + offsetof(Ctl, stats), 0, sizeof(((Ctl *)0)->stats)));
  ix->host_fetched_bytes = 0;
  ix->host_fetched = ix->host_max_out = ix->host_batches = ix->host_search_ns = 0;
  ix->host_service_ns = ix->host_ack_wait = ix->host_window_full = ix->host_ring_empty = ix->host_iters = ix->host_out_sum = 0;
  return GORIO_OK;
}

}  // extern "C"
