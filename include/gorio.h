/*
 * gorio.h -- C ABI of the GPU-owned paged graph beam search.
 *
 * One B200 runs batched DiskANN-style beam search over a graph index stored as 4 KB
 * pages.  The GPU owns query evolution, the HBM page cache, page-miss generation,
 * pending-query state and resume decisions; a thin host proxy thread only services
 * page reads from the "remote" tier, which is emulated as pinned host memory with an
 * injected per-request latency (paper: Section 3.1 ownership split, Section 3.2 request
 * descriptors and per-slot ready table, Section 3.3 persistent scheduler and proxy).
 *
 * Conventions
 *   - Every function returns a gorio_status; nothing throws, aborts or traps.
 *   - "device" pointers are CUDA device memory of the index's device; "host" pointers
 *     are ordinary host memory.  No torch or C++ types cross this boundary.
 *   - The library needs its CUDA kernels: there is no CPU fallback of any kind.
 *   - Calls on one gorio_index are serialised by the library (a search blocks other callers of
 *     that index until it returns); different indexes are independent.  gorio_index_close must
 *     not race with any other call on the same handle.  gorio_last_error returns a pointer
 *     into the index that the next failing call overwrites.
 */
#ifndef GORIO_H
#define GORIO_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gorio_index gorio_index; /* opaque; created by gorio_index_open, freed by gorio_index_close */

typedef enum {
  GORIO_OK = 0,
  GORIO_ERR_INVALID_ARG = 1,   /* a precondition listed at the call does not hold */
  GORIO_ERR_CUDA = 2,          /* a CUDA runtime call failed (see gorio_last_error) */
  GORIO_ERR_NOMEM = 3,         /* device or host allocation failed */
  GORIO_ERR_STATE = 4,         /* call order: search before cache_config, ... */
  GORIO_ERR_TIMEOUT = 5,       /* a bounded device or host wait expired; all kernels have exited */
  GORIO_ERR_CAPACITY = 6,      /* per-query visited/page set or iteration limit exhausted */
  GORIO_ERR_INDEX_CORRUPT = 7, /* neighbour id >= n_nodes or degree > max_degree met in a page */
  GORIO_ERR_INTERNAL = 8       /* a self-check of the cache/scheduler state machine failed */
} gorio_status;

enum { GORIO_DTYPE_U8 = 0, GORIO_DTYPE_F32 = 1 };
enum { GORIO_FLAG_PAGES_ALREADY_PINNED = 1u }; /* host_pages is already page-locked and mapped */

/*
 * Index description (Section 5.1: "on-disk graph index"; the layout below is this
 * library's page-store format).
 *   Node i lives in page i / nodes_per_page at byte (i % nodes_per_page) * node_bytes,
 *   node_bytes = dim*elem_size + 4 + 4*max_degree.  A node is: vector[dim] (u8 or LE f32),
 *   degree (u32 LE), max_degree neighbour ids (u32 LE, unused entries 0xFFFFFFFF).
 *   host_pages: n_pages * 4096 bytes of HOST memory, owned by the caller and borrowed
 *   until gorio_index_close.  It is the emulated remote tier; the library page-locks it
 *   (cudaHostRegister) unless GORIO_FLAG_PAGES_ALREADY_PINNED is set.
 *   PQ navigation (optional): pq_m > 0 enables it; pq_centroids_dev is u8
 *   [pq_m][256][dim/pq_m] and pq_codes_dev is u8 [n_nodes][pq_m], both DEVICE memory
 *   borrowed until close.  Requires dtype u8, dim % pq_m == 0, dim/pq_m in {4, 8, 12, 16}.
 * Preconditions: page_bytes == 4096, dim % 4 == 0, nodes_per_page*node_bytes <= 4096,
 *   n_nodes < 2^31, entry_id < n_nodes, max_degree >= 1.
 */
typedef struct {
  uint64_t n_nodes;
  uint32_t dim;
  uint32_t dtype;
  uint32_t max_degree;
  uint32_t nodes_per_page;
  uint32_t page_bytes;
  uint32_t entry_id; /* medoid entry node */
  const void *host_pages;
  uint32_t pq_m;
  uint32_t flags;
  const uint8_t *pq_centroids_dev;
  const uint8_t *pq_codes_dev;
} gorio_index_desc;

/*
 * Page cache + remote tier configuration (Section 3.2: GPU page-cache slots with one
 * ready entry each; Section 3.3: the CPU proxy groups request submissions and completions
 * and bounds how many remote reads are outstanding).
 *   capacity_pages   HBM cache size in 4 KB slots (>= 16; capped at the number of pages).
 *                    Pages map to slots through a lock-free table with one state word per
 *                    page; victims are chosen by a clock hand with reference bits.
 *   remote_latency_ns  a request's completion is published no earlier than this long
 *                    after the proxy admitted it.
 *   max_outstanding  most requests admitted and not yet published (>= 1).
 *   preload          1: fill the cache with pages 0..capacity-1 now (whole index when
 *                    capacity >= n_pages); 0: start cold.
 *   timeout_ms       bound on one gorio_search call (device and host waits); 0 = 60000.
 *   granularity      GORIO_GRAN_PAGE (0): a miss fetches the whole 4 KB page and a slot holds a
 *                    page.  GORIO_GRAN_RECORD (1): selective materialisation (Section 7.2,
 *                    third direction: return only the graph records that are needed instead of
 *                    whole pages): a miss fetches just the wanted node's record -- the
 *                    16-byte-aligned span of the page that covers it, node_bytes + 12 rounded
 *                    up to 16 (400 bytes for a 388-byte record) -- and the cache holds records:
 *                    capacity_pages * 4096 bytes of HBM are divided into record slots (capped
 *                    at one slot per node), the lookup table has one word per node.  Search
 *                    results and per-query counters are identical in both modes (pages_distinct
 *                    still counts index pages); only the number and size of remote reads
 *                    change.  preload must be 0 in this mode.
 *   copy_mode        who moves a page's bytes from the pinned store into its slot:
 *                    GORIO_COPY_SM_PULL (0, default): the proxy admits the request by advancing a
 *                    counter in host-mapped memory; warps of the search kernel (one puller warp
 *                    per block, in ring order; see gorio_tuning.shared_pull) pull the page over
 *                    the host link and acknowledge; the proxy publishes the completion after the
 *                    latency.  The proxy makes no CUDA call while a search runs.
 *                    GORIO_COPY_ENGINE (1): the proxy thread itself copies the page, one
 *                    cudaMemcpyAsync per request on streams of its own (the GPU's copy engine does
 *                    the transfer), learns from an event that the copy has landed, and then
 *                    publishes the completion.  No SM cycles go into fills.
 *
 * Departure from the benchmark spec: who copies.  Section 3.2 has a CPU worker fill the cache slot
 * and then mark its ready entry, and Section 4 calls the CPU side a transport proxy.  Here the
 * default is GORIO_COPY_SM_PULL, and GORIO_COPY_ENGINE is the literal reading kept as an option.
 * The reason is the request rate: the benchmark configuration needs about 11 million 4 KB fills
 * per second; a small cudaMemcpyAsync issued while the persistent kernel is resident completes about
 * a millisecond after the call (0.23 million fills per second with 256 in flight) and costs the
 * calling thread about 2 microseconds, and no batched-copy runtime call is usable on the target
 * machines; SM reads of pinned memory reach 51 of the 55.5 GB/s a bulk copy gets on the same link.  In both
 * modes the proxy alone admits requests, bounds the number outstanding, applies the latency and
 * publishes completions in ring order, and it never looks at search state.
 * Calling gorio_cache_config again re-creates an empty (or preloaded) cache.
 */
typedef struct {
  uint64_t capacity_pages;
  uint32_t remote_latency_ns;
  uint32_t max_outstanding;
  uint32_t preload;
  uint32_t timeout_ms;
  uint32_t granularity;
  uint32_t copy_mode;
} gorio_cache_cfg;

enum { GORIO_COPY_SM_PULL = 0, GORIO_COPY_ENGINE = 1 };
enum { GORIO_GRAN_PAGE = 0, GORIO_GRAN_RECORD = 1 };

/*
 * Scheduler tuning; all zero = defaults.
 *   max_inflight     query slots resident at once (pending/running queries); default 16384.
 *   visited_capacity per-query exact visited-set entries (power of two), default 32768;
 *                    a query that scores more nodes fails with GORIO_ERR_CAPACITY.  When a
 *                    bitmap over all nodes needs no more memory than that (n_nodes / 32 words
 *                    <= visited_capacity), the bitmap is used instead and can never fill up.
 *   warps_per_block / blocks_per_sm  launch geometry of the persistent kernel (<= 24 warps; with
 *                    PQ navigation at most 12, fewer if the per-warp tables do not fit).
 *   stash_entries    per-query adjacency stash (exact navigation): entries of a direct-mapped
 *                    table that keeps a scored node's neighbour list so that expanding it later
 *                    needs no page; 0 = default 1024, 1 = off, else a power of two >= 64.
 *                    It never changes results, only how many pages are waited for.
 *   request_backlog  most requests posted to the proxy and not yet arrived; 0 = default
 *                    min(4 * max_outstanding, 1024), never below max_outstanding.  More than the proxy can have in service only queues
 *                    in the ring while occupying cache slots that could hold resident pages.
 *   no_fast_path     1 = do not use the whole-index-resident fast path.  When the whole index was
 *                    preloaded (nothing can miss) a warp normally runs each query from admission
 *                    to output without parking it, with the list in registers and the candidates
 *                    in shared memory; with this flag such a search goes through the general
 *                    park-and-resume machinery instead.  Results are identical; for comparisons.
 *   shared_pull      1 = ablation: no dedicated puller warps.  By default (page granularity, SM
 *                    pull) the last warp of every block does nothing but pull admitted pages, in
 *                    ring order: it claims the next request index ahead of time, waits until the
 *                    admission is known on the GPU and issues the page's reads at once; worker
 *                    warps pull nothing.  With this flag, as always at record granularity, worker
 *                    warps take the pulls between their other work (whoever looks first), which
 *                    starts them later and out of order.  Results are identical.
 *   blocking         1 = ablation: a warp that misses keeps its query and waits in place for
 *                    the pages (the demand-paging baseline of Section 5.1) instead of parking
 *                    the query and taking another; results are identical, only slower.
 */
typedef struct {
  uint32_t max_inflight;
  uint32_t visited_capacity;
  uint32_t warps_per_block;
  uint32_t blocks_per_sm;
  uint32_t stash_entries;
  uint32_t blocking;
  uint32_t request_backlog;
  uint32_t no_fast_path;
  uint32_t shared_pull;
} gorio_tuning;

/*
 * Counters since the last gorio_stats_reset.
 *   pages_hit      page lookups satisfied from a resident slot
 *   pages_missed   (query, node) waits registered on a page in flight (owner or joiner)
 *   pages_fetched  request descriptors the proxy serviced (4 KB each; one record each at
 *                  record granularity); fetched_bytes: the bytes they moved over the host link
 *   dedupe_joins   waits that joined another query's or lane's outstanding request
 *   evictions, retries (hits that were evicted under the read and looked up again),
 *   max_outstanding_seen (proxy), queries_done,
 *   n_eval / n_expand / sum_degree: totals of the per-query search counters (used for
 *   the algorithmic byte count), search_ns: wall time of the blocking search calls.
 * Hit/miss/fetch counts depend on timing; they obey invariants, not fixed values.
 */
typedef struct {
  uint64_t pages_hit, pages_missed, pages_fetched;
  uint64_t dedupe_joins, evictions, retries, max_outstanding_seen, queries_done;
  uint64_t n_eval, n_expand, sum_degree, n_iter;
  uint64_t resumes, search_ns, proxy_batches, posted;
  /* proxy diagnostics: sum over published requests of (publish - admit) in ns; loop
     iterations in total / that found the head copy not yet acknowledged / with the window
     full and a descriptor waiting / with room in the window but no descriptor; sum over
     iterations of the requests in service (divide by proxy_iters for the time average) */
  uint64_t proxy_service_ns, proxy_iters, proxy_ack_wait_iters, proxy_window_full_iters;
  uint64_t proxy_ring_empty_iters, proxy_outstanding_sum;
  /* where the worker warps' time went, ns summed over warps: serving arrived pages,
     running query phases, idle; the number of arrival-queue items consumed; ns spent pulling
     pages (by the puller warps, whose waiting for the next admission is not counted anywhere, or in
     the shared scheme by the worker warps) */
  uint64_t warp_ns_arrivals, warp_ns_queries, warp_ns_idle, arrivals_consumed;
  uint64_t warp_ns_copies, stash_hits;   /* expansions served from the adjacency stash */
  uint64_t fetched_bytes;
} gorio_stats_t;

/*
 * Open an index on CUDA device `cuda_device` (Section 5.1: the searches run against one
 * on-disk graph index; Section 3.1: the CPU side keeps the remote tier, the GPU everything
 * else).  Page-locks and maps the page store, starts the proxy thread (idle until a search),
 * loads the kernels.  *out is set only on GORIO_OK; desc is copied, host_pages and the PQ
 * arrays are borrowed until gorio_index_close.  Errors: INVALID_ARG (a precondition of
 * gorio_index_desc), CUDA, NOMEM.
 */
int gorio_index_open(const gorio_index_desc *desc, int cuda_device, gorio_index **out);

/* (Re)create the page cache (Section 3.2) and arm the remote-tier emulation.  Blocking.
 * Errors: INVALID_ARG (capacity_pages < 16, max_outstanding < 1, unknown granularity, preload at
 * record granularity, more than 2^24 slots), CUDA, NOMEM. */
int gorio_cache_config(gorio_index *ix, const gorio_cache_cfg *cfg);

/* Optional; takes effect at the next gorio_search.  (No counterpart in the paper: knobs of this
 * implementation's scheduler.) */
int gorio_set_tuning(gorio_index *ix, const gorio_tuning *t);

/*
 * Batched beam search (Section 2.2: expand nodes, evaluate distances, update the
 * candidate list, discover the next pages; Section 3.3: queries that miss are parked
 * and resumed by the GPU scheduler).  For every query: start at entry_id; repeatedly
 * take the first W unexpanded entries of the L-entry list ordered by (distance, id),
 * read their adjacency from their pages, score every not-yet-visited neighbour (exact
 * navigation: from the neighbour's own page; PQ navigation: from resident codes) and keep
 * the L best; stop when no unexpanded entry remains.  Output the best K by (distance, id)
 * (PQ navigation: best K expanded nodes by exact distance).
 *
 *   queries_dev   DEVICE [nq][dim], index dtype, row major.
 *   out_ids_dev   DEVICE [nq][K] u32; out_dists_dev DEVICE [nq][K] (u32 for u8 data, f32
 *                 for f32 data).  Missing results are 0xFFFFFFFF / 0xFFFFFFFF or +inf.
 *   out_pages_distinct_dev  DEVICE [nq] u32 or NULL: distinct pages each query touched.
 *   out_counters_dev        DEVICE [nq][5] u32 or NULL: pages_distinct, iterations,
 *                 expansions, evaluations, sum of expanded degrees.
 *   cuda_stream   cudaStream_t (or NULL for the default stream) used for the launches.
 * Preconditions: 1 <= K <= L <= 256, 1 <= W <= 16, W*max_degree <= 1024, nq >= 1.
 * Blocking: returns after all queries finished (results visible on the device) or with an
 * error status after every kernel and proxy action of this call has ended.
 */
int gorio_search(gorio_index *ix, const void *queries_dev, uint32_t nq, uint32_t K, uint32_t L,
                 uint32_t W, uint32_t *out_ids_dev, void *out_dists_dev,
                 uint32_t *out_pages_distinct_dev, uint32_t *out_counters_dev, void *cuda_stream);

/*
 * The same search with HOST buffers: queries are copied host->device, results
 * device->host, inside the call (the end-to-end path).  out_pages_distinct_host and
 * out_counters_host may be NULL.
 */
int gorio_search_host(gorio_index *ix, const void *queries_host, uint32_t nq, uint32_t K,
                      uint32_t L, uint32_t W, uint32_t *out_ids_host, void *out_dists_host,
                      uint32_t *out_pages_distinct_host, uint32_t *out_counters_host);

/*
 * Counters since the last reset, gorio_stats_t above (Section 5.1 reports search time only; the
 * hit / miss / fetch counts are what Section 3.2's cache and request protocol make observable, and
 * the proxy figures are Section 3.3's outstanding-I/O control seen from the host).  `out` is HOST
 * memory, fully overwritten.  Blocking (one small device-to-host copy); call it between searches.
 */
int gorio_stats(gorio_index *ix, gorio_stats_t *out);
/* Zero every counter of gorio_stats_t (device and proxy side).  No counterpart in the paper. */
int gorio_stats_reset(gorio_index *ix);

/*
 * Measurement aid (no counterpart in the paper): what the host link delivers to the access pattern
 * of a page fill and nothing else.  `pages_in_flight` warps (rounded up to a multiple of four, at
 * most 16384) each pull whole 4 KB pages of the index's pinned page store into a 4 KB HBM area of
 * their own, one page at a time with the page's loads all in flight -- the loads a fill of the
 * search kernel issues -- until `n_pulls` pages have been pulled; pull i reads page hash(i) mod
 * n_pages (uniformly scattered) or, with `sequential` != 0, page i mod n_pages.  No cache, no proxy,
 * no latency, no window.  `gbs_out` (HOST) receives n_pulls * 4096 bytes over the kernel's duration
 * (CUDA events on `cuda_stream`), in GB/s.  bench.py reports it beside the bulk-copy figure: random
 * 4 KB reads of a store much larger than the host's last-level cache run slower than one long copy.
 * Allocates and frees its scratch (pages_in_flight x 4 KB) inside the call; blocking; must not
 * overlap a search on the same index.  Errors: INVALID_ARG, CUDA.
 */
int gorio_link_probe(gorio_index *ix, uint32_t n_pulls, uint32_t pages_in_flight, int sequential, void *cuda_stream,
                     double *gbs_out);

/* Stops the proxy thread, frees every device and host resource of the index, un-pins the page
 * store if the library pinned it.  The handle is invalid afterwards.  (Resource management: no
 * counterpart in the paper.) */
int gorio_index_close(gorio_index *ix);

/*
 * Search for callers that cannot allocate (the paper has no counterpart: this is a
 * packaging variant of gorio_search, not a step of its method).
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- services whose device
 * memory is a pre-sized arena with every byte accounted for, latency-critical loops that
 * cannot take the allocator's implicit device synchronisation, plugins whose host forbids
 * allocation after start-up.  gorio_index_open / gorio_cache_config / gorio_search allocate
 * device and pinned memory; this call allocates nothing, on the device or on the host, and
 * needs no index handle.
 *
 * What it does: the same beam search (exact navigation only, pq_m must be 0), by the same
 * kernels, over an index whose pages are ALL resident in device memory, so there are no
 * misses and no proxy.  All working state comes from one fixed 12 MiB device array that is
 * part of the library image: every GPU context that loads the library carries it until the
 * process exits.
 *
 *   desc        index description; host_pages, flags and the PQ pointers are ignored.
 *   pages_dev   DEVICE, n_pages * 4096 bytes in the page-store format, read only; at least
 *               4-byte aligned (INVALID_ARG otherwise), 16-byte aligned for the 128-bit load path.
 *               n_pages = ceil(n_nodes / nodes_per_page): the kernels read the page of any
 *               neighbour id below n_nodes, so the buffer must really be that large.
 *   queries_dev, out_ids_dev, out_dists_dev, out_pages_distinct_dev (may be NULL), cuda_stream:
 *               as for gorio_search.  Runs on the CURRENT device; all pointers must belong to it.
 * Limits (fixed by the array's size; beyond them the call returns GORIO_ERR_INVALID_ARG and
 * gorio_last_error(NULL) says which): at most 32768 pages (128 MiB of index),
 * n_nodes < 2^31, 1 <= K <= L <= 256, W <= 16, W * max_degree <= 256.  At most 64 queries are
 * in flight at a time; any nq is accepted, but the whole call has a fixed budget of 60 s on the
 * device (not per wait): a batch that needs longer returns GORIO_ERR_TIMEOUT and its partial
 * results are unspecified -- split such batches.  (12,000 config-1-sized queries take well under
 * a second.)  A query that visits more than 16384 nodes fails the call with GORIO_ERR_CAPACITY.
 * Sharing: every call on a GPU uses the same array, which still holds the previous call's
 * state; the call re-initialises what must start clean.  Calls whose kernels overlap on one
 * GPU race on it -- serialise them.  The call blocks until its kernel has finished.
 * First call on a device: it also resolves the array's device address
 * (cudaGetSymbolAddress) and loads the kernels.  Every call ends with a stream synchronisation
 * and a small device-to-host copy of the status, so it must not be made while a stream capture
 * is in progress.
 */
int gorio_search_resident_noalloc(const gorio_index_desc *desc, const void *pages_dev,
                                  const void *queries_dev, uint32_t nq, uint32_t K, uint32_t L,
                                  uint32_t W, uint32_t *out_ids_dev, void *out_dists_dev,
                                  uint32_t *out_pages_distinct_dev, void *cuda_stream);

/* Static strings; never NULL. */
const char *gorio_status_str(int status);
/* Human-readable detail of the last non-OK status on this index (valid until the next call);
 * with ix == NULL, of the last failed call of this thread that takes no index handle. */
const char *gorio_last_error(gorio_index *ix);

#ifdef __cplusplus
}
#endif
#endif /* GORIO_H */
