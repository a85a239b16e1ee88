// Internal definitions shared by the host API (gorio_api.cu) and the device code
// (search_kernels.cu).  Nothing here is part of the public C ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace gorio {

typedef uint8_t u8;
typedef uint16_t u16;
typedef uint32_t u32;
typedef uint64_t u64;

constexpr u32 kPageBytes = 4096;
constexpr u32 kNil = 0xFFFFFFFFu;     // end of a waiter list
constexpr u32 kClosed = 0xFFFFFFFEu;  // waiter list closed: the page has arrived
constexpr u32 kInvalidId = 0xFFFFFFFFu;
constexpr u64 kPadKey = ~0ull;        // sorts after every real key
constexpr u32 kPqKsub = 256;
constexpr u32 kPqLutWords = 160;       // u32 words of shared memory per subspace: 256 x u16 + 256 x 4 bits

// Query phases: which batch of page items is outstanding for the query slot.
enum Phase : u32 { PH_NEW = 0, PH_EVAL = 1, PH_EXPAND = 2 };

// Per-query-slot header (64 bytes).  Written by the warp that runs the query; `awaiting`
// is decremented by whoever consumes one of the query's page items.
struct QHdr {
  u32 qid;
  u32 phase;
  u32 awaiting;   // outstanding items of the current batch (+1 guard while issuing/retrying)
  u32 n_items;    // items in the current batch
  u32 reserved0;
  u32 list_len;
  u32 n_iter, n_expand, n_eval, sum_deg, pages_distinct;
  u32 pool_len;   // PQ mode: entries in the rerank pool
  u32 worst_lo, worst_hi;   // the list's L-th key as of the last merge (all ones until the list is full)
  u32 pad[2];
};

// Multi-producer multi-consumer ring of u32 values in HBM (cells hold sequence << 32 | value).
struct Queue {
  u32 *buf;
  u32 mask;
  u32 *head;
  u32 *tail;
  int *count;   // items pushed minus items claimed by consumers
};

// Clock hand and never-used-slot bump pointer of the page cache.
struct CacheShared {
  u32 hand;
  u32 bump;
  u32 copy_head;   // next admitted request to copy
  u32 comp_head;   // next published completion to consume
  int in_flight;   // requests posted whose arrival has not been picked up yet
};

// Device-resident control block.
struct Ctl {
  // work counters, together in one 32-byte sector so that an idle warp reads them at once:
  // [0] admitted requests nobody copies yet, [1] published completions nobody consumes yet,
  // [2] arrival queue, [3] runnable queue, [4] want queue (items pushed minus items claimed)
  int counts[8];
  u32 stop;        // 0 run, 1 all queries done, 2 error/abort
  u32 status;      // first gorio_status raised on the device
  u32 next_query;  // next query id to admit when a slot frees
  u32 done;        // queries finished
  u32 ring_head;   // request descriptors posted
  u32 adm_seen;    // admitted-request count the poller last read from the host (puller warps wait on it)
  u32 q_heads[16]; // queue head/tail words: arr(0,1) run(3,4) want(6,7)
  u32 dbg[8];      // detail of the first error
  u32 census[16];  // debug snapshot (see census())
  u64 stats[48];
};

enum StatIdx { S_HIT = 0, S_MISSED, S_JOINS, S_EVICT, S_RETRY, S_DONE, S_NEVAL, S_NEXPAND,
               S_SUMDEG, S_NITER, S_RESUMES, S_POSTED, S_T_ARR, S_T_RUN, S_T_IDLE, S_N_ARR, S_T_CPY, S_STASH,
               // debug profile (Ctx::prof): warp time per query phase step
               S_P_MERGE, S_P_ISSUE_EVAL, S_P_ISSUE_EXP, S_P_COLLECT, S_P_POOL, S_P_LUT, S_P_ADC, S_P_FINISH, S_P_RECYCLE,
               S_I_SETUP, S_I_LOOKUP, S_I_CONSUME, S_I_TAIL,     // inside issue_batch
               S_POLLS,                                           // control reads the poller made
               S_A_HEAD, S_A_WALK, S_A_GROUP, S_A_COMPLETE, S_A_FINISH,     // inside an arrival
               S_C_DATA };                                        // copy: loads issued -> bytes in registers

// Everything the persistent kernel needs, passed by value.
struct Ctx {
  // index
  u32 n_nodes, dim, dtype, R, npp, node_bytes, vec_bytes, entry, n_pages;
  u32 pq_m, pq_dsub;
  const u8 *pq_cent;
  const u8 *pq_codes;
  // page cache
  u8 *slot_data;   // n_slots * 4096
  u64 *ptab;       // [n_units] page words: state, slot, waiter-list head or generation
  u64 *smeta;      // [n_slots] slot words: page, generation, reference bit
  u32 *parts;      // [n_slots] waiter-chain segments still being served
  u32 *filled;     // [n_slots] generation whose bytes the copier has stored into the slot
  CacheShared *cs; // clock hand and bump pointer
  u32 n_slots;
  // cache unit: a 4 KB page (unit = node / npp, slot_bytes = 4096), or with selective
  // materialisation one node record (unit = node; a slot holds the 16-byte-aligned span of the
  // page that covers the record, so the record starts (offset in page) & 15 bytes into it)
  u32 n_units, slot_bytes, record_mode;
  // miss ring: host-mapped, written by the GPU, consumed by the proxy
  u64 *ring;
  u32 ring_mask, ring_shift;
  u64 *ring_dev;        // device copy of every posted descriptor
  // host-mapped words written by the proxy: [0] completions published, [1] abort request,
  // [2] requests admitted (both counts are in ring order)
  const u32 *host_ctl;
  u32 *fdone;           // per-request copy acknowledgement (lap tag), written by the GPU
  const u8 *host_pages; // device view of the pinned host page store
  Queue arr, run, want;   // arrivals (slots / chain continuations), runnable query slots, pages awaiting a slot
  // query state
  u32 n_qslots, nq, K, L, W, WR;
  QHdr *hdr;
  u64 *list;     // [n_qslots][L]
  u64 *cand;     // [n_qslots][WR]
  u32 *items;    // [n_qslots][WR] node id of each item of the current batch
  u32 *wrec;     // [n_qslots][WR] next pointers of waiter records (record id = qs*WR + j)
  u32 *adj;      // [n_qslots][W][R]
  u32 *adjdeg;   // [n_qslots][W]
  u32 *seen;     // [n_qslots][seen_cap]
  u32 *pset;     // [n_qslots][pset_cap]   distinct index pages touched: hash set, or bitmap (pset_bitmap)
  u64 *pool;     // [n_qslots][K + W]   PQ rerank pool (sorted, <= K kept)
  u32 *stash;     // [n_qslots][stash_cap][R + 1] adjacency lists kept from scoring time (exact mode)
  u32 *stash_tag; // [n_qslots][stash_cap] node id of each stash entry (all ones = empty)
  u32 seen_cap, pset_cap, stash_cap;
  u32 pset_bitmap;   // 1: the page set is a bitmap over index pages (pset_cap words) instead of a hash set
  u32 seen_bitmap;   // 1: the visited set is a bitmap over nodes (seen_cap words) instead of a hash set
  const void *queries;
  u32 *out_ids;
  void *out_dists;
  u32 *out_pages;
  u32 *out_counters;
  Ctl *ctl;
  u64 timeout_ns;
  u64 census_ns;   // debug: take a state census this long after the kernel started (0 = never)
  u32 max_iters;
  u32 idle_ns;       // longest sleep of an idle warp between looks at the work counters
  u32 pullers;       // blocks 0 .. pullers-1 (one per SM) give their last warp to pulling pages, in ring order;
                     // worker warps then pull none.  0: the shared scheme (worker warps take the pulls)
  u32 max_in_flight; // cap on posted-but-not-arrived requests
  u32 vec128;      // 1: vectors are whole 16-byte chunks (<= 24) and query rows are 16-byte aligned
  u32 blocking;    // 1: a warp waits in place for its query's pages instead of yielding
  u32 prof;        // debug: 1 = account warp time per query phase step in stats[S_P_*]
  u32 dma_fill;    // 1: the proxy fills slots with the copy engine and publishes a completion only after
                   //    the copy has landed: no warp copies pages and `filled` is not used
  u32 resident_fast; // 1 (needs identity): a warp runs each query from admission to output without parking it;
                   //    list in registers, candidates in shared memory (device/resident.cuh)
  u32 identity;    // 1: every unit is resident in the slot of the same number and nothing can be
                   //    evicted (whole index preloaded): lookups and hit validation are skipped
};

// launchers implemented in search_kernels.cu
cudaError_t preload_kernels();
cudaError_t launch_init(const Ctx &c, cudaStream_t s);
cudaError_t launch_search(const Ctx &c, u32 blocks, u32 warps_per_block, cudaStream_t s);
cudaError_t search_occupancy(const Ctx &c, u32 warps_per_block, int *blocks_per_sm);
size_t search_smem_per_warp(const Ctx &c);
cudaError_t launch_cache_reset(const Ctx &c, u32 preloaded_pages, cudaStream_t s);
cudaError_t launch_link_probe(const u8 *host_pages, u32 n_pages, u32 n_pulls, u32 warps, u32 sequential, u8 *scratch,
                              u32 *next, u32 *sink, cudaStream_t s);

}  // namespace gorio
