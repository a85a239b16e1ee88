/*
 * CPU oracle for paged graph beam search -- TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition that the CUDA path is checked against.
 * Only tests, the smoke check and the benchmark's cpu_baseline leg may build or call
 * it; the product path never does, and the two share no code.
 *
 * What it computes.  The paper (Section 2.2) describes graph ANNS only as a loop of
 * four activities -- node expansion, distance evaluation, candidate-queue update and
 * discovery of the pages needed next -- on a DiskANN-style index (Section 5.1) and
 * gives no further definition.  The reading implemented here is the standard
 * best-first beam search of width W over a bounded sorted list of size L:
 *
 *   dist(q,x)  = sum_i (q_i - x_i)^2      uint8: exact unsigned 32-bit integers
 *                                         fp32 : differences and sum in double,
 *                                                in index order
 *   key(v)     = (dist(q,v), v), compared lexicographically, smaller is better
 *   page(v)    = v / npp; node bytes start at (v % npp) * node_bytes in the page
 *   node       = vector[d] | degree u32 | R neighbour ids u32 (0xFFFFFFFF unused)
 *
 *   1. seen = {s}; P = {page(s)}; list = [(key(s), unexpanded)]     (s = entry)
 *   2. F = the first min(W, #unexpanded) unexpanded list entries in key order;
 *      stop if F is empty; mark all of F expanded before anything is inserted
 *   3. for u in F: P += page(u); read nbrs(u).  C = (union of nbrs(u)) \ seen
 *   4. for v in C: seen += v; P += page(v); read v's vector; compute key(v)
 *   5. list = the L smallest keys of list + {(key(v), unexpanded) : v in C}; goto 2
 *   6. output the first K list entries; counters: |P|, iterations, sum |F|, |seen|,
 *      sum of degree(u) over expanded u
 *
 * PQ navigation (32 x 256 product quantiser with uint8 centroids, codes resident):
 *   LUT[m][c] = sum_j (q[m*dsub+j] - cent[m][c][j])^2,  adc(v) = sum_m LUT[m][code[v][m]]
 *   same loop with key (adc(v), v); steps 1 and 4 touch no page; step 3 reads u's
 *   page, computes the exact dist(q,u) and appends (dist(q,u), u) to a pool; the output
 *   is the first K of the pool sorted by (exact distance, id), and P holds only the
 *   pages of expanded nodes.
 *
 * Parity pins (see tests): closed-form distances, a hand-worked 8-node ring,
 * brute-force exact kNN when L covers every reachable node, complete graphs, an
 * independent set-form restatement, order independence, the integer ADC identity.
 * Page-hit / miss / fetch counts of the cached GPU path are timing dependent and are
 * not defined here: parity unpinned for those (checked by invariants only).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_ERR_ARG 1
#define ORC_ERR_CORRUPT 7
#define ORC_INVALID 0xFFFFFFFFu

typedef struct {
  uint64_t n_nodes;
  uint32_t dim;
  uint32_t dtype;      /* 0 = uint8, 1 = float32 */
  uint32_t max_degree; /* R */
  uint32_t npp;        /* nodes per page */
  uint32_t page_bytes;
  uint32_t entry;
  const uint8_t *pages;
  uint32_t pq_m;            /* 0 = exact navigation */
  uint32_t pq_ksub;         /* 256 */
  const uint8_t *pq_cent;   /* [pq_m][pq_ksub][dim/pq_m] */
  const uint8_t *pq_codes;  /* [n_nodes][pq_m] */
} orc_index;

typedef struct {
  double dist;     /* sort value: exact integer (uint8) or double sum (fp32) */
  uint32_t id;
  uint32_t expanded;
} orc_entry;

static int entry_cmp(const void *a, const void *b) {
  const orc_entry *x = (const orc_entry *)a, *y = (const orc_entry *)b;
  if (x->dist < y->dist) return -1;
  if (x->dist > y->dist) return 1;
  if (x->id < y->id) return -1;
  if (x->id > y->id) return 1;
  return 0;
}

static uint32_t node_bytes_of(const orc_index *ix) {
  uint32_t esz = ix->dtype == 0 ? 1u : 4u;
  return ix->dim * esz + 4u + 4u * ix->max_degree;
}

static const uint8_t *node_ptr(const orc_index *ix, uint32_t v) {
  uint64_t page = v / ix->npp;
  uint64_t off = (uint64_t)(v % ix->npp) * node_bytes_of(ix);
  return ix->pages + page * ix->page_bytes + off;
}

static uint32_t rd_u32(const uint8_t *p) {
  return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24);
}

/* dist(q, x) with x read from v's record in the page store. */
static double exact_dist(const orc_index *ix, const void *q, uint32_t v) {
  const uint8_t *rec = node_ptr(ix, v);
  if (ix->dtype == 0) {
    const uint8_t *qq = (const uint8_t *)q;
    uint32_t s = 0;
    for (uint32_t i = 0; i < ix->dim; i++) {
      int32_t diff = (int32_t)qq[i] - (int32_t)rec[i];
      s += (uint32_t)(diff * diff);
    }
    return (double)s;
  } else {
    const float *qq = (const float *)q;
    double s = 0.0;
    for (uint32_t i = 0; i < ix->dim; i++) {
      float x;
      memcpy(&x, rec + 4u * i, 4);
      double diff = (double)qq[i] - (double)x;
      s += diff * diff;
    }
    return s;
  }
}

static double adc_dist(const orc_index *ix, const uint32_t *lut, uint32_t v) {
  uint32_t s = 0;
  const uint8_t *code = ix->pq_codes + (uint64_t)v * ix->pq_m;
  for (uint32_t m = 0; m < ix->pq_m; m++) s += lut[m * ix->pq_ksub + code[m]];
  return (double)s;
}

static void build_lut(const orc_index *ix, const uint8_t *q, uint32_t *lut) {
  uint32_t dsub = ix->dim / ix->pq_m;
  for (uint32_t m = 0; m < ix->pq_m; m++)
    for (uint32_t c = 0; c < ix->pq_ksub; c++) {
      const uint8_t *cent = ix->pq_cent + ((uint64_t)m * ix->pq_ksub + c) * dsub;
      uint32_t s = 0;
      for (uint32_t j = 0; j < dsub; j++) {
        int32_t diff = (int32_t)q[m * dsub + j] - (int32_t)cent[j];
        s += (uint32_t)(diff * diff);
      }
      lut[m * ix->pq_ksub + c] = s;
    }
}

/* deterministic permutation helpers for the order-independence pin */
static uint32_t lcg(uint32_t *s) { *s = *s * 1664525u + 1013904223u; return *s >> 8; }
static void permute_u32(uint32_t *a, uint32_t n, int order_mode, uint32_t *rs) {
  if (order_mode == 1) {
    for (uint32_t i = 0; i < n / 2; i++) { uint32_t t = a[i]; a[i] = a[n - 1 - i]; a[n - 1 - i] = t; }
  } else if (order_mode == 2) {
    for (uint32_t i = n; i > 1; i--) { uint32_t j = lcg(rs) % i; uint32_t t = a[i - 1]; a[i - 1] = a[j]; a[j] = t; }
  }
}

/* trace record layout per iteration (uint32 words):
 *   [n_frontier, frontier ids..., n_list, then per list entry: dist(as u32, uint8 data only), id, expanded]
 * the list snapshot is taken after step 5 of that iteration. */
static void trace_put(uint32_t *trace, uint64_t cap, uint64_t *pos, uint32_t v) {
  if (trace && *pos < cap) trace[*pos] = v;
  (*pos)++;
}

/*
 * Search queries [q_begin, q_end).  Outputs are indexed by absolute query number.
 *   out_ids   [nq][K] u32 ; out_dists [nq][K] (u32 for uint8 data, f32 for fp32 data)
 *   counters  [nq][5] u32 : pages_distinct, n_iter, n_expand, n_eval, sum_deg (may be NULL)
 *   page_union: n_pages bytes, set to 1 for every page any searched query touched (may be NULL)
 *   order_mode: 0 natural, 1 reversed, 2 shuffled processing order of F and C
 *   trace/trace_cap/trace_len: optional per-iteration trace (single-query use)
 */
int orc_search(const orc_index *ix, const void *queries, uint32_t q_begin, uint32_t q_end,
               uint32_t K, uint32_t L, uint32_t W, uint32_t *out_ids, void *out_dists,
               uint32_t *counters, uint8_t *page_union, int order_mode,
               uint32_t *trace, uint64_t trace_cap, uint64_t *trace_len) {
  if (!ix || !queries || !out_ids || !out_dists) return ORC_ERR_ARG;
  if (K < 1 || K > L || W < 1 || ix->npp < 1 || ix->entry >= ix->n_nodes) return ORC_ERR_ARG;
  if ((uint64_t)ix->npp * node_bytes_of(ix) > ix->page_bytes) return ORC_ERR_ARG;
  const int pq = ix->pq_m != 0;
  if (pq && (ix->dtype != 0 || ix->dim % ix->pq_m != 0 || !ix->pq_cent || !ix->pq_codes)) return ORC_ERR_ARG;

  const uint64_t N = ix->n_nodes;
  const uint32_t R = ix->max_degree;
  const uint64_t n_pages = (N + ix->npp - 1) / ix->npp;
  const uint32_t esz = ix->dtype == 0 ? 1u : 4u;
  const uint64_t qstride = (uint64_t)ix->dim * esz;
  int rc = ORC_OK;
  uint64_t tpos = 0;
  uint32_t rs = 12345u;

  uint8_t *seen = (uint8_t *)malloc(N);
  uint8_t *pset = (uint8_t *)malloc(n_pages);
  orc_entry *list = (orc_entry *)malloc(sizeof(orc_entry) * ((size_t)L + (size_t)W * R + 1));
  uint32_t *front = (uint32_t *)malloc(sizeof(uint32_t) * W);
  uint32_t *cand = (uint32_t *)malloc(sizeof(uint32_t) * ((size_t)W * R + 1));
  uint32_t *lut = pq ? (uint32_t *)malloc(sizeof(uint32_t) * ix->pq_m * ix->pq_ksub) : NULL;
  orc_entry *pool = NULL;
  size_t pool_cap = 0;
  if (!seen || !pset || !list || !front || !cand || (pq && !lut)) { rc = ORC_ERR_ARG; goto done; }

  for (uint32_t qi = q_begin; qi < q_end; qi++) {
    const void *q = (const uint8_t *)queries + qi * qstride;
    memset(seen, 0, N);
    memset(pset, 0, n_pages);
    uint32_t pages_distinct = 0, n_iter = 0, n_expand = 0, n_eval = 0, sum_deg = 0;
    size_t n_list = 0, n_pool = 0;
    if (pq) build_lut(ix, (const uint8_t *)q, lut);

    /* step 1 */
    uint32_t s = ix->entry;
    seen[s] = 1; n_eval = 1;
    if (!pq) {
      pset[s / ix->npp] = 1; pages_distinct = 1;
      list[0].dist = exact_dist(ix, q, s);
    } else {
      list[0].dist = adc_dist(ix, lut, s);
    }
    list[0].id = s; list[0].expanded = 0; n_list = 1;

    for (;;) {
      /* step 2: frontier */
      uint32_t nf = 0;
      for (size_t i = 0; i < n_list && nf < W; i++)
        if (!list[i].expanded) front[nf++] = (uint32_t)i;
      if (nf == 0) break;
      for (uint32_t f = 0; f < nf; f++) { list[front[f]].expanded = 1; front[f] = list[front[f]].id; }
      n_iter++; n_expand += nf;
      permute_u32(front, nf, order_mode, &rs);
      trace_put(trace, trace_cap, &tpos, nf);
      for (uint32_t f = 0; f < nf; f++) trace_put(trace, trace_cap, &tpos, front[f]);

      /* step 3: read adjacency, collect unseen neighbours */
      uint32_t nc = 0;
      for (uint32_t f = 0; f < nf; f++) {
        uint32_t u = front[f];
        uint32_t pg = u / ix->npp;
        if (!pset[pg]) { pset[pg] = 1; pages_distinct++; }
        const uint8_t *rec = node_ptr(ix, u);
        uint32_t deg = rd_u32(rec + qstride);
        if (deg > R) { rc = ORC_ERR_CORRUPT; goto done; }
        sum_deg += deg;
        if (pq) {
          if (n_pool == pool_cap) {
            pool_cap = pool_cap ? pool_cap * 2 : 256;
            pool = (orc_entry *)realloc(pool, sizeof(orc_entry) * pool_cap);
            if (!pool) { rc = ORC_ERR_ARG; goto done; }
          }
          pool[n_pool].dist = exact_dist(ix, q, u);
          pool[n_pool].id = u; pool[n_pool].expanded = 1; n_pool++;
        }
        for (uint32_t j = 0; j < deg; j++) {
          uint32_t v = rd_u32(rec + qstride + 4u + 4u * j);
          if (v >= N) { rc = ORC_ERR_CORRUPT; goto done; }
          if (!seen[v]) { seen[v] = 1; cand[nc++] = v; }   /* seen doubles as the set-union */
        }
      }
      permute_u32(cand, nc, order_mode, &rs);

      /* step 4: evaluate */
      for (uint32_t c = 0; c < nc; c++) {
        uint32_t v = cand[c];
        n_eval++;
        if (!pq) {
          uint32_t pg = v / ix->npp;
          if (!pset[pg]) { pset[pg] = 1; pages_distinct++; }
          list[n_list].dist = exact_dist(ix, q, v);
        } else {
          list[n_list].dist = adc_dist(ix, lut, v);
        }
        list[n_list].id = v; list[n_list].expanded = 0; n_list++;
      }
      /* step 5: keep the L smallest keys */
      qsort(list, n_list, sizeof(orc_entry), entry_cmp);
      if (n_list > L) n_list = L;

      trace_put(trace, trace_cap, &tpos, (uint32_t)n_list);
      for (size_t i = 0; i < n_list; i++) {
        trace_put(trace, trace_cap, &tpos, (uint32_t)list[i].dist);
        trace_put(trace, trace_cap, &tpos, list[i].id);
        trace_put(trace, trace_cap, &tpos, list[i].expanded);
      }
    }

    /* step 6: output */
    const orc_entry *res = list; size_t n_res = n_list;
    if (pq) { qsort(pool, n_pool, sizeof(orc_entry), entry_cmp); res = pool; n_res = n_pool; }
    for (uint32_t k = 0; k < K; k++) {
      uint64_t o = (uint64_t)qi * K + k;
      if (k < n_res) {
        out_ids[o] = res[k].id;
        if (ix->dtype == 0) ((uint32_t *)out_dists)[o] = (uint32_t)res[k].dist;
        else ((float *)out_dists)[o] = (float)res[k].dist;
      } else {
        out_ids[o] = ORC_INVALID;
        if (ix->dtype == 0) ((uint32_t *)out_dists)[o] = ORC_INVALID;
        else { uint32_t inf = 0x7F800000u; memcpy(&((float *)out_dists)[o], &inf, 4); }
      }
    }
    if (counters) {
      uint32_t *c = counters + (uint64_t)qi * 5;
      c[0] = pages_distinct; c[1] = n_iter; c[2] = n_expand; c[3] = n_eval; c[4] = sum_deg;
    }
    if (page_union) for (uint64_t p = 0; p < n_pages; p++) if (pset[p]) page_union[p] = 1;
  }

done:
  if (trace_len) *trace_len = tpos;
  free(seen); free(pset); free(list); free(front); free(cand); free(lut); free(pool);
  return rc;
}

/* dist(q, node v) exposed for the distance pins. */
double orc_exact_dist(const orc_index *ix, const void *q, uint32_t v) { return exact_dist(ix, q, v); }

/* adc(v) for query q (uint8) exposed for the integer ADC identity pin. */
uint32_t orc_adc_dist(const orc_index *ix, const uint8_t *q, uint32_t v) {
  uint32_t *lut = (uint32_t *)malloc(sizeof(uint32_t) * ix->pq_m * ix->pq_ksub);
  build_lut(ix, q, lut);
  uint32_t r = (uint32_t)adc_dist(ix, lut, v);
  free(lut);
  return r;
}
