/*
 * CPU oracle for the retrieve + Chunked-RoPE KV-injection path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is compared against.  It shares no code, header, table or
 * constant with the CUDA path and must never be called from the product path;
 * only the tests, the smoke check and the CPU-baseline leg of the benchmark
 * may load it.
 *
 * Everything is computed in double precision, one pass, no blocking, no
 * fusion.  The optional OpenMP pragmas only split the outermost independent
 * loop (facts, or tokens); they do not change any value.
 *
 * What follows which passage of the paper:
 *   - scoring / top-k:  "Persistent memory store and retrieval" (Sec. 3.2):
 *     a top-k search by inner product over the fact embeddings that returns
 *     fact ids.  Exact search replaces the graph index; ties go to the lower id.
 *   - RoPE:             "Rotary position embeddings" (Sec. 2.4) and the proof
 *     sketch of Theorem 2 (Chunked RoPE Injection): a block-diagonal rotation
 *     R_p with one frequency per 2-d pair, applied after the key projection.
 *   - positions:        "Position policy" (Sec. 5.2): facts are contiguous,
 *     fact i starts at b_i = sum_{j<i} |C_j|, total m = sum_i |C_i|.
 *   - paged placement:  "Paged attention and KV cache management" (Sec. 2.2)
 *     and the worker side of the connector (Sec. 3.4): a token at position
 *     pos lives in slot block_table[pos / bs] * bs + pos % bs.
 *   - V is stored raw and copied unchanged (Sec. 5.1, closing paragraph).
 *   - bytes per fact:   "Storage cost" (Sec. 3.5): 2 * L * c * h * d * b.
 *
 *   - graph index:      "Jasper: a GPU-native vector index" (Sec. 2.5) and the index parameters of the
 *     evaluation setup (Sec. 6.1): a proximity graph searched by a beam search; the concrete algorithm is
 *     fixed in the comment above oracle_ann_search.
 *   - variants beyond the paper's text (its evaluation spans "RoPE parameterizations", Sec. 6.1): the
 *     Llama-3.1 rescaled frequency table, rotation of only the first R coordinates of a head, and an
 *     8-bit e4m3 cache image with per-tensor scales.
 *
 * Parity pins: every exported function is pinned by the CPU tests
 * (closed forms, group law, brute-force joint rotation, numpy float64
 * cross-checks, full-sort comparison, exhaustive e4m3 code tables, torch's
 * float32 division and float8 cast over every bf16 value, planted decision
 * margins of the graph search); none is "parity unpinned".  One function is
 * not an independent definition and says so: score_f32_lanes.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG -1
#define ORACLE_ERR_BLOCK_TABLE -2 /* position needs a block-table entry that is not there */
#define ORACLE_ERR_BLOCK_ID -3    /* block id outside the pool */
#define ORACLE_ERR_FACT_ID -4     /* id outside the fact table */
#define ORACLE_ERR_NOMEM -5

enum { ORACLE_F32 = 0, ORACLE_F16 = 1 };

/* ---------------------------------------------------------------- number formats */

/* IEEE binary16 -> double, exact. */
static double f16_to_double(uint16_t h) {
  int sign = (h >> 15) & 1;
  int exp = (h >> 10) & 0x1f;
  int man = h & 0x3ff;
  double v;
  if (exp == 0) {
    v = ldexp((double)man, -24); /* subnormal: man * 2^-10 * 2^-14 */
  } else if (exp == 31) {
    v = man ? NAN : INFINITY;
  } else {
    v = ldexp((double)(man | 0x400), exp - 25); /* (1024+man) * 2^(exp-15-10) */
  }
  return sign ? -v : v;
}

/* bfloat16 -> double, exact (bfloat16 is the upper half of a binary32). */
static double bf16_to_double(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

/* double -> bfloat16 with ONE round-to-nearest-even (no intermediate float). */
static uint16_t double_to_bf16_rne(double x) {
  if (isnan(x)) return 0x7fc0;
  uint16_t sign = signbit(x) ? 0x8000 : 0;
  double a = fabs(x);
  if (isinf(a)) return sign | 0x7f80;
  if (a == 0.0) return sign;
  int e;
  (void)frexp(a, &e);       /* a = f * 2^e, f in [0.5, 1): leading bit has weight 2^(e-1) */
  int lead = e - 1;
  if (lead < -126) lead = -126; /* subnormal range of bfloat16 shares the quantum of 2^-126 */
  double quantum = ldexp(1.0, lead - 7); /* 8 significant bits */
  double q = nearbyint(a / quantum);     /* default rounding mode: ties to even */
  double y = q * quantum;
  float f = (float)y; /* exact: y has at most 8 significant bits */
  if (isinf(f) || y >= ldexp(1.0, 128)) return sign | 0x7f80;
  uint32_t u;
  memcpy(&u, &f, 4);
  return sign | (uint16_t)(u >> 16);
}

/*
 * 8-bit float "e4m3" as used for quantised KV caches: 1 sign, 4 exponent bits (bias 7), 3 mantissa bits, no
 * infinities, exponent 15 with mantissa 7 is NaN, so the largest finite value is 1.75 * 2^8 = 448; subnormals are
 * multiples of 2^-9.  Decoding is exact.
 */
static double e4m3_to_double(uint8_t c) {
  int e = (c >> 3) & 15, m = c & 7;
  double v;
  if (e == 15 && m == 7) return NAN;
  v = e == 0 ? ldexp((double)m, -9) : ldexp(1.0 + (double)m / 8.0, e - 7);
  return (c & 0x80) ? -v : v;
}

/* double -> e4m3, round to nearest even in ONE step, saturating to +-448 (no NaN is produced from a finite input). */
static uint8_t double_to_e4m3_rne_sat(double x) {
  uint8_t sign = signbit(x) ? 0x80 : 0;
  double a = fabs(x);
  int e;
  double q;
  if (isnan(x)) return 0x7f;
  if (a >= 448.0) return (uint8_t)(sign | 0x7e);
  if (a < ldexp(1.0, -6)) {            /* subnormal range: spacing 2^-9 */
    q = rint(ldexp(a, 9));             /* 0..8, ties to even */
    return (uint8_t)(sign | (uint8_t)q); /* q == 8 is the code of the smallest normal, 2^-6 */
  }
  (void)frexp(a, &e);                  /* a = f * 2^e, f in [0.5, 1)  ->  a in [2^(e-1), 2^e) */
  e -= 1;
  q = rint((ldexp(a, -e) - 1.0) * 8.0); /* 0..8 */
  if (q == 8.0) {
    q = 0.0;
    e += 1;
  }
  return (uint8_t)(sign | (uint8_t)(((e + 7) << 3) | (int)q));
}

/* A bf16 value divided by a per-tensor scale in binary32 (one correctly rounded IEEE division), then rounded once to e4m3. */
static uint8_t e4m3_of_scaled_bf16(uint16_t b, float scale) {
  volatile float x = (float)bf16_to_double(b); /* exact */
  volatile float q = x / scale;                /* binary32 division; volatile keeps it out of wider registers */
  return double_to_e4m3_rne_sat((double)q);
}

/* The 8-bit cache code of each bf16 value under a per-tensor scale (the rule of oracle_inject_ex). */
void oracle_e4m3_from_scaled_bf16(const uint16_t* x, int64_t n, float scale, uint8_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = e4m3_of_scaled_bf16(x[i], scale);
}

void oracle_e4m3_from_double(const double* x, int64_t n, uint8_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = double_to_e4m3_rne_sat(x[i]);
}
void oracle_e4m3_to_double(const uint8_t* x, int64_t n, double* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = e4m3_to_double(x[i]);
}

void oracle_bf16_from_double(const double* x, int64_t n, uint16_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = double_to_bf16_rne(x[i]);
}
void oracle_bf16_to_double(const uint16_t* x, int64_t n, double* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = bf16_to_double(x[i]);
}
void oracle_f16_to_double(const uint16_t* x, int64_t n, double* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = f16_to_double(x[i]);
}

static void set_threads(int n_threads) {
#ifdef _OPENMP
  if (n_threads > 0) omp_set_num_threads(n_threads);
#else
  (void)n_threads;
#endif
}
int oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ---------------------------------------------------------------- storage cost */

/* Sec. 3.5: a fact of c tokens stores 2 * L * c * h * d * b bytes of KV. */
int64_t oracle_kv_bytes(int64_t L, int64_t c, int64_t h, int64_t d, int64_t b) {
  return 2 * L * c * h * d * b;
}

/* ---------------------------------------------------------------- retrieval */

static double emb_at(const void* emb, int dtype, int64_t idx) {
  if (dtype == ORACLE_F32) return (double)((const float*)emb)[idx];
  return f16_to_double(((const uint16_t*)emb)[idx]);
}

/* s[f] = sum_d q[d] * emb[f][d], accumulated left to right in double. */
int oracle_scores(const void* emb, int emb_dtype, int64_t n_facts, int emb_dim, const void* query,
                  double* out_scores, int n_threads) {
  if (!emb || !query || !out_scores || n_facts < 0 || emb_dim <= 0) return ORACLE_ERR_ARG;
  if (emb_dtype != ORACLE_F32 && emb_dtype != ORACLE_F16) return ORACLE_ERR_ARG;
  set_threads(n_threads);
#pragma omp parallel for schedule(static)
  for (int64_t f = 0; f < n_facts; ++f) {
    double s = 0.0;
    for (int d = 0; d < emb_dim; ++d) s += emb_at(query, emb_dtype, d) * emb_at(emb, emb_dtype, f * emb_dim + d);
    out_scores[f] = s;
  }
  return ORACLE_OK;
}

typedef struct {
  double s;
  int32_t id;
} scored_t;

static int cmp_scored(const void* a, const void* b) {
  const scored_t* x = (const scored_t*)a;
  const scored_t* y = (const scored_t*)b;
  if (x->s > y->s) return -1; /* higher score first */
  if (x->s < y->s) return 1;
  if (x->id < y->id) return -1; /* equal score: lower id first */
  if (x->id > y->id) return 1;
  return 0;
}

/*
 * For each of nq queries: score every fact, sort ALL facts by (score desc, id asc),
 * return the first k ids and their scores rounded to float; pad with id -1 / score 0
 * when there are fewer than k facts.  row_ids[f] is the fact id of embedding row f
 * (NULL: the row index is the id).
 */
int oracle_retrieve_masked(const void* emb, int emb_dtype, int64_t n_facts, int emb_dim, const int32_t* row_ids,
                           const uint8_t* removed, const void* queries, int nq, int k, int32_t* out_ids, float* out_scores,
                           int n_threads);

int oracle_retrieve(const void* emb, int emb_dtype, int64_t n_facts, int emb_dim, const int32_t* row_ids,
                    const void* queries, int nq, int k, int32_t* out_ids, float* out_scores, int n_threads) {
  return oracle_retrieve_masked(emb, emb_dtype, n_facts, emb_dim, row_ids, NULL, queries, nq, k, out_ids, out_scores, n_threads);
}

/*
 * The same with removed facts (the paper names deleting and revising facts as future work, "with consistent updates to
 * both the index and the pre-RoPE KV store"; the rule here is the plain one): removed[f] != 0 takes row f out of the
 * search - it is never returned, whatever its score - and everything else is as before: the facts that remain are
 * sorted by (score desc, id asc), the first k are returned, -1 / 0 pad when fewer remain.
 */
int oracle_retrieve_masked(const void* emb, int emb_dtype, int64_t n_facts, int emb_dim, const int32_t* row_ids,
                           const uint8_t* removed, const void* queries, int nq, int k, int32_t* out_ids, float* out_scores,
                           int n_threads) {
  if (nq < 0 || k < 0 || !out_ids) return ORACLE_ERR_ARG;
  if (n_facts > 0 && (!emb || !queries)) return ORACLE_ERR_ARG;
  size_t esz = emb_dtype == ORACLE_F32 ? 4 : 2;
  double* s = (double*)malloc(sizeof(double) * (size_t)(n_facts > 0 ? n_facts : 1));
  scored_t* all = (scored_t*)malloc(sizeof(scored_t) * (size_t)(n_facts > 0 ? n_facts : 1));
  if (!s || !all) {
    free(s);
    free(all);
    return ORACLE_ERR_NOMEM;
  }
  for (int q = 0; q < nq; ++q) {
    if (n_facts > 0) {
      int rc = oracle_scores(emb, emb_dtype, n_facts, emb_dim, (const char*)queries + (size_t)q * emb_dim * esz, s,
                             n_threads);
      if (rc != ORACLE_OK) {
        free(s);
        free(all);
        return rc;
      }
    }
    int64_t n_left = 0;
    for (int64_t f = 0; f < n_facts; ++f) {
      if (removed && removed[f]) continue;
      all[n_left].s = s[f];
      all[n_left].id = row_ids ? row_ids[f] : (int32_t)f;
      ++n_left;
    }
    qsort(all, (size_t)n_left, sizeof(scored_t), cmp_scored);
    for (int r = 0; r < k; ++r) {
      if (r < n_left) {
        out_ids[(size_t)q * k + r] = all[r].id;
        if (out_scores) out_scores[(size_t)q * k + r] = (float)all[r].s;
      } else {
        out_ids[(size_t)q * k + r] = -1;
        if (out_scores) out_scores[(size_t)q * k + r] = 0.0f;
      }
    }
  }
  free(s);
  free(all);
  return ORACLE_OK;
}

/* ---------------------------------------------------------------- graph index (approximate retrieval) */

/*
 * The paper retrieves with a GPU-resident proximity-graph index searched by a beam search (Sec. 2.5; Sec. 6.1:
 * inner-product distance, 64 graph neighbours, beam width 64) and does not print the index's algorithm.  The
 * algorithm fixed here, step by step, is the one this oracle and the library both follow:
 *
 *   graph    G[n][deg]: row r lists the deg rows with the largest inner product with row r, r itself
 *            excluded, best first, ties to the lower row (an exact k-nearest-neighbour graph); -1 pads.
 *   scores   inner products.  oracle_ann_search_exact ranks by the plain double sums and reports the smallest
 *            score difference that decided anything; oracle_ann_search ranks by binary32 sums taken in one stated
 *            order (score_f32_lanes), for the cases whose decisions are closer than binary32 rounding.
 *   list     at most L = max(beam, k) entries (score, row, expanded?), ordered by score descending, ties to
 *            the lower row; V = the set of rows ever scored.
 *   start    rows e_i = ((i + 1) * 2654435761) mod n, i < n_entry (duplicates dropped), scored and listed.
 *   step     take the first `parents` unexpanded entries of the list in list order (stop when there is none, or
 *            after max_iters steps), mark them expanded; collect their neighbours that are valid rows and
 *            not in V, add them to V, score them, and keep the best L of list + new.
 *   result   the first k entries of the list; -1 / 0 pads.  With removed rows: they walk along like any other row
 *            (scored, listed, expanded) and are passed over when the result is read out.
 */

/*
 * NOT an independent definition: this order restates the summation schedule of the CUDA scoring kernels, so that a
 * search whose decisions hinge on the last bits of a binary32 sum can still be followed.  It is pinned by rounding
 * behaviour built into test inputs and, through the search, against oracle_ann_search_exact wherever the margin of
 * that search exceeds binary32 rounding.
 * Inner product in binary32 with a fixed order: the row is cut into vectors of 16 bytes (8 halves or 4
 * floats); vector v belongs to "lane" v mod 32; a lane adds its products one fused multiply-add at a time in
 * increasing element order; the 32 lane sums are then combined by a butterfly (lane l adds lane l xor 16,
 * then xor 8, 4, 2, 1).  Every lane ends with the same value.
 */
static float score_f32_lanes(const void* emb, int dtype, int64_t row, int dim, const void* query) {
  int vec = dtype == ORACLE_F32 ? 4 : 8;
  int nvec = dim / vec;
  float acc[32], tmp[32];
  for (int l = 0; l < 32; ++l) acc[l] = 0.0f;
  for (int v0 = 0; v0 < nvec; v0 += 128)
    for (int l = 0; l < 32; ++l)
      for (int u = 0; u < 4; ++u) {
        int v = v0 + u * 32 + l;
        if (v >= nvec) continue;
        for (int i = 0; i < vec; ++i) {
          float a = (float)emb_at(emb, dtype, row * dim + (int64_t)v * vec + i);
          float b = (float)emb_at(query, dtype, (int64_t)v * vec + i);
          acc[l] = fmaf(a, b, acc[l]);
        }
      }
  for (int o = 16; o > 0; o >>= 1) {
    for (int l = 0; l < 32; ++l) tmp[l] = acc[l] + acc[l ^ o];
    for (int l = 0; l < 32; ++l) acc[l] = tmp[l];
  }
  return acc[0] + 0.0f; /* -0 becomes +0 */
}

int oracle_scores_f32(const void* emb, int emb_dtype, int64_t n_rows, int emb_dim, const void* query, float* out) {
  if (!emb || !query || !out || emb_dim <= 0 || emb_dim % 8) return ORACLE_ERR_ARG;
  for (int64_t r = 0; r < n_rows; ++r) out[r] = score_f32_lanes(emb, emb_dtype, r, emb_dim, query);
  return ORACLE_OK;
}

/* Exact k-nearest-neighbour graph by inner product (double scores, full sort per row). */
int oracle_knn_graph_masked(const void* emb, int emb_dtype, int64_t n, int emb_dim, int deg, const uint8_t* removed, int32_t* out_graph,
                            int n_threads);
int oracle_knn_graph(const void* emb, int emb_dtype, int64_t n, int emb_dim, int deg, int32_t* out_graph, int n_threads) {
  return oracle_knn_graph_masked(emb, emb_dtype, n, emb_dim, deg, NULL, out_graph, n_threads);
}
/* A graph built after removals: removed rows are nobody's neighbours (a removed row still gets a list of its own, so
 * that a walk that reaches it through an older edge can go on). */
int oracle_knn_graph_masked(const void* emb, int emb_dtype, int64_t n, int emb_dim, int deg, const uint8_t* removed, int32_t* out_graph,
                            int n_threads) {
  if (!emb || !out_graph || n < 0 || deg <= 0 || emb_dim <= 0) return ORACLE_ERR_ARG;
  size_t esz = emb_dtype == ORACLE_F32 ? 4 : 2;
  int rc_all = ORACLE_OK;
  set_threads(n_threads);
#pragma omp parallel for schedule(dynamic, 8)
  for (int64_t r = 0; r < n; ++r) {
    scored_t* all = (scored_t*)malloc(sizeof(scored_t) * (size_t)n);
    if (!all) {
      rc_all = ORACLE_ERR_NOMEM;
      continue;
    }
    const char* q = (const char*)emb + (size_t)r * emb_dim * esz;
    int64_t m = 0;
    for (int64_t f = 0; f < n; ++f) {
      if (f == r || (removed && removed[f])) continue;
      double sc = 0.0;
      for (int d = 0; d < emb_dim; ++d) sc += emb_at(q, emb_dtype, d) * emb_at(emb, emb_dtype, f * emb_dim + d);
      all[m].s = sc;
      all[m].id = (int32_t)f;
      ++m;
    }
    qsort(all, (size_t)m, sizeof(scored_t), cmp_scored);
    for (int j = 0; j < deg; ++j) out_graph[r * deg + j] = j < m ? all[j].id : -1;
    free(all);
  }
  return rc_all;
}

/*
 * Growing the graph when rows n_old .. n-1 have been appended to the store (the paper lists online insertion as future
 * work; the rule fixed here is the usual one for incremental neighbour graphs):
 *   - a new row gets its exact list over all n rows, like any row of a fresh graph;
 *   - an old row nb is offered every new row that lists nb among its own neighbours; its list becomes the best deg
 *     of (old list + offers) by inner product with nb, best first, ties to the lower row.  Old rows that nobody
 *     offers anything keep their list.  (A fresh build could differ: it would also give nb a new row that does
 *     not list nb back.)
 * Scores in double, full sorts.  old_graph [n_old][deg], out_graph [n][deg].
 */
int oracle_graph_append(const void* emb, int emb_dtype, int64_t n_old, int64_t n, int emb_dim, const int32_t* old_graph,
                        int deg, int32_t* out_graph, int n_threads) {
  if (!emb || !out_graph || n_old < 0 || n < n_old || deg <= 0 || emb_dim <= 0 || (n_old > 0 && !old_graph)) return ORACLE_ERR_ARG;
  size_t esz = emb_dtype == ORACLE_F32 ? 4 : 2;
  int rc_all = ORACLE_OK;
  set_threads(n_threads);
  /* new rows: exact lists over everything */
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t r = n_old; r < n; ++r) {
    scored_t* all = (scored_t*)malloc(sizeof(scored_t) * (size_t)n);
    if (!all) {
      rc_all = ORACLE_ERR_NOMEM;
      continue;
    }
    const char* q = (const char*)emb + (size_t)r * emb_dim * esz;
    int64_t m = 0;
    for (int64_t f = 0; f < n; ++f) {
      if (f == r) continue;
      double sc = 0.0;
      for (int d = 0; d < emb_dim; ++d) sc += emb_at(q, emb_dtype, d) * emb_at(emb, emb_dtype, f * emb_dim + d);
      all[m].s = sc;
      all[m].id = (int32_t)f;
      ++m;
    }
    qsort(all, (size_t)m, sizeof(scored_t), cmp_scored);
    for (int j = 0; j < deg; ++j) out_graph[r * deg + j] = j < m ? all[j].id : -1;
    free(all);
  }
  if (rc_all != ORACLE_OK) return rc_all;
  /* old rows: old list plus the new rows that list them */
  int64_t n_add = n - n_old;
  scored_t* cand = (scored_t*)malloc(sizeof(scored_t) * (size_t)(deg + n_add + 1));
  if (!cand) return ORACLE_ERR_NOMEM;
  for (int64_t nb = 0; nb < n_old; ++nb) {
    const char* q = (const char*)emb + (size_t)nb * emb_dim * esz;
    int64_t m = 0, offers = 0;
    for (int j = 0; j < deg; ++j) {
      int32_t f = old_graph[nb * deg + j];
      if (f < 0 || f >= n_old) continue;
      cand[m++].id = f;
    }
    for (int64_t r = n_old; r < n; ++r)
      for (int j = 0; j < deg; ++j)
        if (out_graph[r * deg + j] == nb) {
          cand[m++].id = (int32_t)r;
          ++offers;
          break;
        }
    if (offers == 0) {
      for (int j = 0; j < deg; ++j) out_graph[nb * deg + j] = old_graph[nb * deg + j];
      continue;
    }
    for (int64_t i = 0; i < m; ++i) {
      double sc = 0.0;
      for (int d = 0; d < emb_dim; ++d) sc += emb_at(q, emb_dtype, d) * emb_at(emb, emb_dtype, (int64_t)cand[i].id * emb_dim + d);
      cand[i].s = sc;
    }
    qsort(cand, (size_t)m, sizeof(scored_t), cmp_scored);
    for (int j = 0; j < deg; ++j) out_graph[nb * deg + j] = j < m ? cand[j].id : -1;
  }
  free(cand);
  return ORACLE_OK;
}

typedef struct {
  double s; /* the score the search ranks by: a double sum, or a binary32 sum held exactly in a double */
  int32_t row;
  int32_t expanded;
} beam_t;

static int cmp_beam(const void* a, const void* b) {
  const beam_t* x = (const beam_t*)a;
  const beam_t* y = (const beam_t*)b;
  if (x->s > y->s) return -1;
  if (x->s < y->s) return 1;
  if (x->row < y->row) return -1;
  if (x->row > y->row) return 1;
  return 0;
}

/* Score of `row` for the search: the plain double sum (exact = 1) or the binary32 lane sum (exact = 0). */
static double search_score(const void* emb, int dtype, int64_t row, int dim, const void* query, int exact) {
  if (!exact) return (double)score_f32_lanes(emb, dtype, row, dim, query);
  double s = 0.0;
  for (int d = 0; d < dim; ++d) s += emb_at(query, dtype, d) * emb_at(emb, dtype, row * dim + d);
  return s;
}

/*
 * The comparisons that decide a step are those between neighbours of the sorted list down to the cut at L: they fix
 * the order of the kept entries (hence the parents of the next step and the result) and which entry is the first one
 * dropped.  The smallest score difference among them is the margin by which this step would survive another
 * arithmetic.  Two rows with identical embedding bytes score alike in any arithmetic and are ordered by row: their
 * pair is no decision.
 */
static double step_margin(const beam_t* list, int len, int L, const void* emb, size_t row_bytes, double margin) {
  for (int i = 0; i < L && i + 1 < len; ++i) {
    double gap = list[i].s - list[i + 1].s;
    if (gap >= margin) continue;
    if (memcmp((const char*)emb + (size_t)list[i].row * row_bytes, (const char*)emb + (size_t)list[i + 1].row * row_bytes,
               row_bytes) == 0)
      continue;
    margin = gap;
  }
  return margin;
}

static int ann_search_core(const void* emb, int emb_dtype, int64_t n, int emb_dim, const int32_t* graph, int deg,
                           const void* query, int k, int beam, int parents, int n_entry, int max_iters, int exact,
                           const uint8_t* removed, int32_t* out_ids, float* out_scores, int32_t* out_iters,
                           int64_t* out_scored, double* out_margin) {
  if (!out_ids || k <= 0 || beam <= 0 || parents <= 0 || n_entry <= 0 || max_iters < 0 || deg <= 0 || n < 0 ||
      emb_dim <= 0 || emb_dim % 8)
    return ORACLE_ERR_ARG;
  if (n > 0 && (!emb || !graph || !query)) return ORACLE_ERR_ARG;
  int L = beam > k ? beam : k;
  int cap = L + (parents * deg > n_entry ? parents * deg : n_entry);
  size_t row_bytes = (size_t)emb_dim * (emb_dtype == ORACLE_F32 ? 4 : 2);
  beam_t* list = (beam_t*)malloc(sizeof(beam_t) * (size_t)cap);
  unsigned char* seen = (unsigned char*)calloc((size_t)(n > 0 ? n : 1), 1);
  int32_t* chosen = (int32_t*)malloc(sizeof(int32_t) * (size_t)parents);
  if (!list || !seen || !chosen) {
    free(list);
    free(seen);
    free(chosen);
    return ORACLE_ERR_NOMEM;
  }
  int len = 0, iters = 0;
  int64_t scored = 0;
  double margin = INFINITY;
  if (n > 0) {
    for (int i = 0; i < n_entry; ++i) {
      int64_t e = (int64_t)(((uint64_t)(i + 1) * 2654435761ull) % (uint64_t)n);
      if (seen[e]) continue;
      seen[e] = 1;
      list[len].s = search_score(emb, emb_dtype, e, emb_dim, query, exact);
      list[len].row = (int32_t)e;
      list[len].expanded = 0;
      ++len;
      ++scored;
    }
    qsort(list, (size_t)len, sizeof(beam_t), cmp_beam);
    margin = step_margin(list, len, L, emb, row_bytes, margin);
    if (len > L) len = L;
    for (; iters < max_iters; ++iters) {
      int np = 0;
      for (int i = 0; i < len && np < parents; ++i)
        if (!list[i].expanded) {
          list[i].expanded = 1;
          chosen[np++] = list[i].row;
        }
      if (np == 0) break;
      int added = 0;
      for (int p = 0; p < np; ++p)
        for (int j = 0; j < deg; ++j) {
          int32_t nb = graph[(int64_t)chosen[p] * deg + j];
          if (nb < 0 || nb >= n || seen[nb]) continue;
          seen[nb] = 1;
          list[len + added].s = search_score(emb, emb_dtype, nb, emb_dim, query, exact);
          list[len + added].row = nb;
          list[len + added].expanded = 0;
          ++added;
          ++scored;
        }
      len += added;
      qsort(list, (size_t)len, sizeof(beam_t), cmp_beam);
      margin = step_margin(list, len, L, emb, row_bytes, margin);
      if (len > L) len = L;
    }
  }
  /* result: the first k entries of the list; a removed row takes part in the walk like any other (its edges still lead
   * somewhere) but is passed over here, so it is never returned */
  int w = 0;
  for (int i = 0; i < len && w < k; ++i) {
    if (removed && removed[list[i].row]) continue;
    out_ids[w] = list[i].row;
    if (out_scores) out_scores[w] = (float)list[i].s;
    ++w;
  }
  for (; w < k; ++w) {
    out_ids[w] = -1;
    if (out_scores) out_scores[w] = 0.0f;
  }
  if (out_iters) *out_iters = iters;
  if (out_scored) *out_scored = scored;
  if (out_margin) *out_margin = margin;
  free(list);
  free(seen);
  free(chosen);
  return ORACLE_OK;
}

/*
 * Beam search of one query over the graph, as defined above, ranking by the binary32 lane sums.  out_ids /
 * out_scores [k]; out_iters (optional): steps taken; out_scored (optional): |V|, the number of rows scored.
 */
int oracle_ann_search(const void* emb, int emb_dtype, int64_t n, int emb_dim, const int32_t* graph, int deg,
                      const void* query, int k, int beam, int parents, int n_entry, int max_iters, int32_t* out_ids,
                      float* out_scores, int32_t* out_iters, int64_t* out_scored) {
  return ann_search_core(emb, emb_dtype, n, emb_dim, graph, deg, query, k, beam, parents, n_entry, max_iters, 0, NULL, out_ids,
                         out_scores, out_iters, out_scored, NULL);
}

/*
 * The same search ranking by the plain double-precision inner products of oracle_scores: the definition of the walk
 * with no assumption about the order in which a device adds its products.  out_scores are the double scores
 * rounded to binary32.  out_margin receives the smallest score difference that decided any step (see step_margin;
 * infinity when nothing was ever compared): a search in another arithmetic whose scores are all within less than
 * half of it of the exact ones must take the same walk and return the same rows.
 */
int oracle_ann_search_exact(const void* emb, int emb_dtype, int64_t n, int emb_dim, const int32_t* graph, int deg,
                            const void* query, int k, int beam, int parents, int n_entry, int max_iters, int32_t* out_ids,
                            float* out_scores, int32_t* out_iters, int64_t* out_scored, double* out_margin) {
  return ann_search_core(emb, emb_dtype, n, emb_dim, graph, deg, query, k, beam, parents, n_entry, max_iters, 1, NULL, out_ids,
                         out_scores, out_iters, out_scored, out_margin);
}

/* Both forms with removed rows (removed[row] != 0, or NULL): exact != 0 ranks by the double scores and reports the margin. */
int oracle_ann_search_masked(const void* emb, int emb_dtype, int64_t n, int emb_dim, const int32_t* graph, int deg,
                             const void* query, int k, int beam, int parents, int n_entry, int max_iters, int exact,
                             const uint8_t* removed, int32_t* out_ids, float* out_scores, int32_t* out_iters,
                             int64_t* out_scored, double* out_margin) {
  return ann_search_core(emb, emb_dtype, n, emb_dim, graph, deg, query, k, beam, parents, n_entry, max_iters, exact, removed,
                         out_ids, out_scores, out_iters, out_scored, out_margin);
}

/* ---------------------------------------------------------------- RoPE */

/*
 * Frequency of pair i: theta^(-2i/R) for a rotary dimension R (the whole head unless the model rotates only the
 * first R coordinates), evaluated in double and rounded ONCE to binary32 (models keep this vector in fp32).  An
 * override vector replaces it.
 */
static double pair_freq(int i, int R, double theta, const float* inv_freq_override) {
  if (inv_freq_override) return (double)inv_freq_override[i];
  return (double)(float)pow(theta, -(double)(2 * i) / (double)R);
}

void oracle_inv_freq(int D, double theta, float* out) {
  for (int i = 0; i < D / 2; ++i) out[i] = (float)pair_freq(i, D, theta, NULL);
}

/*
 * The rescaled frequency table of the Llama-3.1 family ("the model's own rotary tables", Sec. 3.3; the primary
 * model of the evaluation, Sec. 6.1): a pair whose wavelength 2*pi/f exceeds original_max / low_freq_factor is
 * slowed down by `factor`, one whose wavelength is below original_max / high_freq_factor is kept, and in between
 * the two are blended linearly in  s = (original_max / wavelength - low_freq_factor) / (high - low).
 * Computed in double from the unrounded theta^(-2i/R) and rounded once to binary32.
 */
int oracle_inv_freq_llama3(int R, double theta, double factor, double low_freq_factor, double high_freq_factor,
                           double original_max, float* out) {
  const double two_pi = 6.283185307179586476925286766559;
  if (R <= 0 || (R & 1) || !out || !(factor > 0) || !(high_freq_factor > low_freq_factor) || !(original_max > 0))
    return ORACLE_ERR_ARG;
  for (int i = 0; i < R / 2; ++i) {
    double f = pow(theta, -(double)(2 * i) / (double)R);
    double wavelen = two_pi / f;
    double g;
    if (wavelen > original_max / low_freq_factor) {
      g = f / factor;
    } else if (wavelen < original_max / high_freq_factor) {
      g = f;
    } else {
      double sm = (original_max / wavelen - low_freq_factor) / (high_freq_factor - low_freq_factor);
      g = (1.0 - sm) * f / factor + sm * f;
    }
    out[i] = (float)g;
  }
  return ORACLE_OK;
}

/*
 * Rotate one head vector x[0..D) at position pos into y.  Only the first R coordinates rotate (R = D for the
 * models of the paper; R < D is the "partial rotary" parameterisation); the rest is copied.
 * style 0 (half-split): pair i is (x[i], x[i + R/2]);  style 1 (interleaved): (x[2i], x[2i+1]);  i < R/2.
 * (x1, x2) -> (x1 cos a - x2 sin a,  x2 cos a + x1 sin a),  a = pos * freq_i.
 */
static void rope_head(const double* x, double* y, int D, int R, int64_t pos, double theta, int style,
                      const float* inv_freq_override) {
  int half = R / 2;
  for (int i = 0; i < half; ++i) {
    int i1 = style == 0 ? i : 2 * i;
    int i2 = style == 0 ? i + half : 2 * i + 1;
    double angle = (double)pos * pair_freq(i, R, theta, inv_freq_override);
    double c = cos(angle), s = sin(angle);
    double x1 = x[i1], x2 = x[i2];
    y[i1] = x1 * c - x2 * s;
    y[i2] = x2 * c + x1 * s;
  }
  for (int d = R; d < D; ++d) y[d] = x[d];
}

/* Rotate n_rows independent head vectors (row r at position pos[r]); rotary_dim = 0 means the whole head. */
int oracle_rope_rows_partial(const double* x, int64_t n_rows, int D, int rotary_dim, const int64_t* pos, double theta,
                             int style, const float* inv_freq_override, double* y) {
  int R = rotary_dim ? rotary_dim : D;
  if (!x || !y || !pos || D <= 0 || R <= 0 || R > D || (R & 1) || (style != 0 && style != 1)) return ORACLE_ERR_ARG;
  for (int64_t r = 0; r < n_rows; ++r) rope_head(x + r * D, y + r * D, D, R, pos[r], theta, style, inv_freq_override);
  return ORACLE_OK;
}
int oracle_rope_rows(const double* x, int64_t n_rows, int D, const int64_t* pos, double theta, int style,
                     const float* inv_freq_override, double* y) {
  if (D & 1) return ORACLE_ERR_ARG;
  return oracle_rope_rows_partial(x, n_rows, D, 0, pos, theta, style, inv_freq_override, y);
}

/* ---------------------------------------------------------------- injection */

/*
 * Compose the facts `ids` (placement order; negative ids are skipped) at positions
 * start_pos, start_pos+1, ... and place every token in the paged cache.
 *
 * Store side (host arrays): fact f owns tokens [fact_offset[f], fact_offset[f] + fact_len[f])
 * of k_pre / v, both bf16 with layout [n_layers][store_tokens][H][D].
 *
 * Only layers [layer_begin, layer_end) are produced (lets a caller bound memory); nl = their count.
 * Outputs, all optional except out_m:
 *   out_slots   [m]              slot of every composed token
 *   out_k_ref   [nl][m][H][D]    rotated keys in double (before any rounding)
 *   out_k_bf16  [nl][m][H][D]    the same rounded once to bf16 (round-to-nearest-even)
 *   out_v       [nl][m][H][D]    values, bit copies
 *   k_cache / v_cache            a host image of the paged cache (bf16), written in place at
 *                                layer*layer_stride + block*block_stride + (slot % bs)*token_stride
 *                                + head*head_stride + d   (strides in elements; layer = absolute index)
 *
 * Variants of the model / cache parameterisation (defaults reproduce the plain path):
 *   rotary_dim       0 = the whole head, else only the first rotary_dim coordinates of a head rotate
 *   k_scale, v_scale quantised (e4m3) cache with per-tensor scales.  Used only for out_k_fp8 / out_v_fp8
 *                    [nl][m][H][D] bytes, both optional.  The paper has no 8-bit cache; the rule is the one of the
 *                    serving engines whose paged cache this fills: their cache-write kernel takes the bf16 key or
 *                    value that a bf16 cache would hold, divides it by the scale in binary32 (an IEEE division, not a
 *                    product with a reciprocal) and rounds the quotient once to e4m3, saturating.  So
 *                      K code = e4m3( binary32( bf16(rotated key) ) / k_scale ),   V code = e4m3( binary32(v) / v_scale ):
 *                    an injected 8-bit cache is then byte-identical to the one the engine would have written itself
 *                    from the bf16 cache contents, which is what output equivalence (Theorem 1) asks of an injection.
 * Returns ORACLE_OK or a negative error; on error the outputs are unspecified.
 */
int oracle_inject_ex(const int32_t* ids, int k, int64_t n_facts, const int64_t* fact_offset, const int32_t* fact_len,
                     const uint16_t* k_pre, const uint16_t* v, int64_t store_tokens, int n_layers, int H, int D,
                     double theta, int style, const float* inv_freq_override, int64_t start_pos,
                     const int32_t* block_table, int64_t n_table, int bs, int64_t num_blocks, int layer_begin,
                     int layer_end, int64_t* out_m, int64_t* out_slots, double* out_k_ref, uint16_t* out_k_bf16,
                     uint16_t* out_v, uint16_t* k_cache, uint16_t* v_cache, int64_t layer_stride, int64_t block_stride,
                     int64_t token_stride, int64_t head_stride, int n_threads, int rotary_dim, float k_scale,
                     float v_scale, uint8_t* out_k_fp8, uint8_t* out_v_fp8) {
  const int R = rotary_dim ? rotary_dim : D;
  if (!out_m || k < 0 || (k > 0 && !ids) || !fact_offset || !fact_len || H <= 0 || D <= 0 || (D & 1) || D > 1024 ||
      bs <= 0 || R <= 0 || R > D || (R & 1))
    return ORACLE_ERR_ARG;
  if ((out_k_fp8 && !(k_scale > 0.0f)) || (out_v_fp8 && !(v_scale > 0.0f))) return ORACLE_ERR_ARG;
  if (layer_begin < 0 || layer_end > n_layers || layer_begin > layer_end) return ORACLE_ERR_ARG;
  if (start_pos < 0) return ORACLE_ERR_ARG;

  /* Position policy: m = sum of the lengths of the facts that are placed. */
  int64_t m = 0;
  for (int i = 0; i < k; ++i) {
    if (ids[i] < 0) continue;
    if (ids[i] >= n_facts) return ORACLE_ERR_FACT_ID;
    m += fact_len[ids[i]];
  }
  *out_m = m;
  if (m == 0) return ORACLE_OK;
  if (!block_table || !k_pre || !v) return ORACLE_ERR_ARG;

  /* token t of the composed segment comes from store token src[t] */
  int64_t* src = (int64_t*)malloc(sizeof(int64_t) * (size_t)m);
  int64_t* slots = (int64_t*)malloc(sizeof(int64_t) * (size_t)m);
  if (!src || !slots) {
    free(src);
    free(slots);
    return ORACLE_ERR_NOMEM;
  }
  int64_t t = 0;
  for (int i = 0; i < k; ++i) {
    if (ids[i] < 0) continue;
    int32_t f = ids[i];
    for (int32_t j = 0; j < fact_len[f]; ++j, ++t) {
      int64_t pos = start_pos + t; /* = start_pos + b_i + j */
      int64_t bi = pos / bs;
      if (bi >= n_table) {
        free(src);
        free(slots);
        return ORACLE_ERR_BLOCK_TABLE;
      }
      int64_t blk = block_table[bi];
      if (blk < 0 || blk >= num_blocks) {
        free(src);
        free(slots);
        return ORACLE_ERR_BLOCK_ID;
      }
      if (fact_offset[f] + j >= store_tokens) {
        free(src);
        free(slots);
        return ORACLE_ERR_ARG;
      }
      src[t] = fact_offset[f] + j;
      slots[t] = blk * bs + pos % bs;
    }
  }
  if (out_slots) memcpy(out_slots, slots, sizeof(int64_t) * (size_t)m);

  int64_t row = (int64_t)H * D;
  set_threads(n_threads);
#pragma omp parallel for schedule(static)
  for (int64_t tt = 0; tt < m; ++tt) {
    double xin[1024], yout[1024]; /* one head */
    int64_t pos = start_pos + tt;
    for (int l = layer_begin; l < layer_end; ++l) {
      const uint16_t* ksrc = k_pre + ((int64_t)l * store_tokens + src[tt]) * row;
      const uint16_t* vsrc = v + ((int64_t)l * store_tokens + src[tt]) * row;
      int64_t o = ((int64_t)(l - layer_begin) * m + tt) * row; /* compact outputs */
      int64_t blk = slots[tt] / bs, inb = slots[tt] % bs;
      int64_t cbase = (int64_t)l * layer_stride + blk * block_stride + inb * token_stride;
      for (int h = 0; h < H; ++h) {
        for (int d = 0; d < D; ++d) xin[d] = bf16_to_double(ksrc[h * D + d]);
        rope_head(xin, yout, D, R, pos, theta, style, inv_freq_override);
        for (int d = 0; d < D; ++d) {
          uint16_t kb = double_to_bf16_rne(yout[d]);
          uint16_t vb = vsrc[h * D + d];
          if (out_k_ref) out_k_ref[o + h * D + d] = yout[d];
          if (out_k_bf16) out_k_bf16[o + h * D + d] = kb;
          if (out_v) out_v[o + h * D + d] = vb;
          if (out_k_fp8) out_k_fp8[o + h * D + d] = e4m3_of_scaled_bf16(kb, k_scale);
          if (out_v_fp8) out_v_fp8[o + h * D + d] = e4m3_of_scaled_bf16(vb, v_scale);
          if (k_cache) k_cache[cbase + h * head_stride + d] = kb;
          if (v_cache) v_cache[cbase + h * head_stride + d] = vb;
        }
      }
    }
  }
  free(src);
  free(slots);
  return ORACLE_OK;
}

/* The plain path: every coordinate rotates, bf16 cache. */
int oracle_inject(const int32_t* ids, int k, int64_t n_facts, const int64_t* fact_offset, const int32_t* fact_len,
                  const uint16_t* k_pre, const uint16_t* v, int64_t store_tokens, int n_layers, int H, int D,
                  double theta, int style, const float* inv_freq_override, int64_t start_pos,
                  const int32_t* block_table, int64_t n_table, int bs, int64_t num_blocks, int layer_begin,
                  int layer_end, int64_t* out_m, int64_t* out_slots, double* out_k_ref, uint16_t* out_k_bf16,
                  uint16_t* out_v, uint16_t* k_cache, uint16_t* v_cache, int64_t layer_stride, int64_t block_stride,
                  int64_t token_stride, int64_t head_stride, int n_threads) {
  return oracle_inject_ex(ids, k, n_facts, fact_offset, fact_len, k_pre, v, store_tokens, n_layers, H, D, theta, style,
                          inv_freq_override, start_pos, block_table, n_table, bs, num_blocks, layer_begin, layer_end, out_m,
                          out_slots, out_k_ref, out_k_bf16, out_v, k_cache, v_cache, layer_stride, block_stride,
                          token_stride, head_stride, n_threads, 0, 0.0f, 0.0f, NULL, NULL);
}
