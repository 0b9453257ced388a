/*
 * memstore.h - C ABI of libmemstore.so: an HBM-resident fact store with exact top-k
 * retrieval and fused Chunked-RoPE injection into a paged KV cache (NVIDIA B200, sm_100a).
 *
 * The calls follow the paper's statement of the serving path:
 *   - a store keyed by fact id that holds, per fact, one retrieval embedding and the fact's
 *     PRE-rotation keys and raw values for every layer, with no positional metadata
 *     ("Persistent memory store and retrieval", Sec. 3.2; "Position-agnostic storage", Sec. 5.1);
 *   - a top-k search by inner product that returns fact ids (Sec. 3.2);
 *   - composition of the retrieved facts at contiguous positions with RoPE applied to the stored
 *     keys at those positions ("Chunked-RoPE composition", Sec. 3.3; Theorem 2; "Position policy",
 *     Sec. 5.2), and a scatter of K and V into the request's paged blocks through the slot mapping
 *     (Sec. 2.2; worker side of the connector, Sec. 3.4).
 *
 * Conventions
 *   - Every call returns an ms_status and never throws or aborts.  memstore_last_error() gives text.
 *   - "device" pointers are CUDA device pointers on the store's device; "host" pointers are ordinary
 *     host memory.  Nothing here takes a framework tensor.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  retrieve and
 *     inject only ENQUEUE work on it and never synchronise with the host; ids flow device to device.
 *   - Errors the host can see (bad arguments, capacity) are returned at once and enqueue nothing.
 *     Errors that depend on device data (a bad id inside a request, a block table that is too
 *     short ...) set bits in that request's status word and SKIP the offending tokens; the kernels
 *     never read or write out of bounds, never trap and contain no unbounded wait.
 *   - The store copies what add_fact(s) is given; the caller keeps ownership of its buffers.  The
 *     caller owns queries, id lists, block tables and the paged cache.
 *   - Fact ids are dense int32 numbers assigned in insertion order, global across users.  The store
 *     is append-only (the paper's store is built once and then read).
 *   - Calls on one store may be issued from several streams; the store orders them on the device
 *     (they share scratch memory).  add_fact(s) must not run concurrently with other calls from
 *     another host thread.
 *   - CUDA graphs: memstore_retrieve, memstore_inject and memstore_retrieve_inject may be recorded on a stream
 *     that is being captured, once a call of the same shape has run eagerly (scratch is sized, and grown with
 *     cudaMalloc, on first use, which a capture does not allow).  A call depends on no earlier call (its kernels
 *     leave the store's control state clean), so a graph may hold any number of calls and be replayed any number
 *     of times, also between eager calls.  The store cannot see replays: the caller orders a replay against every other use of
 *     the same store (same stream, or events), as the store does for eager calls.
 *   - There is no CPU fallback: every step runs in CUDA kernels of this library.
 */
#ifndef MEMSTORE_H
#define MEMSTORE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct memstore memstore_t;
typedef void* ms_stream; /* cudaStream_t */

typedef enum {
  MS_OK = 0,
  MS_ERR_INVALID_ARG = 1,
  MS_ERR_UNSUPPORTED = 2,
  MS_ERR_OOM = 3,      /* device or host allocation failed */
  MS_ERR_CAPACITY = 4, /* store full: facts per user or KV arena tokens */
  MS_ERR_CUDA = 5
} ms_status;

/* per-request status bits written by memstore_inject (0 = clean) */
enum {
  MS_REQ_BAD_FACT_ID = 1,       /* id >= number of facts: contributes no tokens */
  MS_REQ_NOT_RESIDENT = 2,      /* fact has no K/V in the arena: contributes no tokens */
  MS_REQ_BLOCK_TABLE_SHORT = 4, /* pos / block_size >= max_blocks: token skipped */
  MS_REQ_BAD_BLOCK_ID = 8,      /* table entry < 0 or >= num_blocks: token skipped */
  MS_REQ_POSITION_OVERFLOW = 16, /* pos >= max_position: token skipped */
  MS_REQ_KERNEL_TIMEOUT = 32,    /* a bounded wait inside the copy kernel ran out: the cache contents of this call are incomplete */
  MS_REQ_BAD_START = 64          /* start_pos < 0: no token of the request is placed */
};

enum { MS_DTYPE_F32 = 0, MS_DTYPE_F16 = 1, MS_DTYPE_BF16 = 2 };
enum { MS_ROPE_HALF_SPLIT = 0, MS_ROPE_INTERLEAVED = 1 };
enum {
  MS_INJECT_REVERSE = 1u, /* place ids[k-1] first, so that ids[0] ends next to the query */
  MS_INJECT_PREFIX = 2u,  /* place the store's instruction prefix (memstore_set_prefix) before the facts */
  MS_RETRIEVE_ANN = 4u,   /* memstore_retrieve_inject / memstore_serve_host only: retrieve through the graph index
                             (memstore_retrieve_ann with its default parameters) instead of the exact scan */
  MS_INPUTS_STABLE = 8u,  /* memstore_retrieve_inject only: the caller vouches that queries, query_users, start_pos and
                             block_tables were completely written before the work that precedes this call in the stream
                             began (a serving loop whose next query is ready before the previous injection is enqueued),
                             or that the host has seen them complete before it makes this call (a transfer on another
                             stream that the host waited for).
                             The scoring and selection of this call may then overlap the tail of the preceding kernel -
                             typically the previous request's copy kernel, whose draining SMs they use; ids, plan and
                             cache are still written strictly after it.  Without the flag - and for the first such
                             call after the store itself was changed (facts added or removed, a new prefix) - the call
                             orders itself after all preceding work, as any launch does.  Results are the same either
                             way. */
  MS_SERVE_EARLY_RETURN = 16u /* memstore_serve_host only: return as soon as the ids, the token count and the status
                             have reached the host - they are final once the request is planned - instead of waiting
                             for the stream; the copy of K and V into the cache completes in stream order, as after any
                             asynchronous call (later work on the same stream sees the injected tokens; the host
                             synchronises the stream before it reads the cache itself) */
};
/* store flag: inject through the bulk-async (TMA) staged copy kernel instead of the direct one (kept for
 * comparison; it is slower on B200 and serves rows of at most 16 KiB, larger rows fall back to the direct kernel) */
enum { MS_STORE_TMA_COPY_PATH = 1u };

typedef struct {
  int32_t device;         /* CUDA device ordinal */
  int32_t n_layers;       /* L */
  int32_t n_kv_heads;     /* h */
  int32_t head_dim;       /* d: 16, 32, 64, 128 or 256 */
  int32_t kv_dtype;       /* dtype of the STORED K/V: MS_DTYPE_BF16 only (Sec. 3.5 counts bfloat16 bytes) */
  int32_t emb_dim;        /* a multiple of 8 */
  int32_t emb_dtype;      /* MS_DTYPE_F32 or MS_DTYPE_F16 */
  int32_t rope_style;     /* MS_ROPE_HALF_SPLIT pairs (i, i+d/2); MS_ROPE_INTERLEAVED pairs (2i, 2i+1) */
  double rope_theta;      /* frequency of pair i is theta^(-2i/R), R = rotary_dim (d by default), rounded once to fp32 */
  const float* inv_freq_override; /* host, R/2 floats, or NULL; replaces the formula above (copied) */
  int64_t max_position;   /* tokens at pos >= max_position are refused; 0 < max_position <= 2^24 */
  int32_t n_users;        /* number of private embedding segments (>= 1) */
  uint32_t flags;         /* MS_STORE_* bits, normally 0 */
  int64_t max_facts_per_user; /* capacity of each user's embedding segment */
  int64_t max_kv_tokens;  /* capacity of the K/V arena in tokens (0: embedding-only store) */
  void* kv_arena;         /* optional caller-provided DEVICE buffer for the arena, else NULL */
  size_t kv_arena_bytes;  /* its size; must be >= memstore_arena_bytes(config) */
  int64_t max_host_kv_tokens; /* capacity in tokens of the second K/V arena in pinned HOST memory (0: none), < 2^30 */
  int32_t rotary_dim;     /* R: only the first R coordinates of a head rotate (pairs (i, i+R/2) or (2i, 2i+1), i < R/2,
                             frequencies theta^(-2i/R); the rest is copied).  0 = head_dim, the paper's models; else a
                             multiple of 16, <= head_dim.  inv_freq_override then holds R/2 floats. */
  int32_t reserved1;      /* 0 */
} memstore_config;

/*
 * The rescaled frequency table of the Llama-3.1 family, the paper's primary model ("the model's own rotary
 * tables", Sec. 3.3; Sec. 6.1): pair i of an R-dimensional rotation starts from f = theta^(-2i/R); a wavelength
 * 2*pi/f above original_max_position / low_freq_factor is slowed down by `factor`, one below
 * original_max_position / high_freq_factor is kept, and in between the two are blended linearly in
 * (original_max_position / wavelength - low_freq_factor) / (high_freq_factor - low_freq_factor).  Evaluated in
 * double, rounded once to fp32.  Pure host arithmetic: out (host, R/2 floats) is meant for inv_freq_override.
 * Llama-3.1: factor 8, low 1, high 4, original_max_position 8192.
 */
ms_status memstore_rope_table_llama3(int32_t rotary_dim, double rope_theta, double factor, double low_freq_factor,
                                     double high_freq_factor, double original_max_position, float* out);

/* Bytes of the K/V arena for this configuration: 2 * L * max_kv_tokens * h * d * 2
 * (the paper's storage formula, Sec. 3.5, with c = max_kv_tokens and bf16). */
size_t memstore_arena_bytes(const memstore_config* config);

/* Create a store on config->device.  Allocates the arena (unless given), the embedding segments
 * and the fact table with cudaMalloc.  *out is NULL on failure. */
ms_status memstore_create(const memstore_config* config, memstore_t** out);
ms_status memstore_destroy(memstore_t* store);

/*
 * Append one fact to `user`'s segment (Sec. 3.1/3.2: a fact is an embedding plus the fact's slice of
 * pre-RoPE K and raw V).
 *   emb    device, [emb_dim] in emb_dtype
 *   k_pre  device, bf16, [n_layers][n_tokens][n_kv_heads][head_dim], keys BEFORE any rotation
 *   v      device, bf16, same layout
 * k_pre == v == NULL with n_tokens == 0 adds an embedding-only fact (not resident: it can be
 * retrieved but not injected).  *out_fact_id (host, optional) receives the new id.
 * Copies are enqueued on `stream`; the source buffers may be reused once the stream has passed them.
 */
ms_status memstore_add_fact(memstore_t* store, int32_t user, const void* emb, const void* k_pre, const void* v,
                            int32_t n_tokens, int32_t* out_fact_id, ms_stream stream);

/*
 * Append n facts to `user`'s segment in one call.
 *   embs      device, [n][emb_dim]
 *   n_tokens  HOST, [n]; 0 marks an embedding-only fact
 *   k_pre, v  device, bf16, [n_layers][T][n_kv_heads][head_dim] with T = sum(n_tokens): the facts' tokens
 *             one after another along the token axis (NULL allowed when T == 0)
 * *out_first_id (host, optional) receives the id of the first fact; the others follow densely.
 */
ms_status memstore_add_facts(memstore_t* store, int32_t user, int64_t n, const void* embs, const void* k_pre,
                             const void* v, const int32_t* n_tokens, int32_t* out_first_id, ms_stream stream);

/*
 * Append n facts whose K/V stay in HOST memory (the paper's CPU-offloaded store, Sec. 6.8: the KV store moves to
 * pinned host DRAM and retrieved facts are streamed over PCIe).  Same arguments as memstore_add_facts except that
 * k_pre and v are HOST pointers; embs is still a device pointer (retrieval always runs from HBM).  The rows are copied
 * into the store's pinned host arena (capacity max_host_kv_tokens) before the call returns.  memstore_inject reads the
 * rows of such facts directly over PCIe inside the same copy kernel; a request may mix facts of both tiers.
 */
ms_status memstore_add_facts_host(memstore_t* store, int32_t user, int64_t n, const void* embs, const void* k_pre_host,
                                  const void* v_host, const int32_t* n_tokens, int32_t* out_first_id, ms_stream stream);

/*
 * Score each query against every fact of its user by inner product and select the k best
 * (Sec. 3.2; exact search instead of the paper's graph index).
 *   queries      device, [nq][emb_dim] in emb_dtype
 *   query_users  device int32 [nq], or NULL (every query searches user 0)
 *   out_ids      device int32 [nq][k]: rank 0 = highest score; equal scores: lower fact id first;
 *                padded with -1 when the user has fewer than k facts
 *   out_scores   device fp32 [nq][k] or NULL (0 where the id is -1)
 * Products of the stored values are accumulated in fp32.  1 <= k <= 2048.
 * Kernel choice: segments of at most 8192 rows are scored and selected in one launch; larger segments use a
 * scoring launch and a selection launch; with 8 or more fp16 queries (emb_dim a multiple of 64, at most 1024,
 * k <= 256, no per-query users) on a large segment the scoring runs on the tensor cores (tcgen05) as a filter
 * that is followed by an exact fp32 rescoring of the surviving rows, so results do not depend on the path.
 */
ms_status memstore_retrieve(memstore_t* store, const void* queries, const int32_t* query_users, int32_t nq, int32_t k,
                            int32_t* out_ids, float* out_scores, ms_stream stream);

/*
 * memstore_retrieve without any allocation (the paper has no counterpart: this exists for callers, not for the
 * method).  Some callers cannot let a library allocate device memory while they serve requests: an inference
 * engine that has already claimed almost all of HBM for its KV cache leaves nothing for a later cudaMalloc to
 * succeed with, and a latency-critical loop cannot afford the device-wide synchronisation a cudaMalloc or
 * cudaFree may cause.  memstore_retrieve grows its score scratch with cudaMalloc the first time it sees a batch
 * size; this entry point never allocates or frees anything.  Same arguments, same results as memstore_retrieve.
 *
 * Its scratch is a fixed array inside the library: MEMSTORE_STATIC_SCRATCH_BYTES (4 MiB + 4 KiB) of device
 * memory that every GPU holds from the moment it loads the library until the process exits.  Limits, checked
 * before anything is enqueued (MS_ERR_CAPACITY with a message otherwise):
 *     nq <= MEMSTORE_STATIC_MAX_QUERIES  and  nq * max_facts_per_user <= MEMSTORE_STATIC_MAX_SCORES.
 * The first call on a device looks up the array's device address (no allocation, but a set-up step): make that
 * first call before any stream capture begins on that device.
 * The array is shared by EVERY call of this entry point on the device, whichever store or stream: two such calls
 * whose kernels could overlap on the GPU race on it, so the caller must order them (one stream, or events).  It
 * keeps the previous call's contents; the part that must start at zero is cleared on the stream by each call.
 */
#define MEMSTORE_STATIC_MAX_QUERIES 1024
#define MEMSTORE_STATIC_MAX_SCORES (1 << 20)
#define MEMSTORE_STATIC_SCRATCH_BYTES (MEMSTORE_STATIC_MAX_SCORES * 4 + MEMSTORE_STATIC_MAX_QUERIES * 4)
ms_status memstore_retrieve_static(memstore_t* store, const void* queries, const int32_t* query_users, int32_t nq,
                                   int32_t k, int32_t* out_ids, float* out_scores, ms_stream stream);

/*
 * Approximate retrieval over a proximity graph (Sec. 2.5: the paper retrieves with a GPU-resident graph index
 * searched by a beam search; Sec. 6.1: inner-product distance, 64 graph neighbours, beam width 64).  The paper
 * does not print the index's algorithm; this library's is:
 *   graph   G[n][degree], row r = the `degree` rows with the largest inner product with row r (r excluded), best
 *           first, -1 padded: an exact neighbour graph, built on the device by the exact retrieval kernels with
 *           the rows themselves as queries (n / 64 retrieval calls: an offline step, as in the paper);
 *   search  a list of at most max(beam, k) rows ordered by score (ties to the lower row) starts from the rows
 *           ((i + 1) * 2654435761) mod n, i < n_entry; each step marks the first `parents` unexpanded rows of the
 *           list expanded, scores their neighbours that were never scored before, and keeps the best; it ends
 *           when no unexpanded row is left or after max_iters steps.  Scores are the fp32 sums of
 *           memstore_retrieve, so a result differs from the exact one only in which rows were looked at.
 * Every user segment has a graph of its own (the evaluation keeps one index per conversation, Sec. 6.7): rows of a
 * user's graph are rows of that user's segment (= fact ids in a single-segment store), all graphs share one degree, and
 * a query searches the graph of its user.  A graph covers the facts present when it was built, set or last grown
 * (memstore_graph_append): facts added later are not found until then.  A removed fact (memstore_remove_fact) stays
 * in the graph: a walk goes through it like through any row and passes it over when the result is read out.
 */
typedef struct {
  int32_t beam;      /* list length (the result needs max(beam, k) <= 256); 0 = 64 */
  int32_t parents;   /* rows expanded per step, <= 32 and parents * degree <= 512; 0 = min(8, 512 / degree) */
  int32_t n_entry;   /* starting rows, <= 512; 0 = 64 */
  int32_t max_iters; /* step limit; max_iters * parents * degree + n_entry rows must fit the visited table
                        (about 39,000 rows for 1024-d embeddings); 0 = 32 */
} ms_ann_params;

/* Build the graphs of all segments from the facts present (degree <= 255); replaces earlier graphs.  Removed facts
 * are nobody's neighbours in a graph built after their removal.  Synchronises the device once (allocation), then
 * enqueues the retrieval calls on `stream`. */
ms_status memstore_build_graph(memstore_t* store, int32_t degree, ms_stream stream);
/*
 * Grow the graph for the facts added since it was built, set or last grown (the paper names online insertion as future
 * work; the rule is this library's): a new row gets its exact neighbour list over all rows; an old row is offered
 * every new row that lists it and keeps the best `degree` of its old list plus those offers, best first.  One exact
 * retrieval call and two small kernels per 64 new rows (fewer when degree > 64), instead of a rebuild.  Old rows that
 * no new row lists keep their lists, so the result can differ from a fresh build.  Synchronises the device once
 * (allocation of the larger graph).  No-op when nothing was added; MS_ERR_INVALID_ARG when there is no graph.
 */
ms_status memstore_graph_append(memstore_t* store, ms_stream stream);
/* Install a caller-made graph for user 0: device int32 [n_rows][degree], entries are rows of the segment (others are
 * ignored by the search), n_rows <= number of facts of the segment.  Copied on `stream`.  memstore_set_graph_user does
 * the same for any user; a degree other than the store's current one starts every segment's graph over. */
ms_status memstore_set_graph(memstore_t* store, const int32_t* graph, int64_t n_rows, int32_t degree, ms_stream stream);
ms_status memstore_set_graph_user(memstore_t* store, int32_t user, const int32_t* graph, int64_t n_rows, int32_t degree,
                                  ms_stream stream);
/* Copy the graph out: out = device int32 buffer of out_capacity entries or NULL; *out_rows, *out_degree (host,
 * optional) receive its shape.  MS_ERR_CAPACITY when the buffer is too small. */
ms_status memstore_get_graph(memstore_t* store, int32_t* out, int64_t out_capacity, int64_t* out_rows, int32_t* out_degree,
                             ms_stream stream);
ms_status memstore_get_graph_user(memstore_t* store, int32_t user, int32_t* out, int64_t out_capacity, int64_t* out_rows,
                                  int32_t* out_degree, ms_stream stream);
/*
 * The search.  queries: device [nq][emb_dim]; params NULL = defaults; out_ids device int32 [nq][k] (best first, -1
 * padded), out_scores device fp32 [nq][k] or NULL, out_counters device int32 [nq][2] or NULL: steps taken and rows
 * scored per query.  One thread-block cluster per query; asynchronous on `stream`.  memstore_retrieve_ann searches user
 * 0's graph for every query; memstore_retrieve_ann_users takes query_users (device int32 [nq], or NULL = user 0) and
 * returns fact ids of the query's user.
 */
ms_status memstore_retrieve_ann(memstore_t* store, const void* queries, int32_t nq, int32_t k, const ms_ann_params* params,
                                int32_t* out_ids, float* out_scores, int32_t* out_counters, ms_stream stream);
ms_status memstore_retrieve_ann_users(memstore_t* store, const void* queries, const int32_t* query_users, int32_t nq, int32_t k,
                                      const ms_ann_params* params, int32_t* out_ids, float* out_scores, int32_t* out_counters,
                                      ms_stream stream);

/*
 * Take a fact out of the store (the paper names "incrementally inserting, revising, and deleting facts, with consistent
 * updates to both the index and the pre-RoPE KV store" as future work; insertion is memstore_add_fact(s) +
 * memstore_graph_append, revision is removal + insertion, and the removal rule is this library's):
 *   - exact retrieval, on every kernel path, never returns the fact again (it scores minus infinity; a list that would
 *     reach it because fewer than k facts are left is padded with -1 instead);
 *   - the graph search still walks through its row (its edges lead on) but passes it over when the result is read out;
 *   - memstore_inject treats its id like that of a fact without K/V: MS_REQ_NOT_RESIDENT, no tokens;
 *   - composed segments in the composition cache are dropped.
 * The id is not reused and the fact's arena tokens and embedding row are not reclaimed (the store stays append-only
 * underneath).  Enqueued on `stream`, ordered after earlier calls on the store.  MS_ERR_INVALID_ARG for an unknown id
 * or one removed before.
 */
ms_status memstore_remove_fact(memstore_t* store, int32_t fact_id, ms_stream stream);

/* element type of the paged cache */
enum {
  MS_CACHE_BF16 = 0,    /* the paper's cache */
  MS_CACHE_FP8_E4M3 = 1 /* one byte per element: sign, 4 exponent bits (bias 7), 3 mantissa bits, finite maximum 448 */
};

/* A caller-owned paged KV cache, bf16 unless dtype says otherwise, described by strides in ELEMENTS:
 *   element (layer, block, token-in-block, head, d) of K is at
 *   k_base[layer*layer_stride + block*block_stride + token*token_stride + head*head_stride + d]
 * and the same for V from v_base.  All strides must be multiples of 8 and the bases 16-byte aligned.
 * An 8-bit cache takes half the write traffic; its strides are still counted in elements (= bytes).
 * This covers separate K/V planes, stacked planes, token-major and head-major blocks. */
typedef struct {
  void* k_base;
  void* v_base;
  int64_t layer_stride, block_stride, token_stride, head_stride;
  int64_t num_blocks;
  int32_t block_size;
  int32_t dtype;            /* MS_CACHE_BF16 (0) or MS_CACHE_FP8_E4M3 */
  float k_scale, v_scale;   /* MS_CACHE_FP8_E4M3 only, both > 0: the cache holds K / k_scale and V / v_scale (per-tensor
                               scales), formed as a serving engine's own cache write forms them: the bf16 key (rotated
                               and rounded as for a bf16 cache) or bf16 value is divided by the scale in fp32 (IEEE
                               division) and the quotient rounded once to e4m3, to nearest even, saturating at +-448. */
} ms_paged_cache;

/*
 * For each of nreq requests, compose its facts and write them into the paged cache
 * (Sec. 3.3, Theorem 2, Sec. 5.2, Sec. 3.4):
 *   facts are laid out contiguously in the order given, fact i starting at b_i = sum_{j<i} n_j;
 *   token j of fact i gets pos = start_pos + b_i + j and slot = block_table[pos / bs] * bs + pos % bs;
 *   K rows are rotated by RoPE at pos (fp32 arithmetic on the stored bf16 values, cos/sin evaluated
 *   on the fly, one round-to-nearest-even to bf16), V rows are copied bit for bit.
 *
 *   fact_ids      device int32 [nreq][k], placement order; entries < 0 are skipped
 *   start_pos     device int32 [nreq]; the position of the first composed token (Sec. 3.3 / 5.2: positions are
 *                 contiguous from there).  A negative value places nothing and sets MS_REQ_BAD_START; a value at or
 *                 beyond max_position places nothing and sets MS_REQ_POSITION_OVERFLOW
 *   block_tables  device int32 [nreq][max_blocks]
 *   out_n_tokens  device int32 [nreq] or NULL: m = number of tokens composed (including skipped ones)
 *   out_status    device int32 [nreq] or NULL: MS_REQ_* bits
 *   out_slot_mapping  device int64 [nreq][slot_stride] or NULL: slot of each composed token
 *                 (-1 for a skipped token; entries beyond min(m, slot_stride) are not written)
 *   flags         MS_INJECT_REVERSE: place ids in reverse order (the paper's policy for a best-first list)
 *                 MS_INJECT_PREFIX: the composed segment of every request starts with the stored instruction
 *                 prefix (positions start_pos .. start_pos + n_prefix - 1), the facts follow; m counts its tokens,
 *                 the slot mapping lists them first; k is then at most 4095 (2047 in memstore_retrieve_inject's
 *                 two-launch form).  MS_ERR_INVALID_ARG when no prefix is stored.
 * Two requests that map to the same cache slot race (last writer wins, undetected).
 */
ms_status memstore_inject(memstore_t* store, const int32_t* fact_ids, int32_t nreq, int32_t k, const int32_t* start_pos,
                          const int32_t* block_tables, int32_t max_blocks, const ms_paged_cache* cache,
                          int32_t* out_n_tokens, int32_t* out_status, int64_t* out_slot_mapping, int64_t slot_stride,
                          uint32_t flags, ms_stream stream);

/*
 * The fixed instruction prefix of the composed segment (Sec. 3.3: the retrieved facts are gathered, a fixed
 * instruction prefix is prepended, and the whole is given contiguous positions).  It is kept like a fact - keys
 * BEFORE RoPE and raw values, appended to the device K/V arena (n_tokens of max_kv_tokens) - but has no embedding
 * and no fact id, so retrieval never returns it; injections with MS_INJECT_PREFIX rotate it at its serving-time
 * positions together with the facts.
 *   k_pre, v   device bf16 [n_layers][n_tokens][n_kv_heads][head_dim], 16-byte aligned; copied on `stream`
 *   n_tokens   0 removes the prefix.  A second call replaces the prefix; the arena tokens of the old one are not
 *              reclaimed (the arena is append-only).
 * MS_ERR_CAPACITY when the arena cannot take n_tokens more.
 */
ms_status memstore_set_prefix(memstore_t* store, const void* k_pre, const void* v, int32_t n_tokens, ms_stream stream);

/*
 * memstore_retrieve immediately followed by memstore_inject of every query's id list (query q = request q), with
 * the ids handed over on the device and, for segments of at most 8192 rows, the requests planned inside the
 * retrieval kernel, so that the whole path is two launches (Sec. 3.3: search, compose and scatter per request).
 * Arguments as in the two calls; out_ids [nq][k] is both the retrieval output and the injection input.
 * With MS_RETRIEVE_ANN in flags the ids come from the graph search (the paper's own pipeline: index search, compose,
 * scatter), followed by the planning and copy kernels; k <= 256.
 */
ms_status memstore_retrieve_inject(memstore_t* store, const void* queries, const int32_t* query_users, int32_t nq, int32_t k,
                                   const int32_t* start_pos, const int32_t* block_tables, int32_t max_blocks,
                                   const ms_paged_cache* cache, int32_t* out_ids, float* out_scores, int32_t* out_n_tokens,
                                   int32_t* out_status, int64_t* out_slot_mapping, int64_t slot_stride, uint32_t flags,
                                   ms_stream stream);

/*
 * One request end to end from HOST buffers, for a caller that holds its query and block table in host memory
 * (Sec. 3.3 and 3.4 in one call: search, compose, scatter).  Copies the query, the start position and the block table
 * to the device in one transfer (through a pinned staging buffer owned by the store, allocated on first use),
 * retrieves the k best facts of `user`, injects them (flags: MS_INJECT_*), has the kernels write ids, token count and
 * status into pinned host memory and waits for the stream (with MS_SERVE_EARLY_RETURN: only for those results).
 *   query        host, [emb_dim] in emb_dtype          block_table  host int32 [max_blocks]
 *   out_ids      host int32 [k] (best first, -1 padded) out_n_tokens, out_status  host, optional
 * The paged cache itself stays on the device.  Not thread-safe against other calls on the same store.
 */
ms_status memstore_serve_host(memstore_t* store, const void* query, int32_t user, int32_t k, int32_t start_pos,
                              const int32_t* block_table, int32_t max_blocks, const ms_paged_cache* cache, uint32_t flags,
                              int32_t* out_ids, int32_t* out_n_tokens, int32_t* out_status, ms_stream stream);

/* Counters since creation (host side; bytes are the algorithmic ones, not measured traffic).  Reading
 * kernel_timeouts synchronises the device. */
typedef struct {
  int64_t n_facts, n_resident_facts, kv_tokens_used;
  int64_t retrieve_calls, inject_calls;
  int64_t kernels_launched; /* kernels of this library enqueued so far */
  int64_t arena_bytes, embedding_bytes;
  int64_t host_kv_tokens_used;
  int64_t kernel_timeouts; /* 1 if a bounded wait inside the tensor-core scoring kernel ever ran out (results of that call are invalid) */
  int64_t filter_fixups;   /* queries of the tensor-core retrieve path that were re-scanned exactly because the filter's margin
                              check failed (more groups within rounding of the k-th score than the margin keeps) */
  int64_t n_removed_facts;  /* facts taken out by memstore_remove_fact */
  int64_t compose_cache_hits, compose_cache_fills; /* requests served from / recorded into the composition cache */
  int64_t compose_cache_segments;                  /* segments the composition cache can hold (0: none) */
  int64_t filter_fixup_overflows; /* 1 if such a re-scan ever met more than 4096 rows within rounding of the k-th score: that
                                     query kept the filter's answer (ids inside the 1e-5 near-tie rule, exact ties unordered) */
  int64_t filter_list_queries;   /* queries of the tensor-core retrieve path served from the candidate rows the scoring kernel
                                    listed for them, */
  int64_t filter_list_rows;      /* the rows it listed for those queries in all (a few hundred to a thousand each), and */
  int64_t filter_list_fallbacks; /* the queries whose list was too short, too long or tied at its cut and that were served
                                    from the group maxima instead (same results, slower) */
} memstore_stats_t;
ms_status memstore_stats(memstore_t* store, memstore_stats_t* out);

/*
 * Measurement aid (no counterpart in the paper).  While both events are non-NULL, every memstore_inject
 * records `before_copy` (a cudaEvent_t) on the call's stream just before the gather/rotate/scatter kernel
 * and `after_copy` just after it, so that a benchmark can time that kernel alone with CUDA events.  The
 * record between the plan kernel and the copy kernel removes their launch overlap, so leave this off
 * (NULL, NULL) when timing whole calls.  The caller owns the events.
 */
ms_status memstore_set_profile_events(memstore_t* store, void* before_copy, void* after_copy);
/*
 * Measurement aid, with the events above: while they are set, every memstore_inject launches its direct
 * gather/rotate/scatter kernel n times in a row on the same plan (the writes are the same every time), as ordinary
 * launches - each starts when the one before it has ended - between the two event records.  (after - before) / n is then
 * the duration of one launch with the cost of the event records (a few microseconds: nothing of a kernel launch overlaps
 * an event record) spread over n launches.  n = 1 restores one launch per call.  1 <= n <= 1024.
 */
ms_status memstore_set_profile_repeats(memstore_t* store, int32_t n);

/*
 * The composition cache (appendix "Position independence and rotation fidelity", closing remark: the one-time
 * composition is cached across queries that reuse the same memory).  In this library composing IS the scatter, so for
 * facts in HBM a cached segment saves nothing; it pays for facts of the host tier (Sec. 6.8), whose rows cross PCIe
 * every time they are composed: a request that repeats an earlier one is served by an HBM-rate copy instead.
 *   budget_bytes            device memory for cached segments (0: switch the cache off and free it)
 *   max_tokens_per_segment  longest composed segment that is kept; the cache holds budget / (that many tokens' K and V
 *                           over all layers) segments, at most 64
 *   flags                   0: only requests that name at least one host-tier fact are recorded;
 *                           MS_COMPOSE_CACHE_ALL: every eligible request
 * A segment is the composed K (rotated, rounded to bf16) and V of one request.  Its key is the request's id list as
 * given (at most 256 ids), its start position, MS_INJECT_REVERSE / MS_INJECT_PREFIX and the stored prefix: a request
 * with the same key is a hit and is served by copying the segment through its own block table - byte for byte what
 * composing again would write, into a bf16 or an 8-bit cache alike; anything else (another start position, another
 * order) is a miss.  Requests are looked up by memstore_inject, memstore_retrieve_inject and memstore_serve_host on
 * the device (the ids never reach the host); a miss is recorded, the least recently used segment making room, when the
 * call holds ONE request whose status word is clean (multi-request calls only look up).  Synchronises the device.
 */
enum { MS_COMPOSE_CACHE_ALL = 1u };
ms_status memstore_compose_cache(memstore_t* store, size_t budget_bytes, int32_t max_tokens_per_segment, uint32_t flags);

/*
 * Size every scratch buffer ahead of serving (no counterpart in the paper; Sec. 3.3 / 3.4 only ask that the serving
 * path be search, compose, scatter).  memstore_retrieve, memstore_inject, memstore_retrieve_inject and
 * memstore_serve_host allocate their scratch (scores, tickets, tile descriptors, staging buffers, the tensor-core
 * path's buffers) the first time a call needs more than there is, which synchronises the device once; after this
 * call, calls within the stated sizes allocate nothing and never synchronise with the host (memstore_serve_host still
 * waits for its own stream at its end):
 *   nq                      queries per retrieve / retrieve_inject call (0: leave the retrieval scratch alone)
 *   k                       ids per query or request (sizes memstore_serve_host's buffers together with max_blocks)
 *   nreq                    requests per inject call (0: leave the injection scratch alone)
 *   max_tokens_per_request  most tokens one request composes (k x longest fact + prefix)
 *   max_blocks              block-table length given to memstore_serve_host (0: leave its staging buffers alone)
 * Larger calls later still work: they grow the scratch as before.  Call it with no work of this store in flight.
 */
ms_status memstore_reserve(memstore_t* store, int32_t nq, int32_t k, int32_t nreq, int64_t max_tokens_per_request, int32_t max_blocks);

/*
 * Test aid (no counterpart in the paper).  The kernels of this library that wait on a barrier (the bulk-async staged
 * copy kernel, the tensor-core scoring kernel) bound every wait and report a time-out - MS_REQ_KERNEL_TIMEOUT in the
 * requests' status words, kernel_timeouts in the statistics - instead of hanging.  That path cannot be reached by
 * valid inputs, so this call lets a test reach it without any fault: with mute_producers != 0 the producer role of
 * those kernels issues nothing at all (no copy is ever in flight), and with wait_poll_limit != 0 every wait gives up
 * after that many polls (a few thousand polls are a fraction of a millisecond).  The kernels then return normally
 * with the time-out reported; the call's outputs are unspecified but stay inside the caller's buffers.  (0, 0)
 * restores normal behaviour and clears the recorded kernel_timeouts.
 */
ms_status memstore_test_hooks(memstore_t* store, uint32_t wait_poll_limit, int32_t mute_producers);

/* Text of the last error on this store (never NULL; valid until the next call on the store). */
const char* memstore_last_error(memstore_t* store);

/* Library version string, e.g. "memstore 0.1 sm_100a". */
const char* memstore_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MEMSTORE_H */
