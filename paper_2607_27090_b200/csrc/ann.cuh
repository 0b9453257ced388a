// Approximate retrieval: beam search over a fixed-degree proximity graph held in HBM next to the embeddings
// (Sec. 2.5 of the paper: a GPU-resident graph index searched by a beam search on the device; Sec. 6.1:
// inner-product distance, 64 graph neighbours, beam width 64).  The paper does not print the index's algorithm;
// the one implemented here, step by step:
//
//   graph    G[n][deg]: row r lists the deg rows with the largest inner product with row r (r excluded), best
//            first; -1 pads.  Built by the exact retrieval kernels with the rows themselves as queries.
//   list     at most L = max(beam, k) entries (score, row, expanded?), ordered by score descending, ties to the
//            lower row; V = the set of rows ever scored (exact: an open-addressing table in shared memory).
//   start    rows e_i = ((i + 1) * 2654435761) mod n, i < n_entry (duplicates dropped), scored and listed.
//   step     the first `parents` unexpanded entries of the list are marked expanded (none left, or max_iters
//            steps done: stop); their neighbours that are valid rows and not in V join V and are scored;
//            the best L of list + new form the next list.
//   result   the first k entries of the list; -1 / 0 pads.
//
// Scores are the fp32 sums of the exact retrieval kernels (same lane layout and summation order), so an approximate
// result differs from the exact one only in WHICH rows were looked at.  Every decision (membership in V, the order
// of the list) is independent of the order in which threads work, so the result is deterministic.
#pragma once
#include <cooperative_groups.h>

#include "retrieve.cuh"

namespace ms {

constexpr int kAnnThreads = 1024;
constexpr int kAnnMaxList = 256;   // L = max(beam, k)
constexpr int kAnnMaxCand = 512;   // rows scored in one step: parents * degree, and n_entry
constexpr uint32_t kAnnEmpty = 0xffffffffu;

struct AnnParams {
  const void* emb;      // [n_users][seg_capacity][E]
  const int32_t* graph; // [n_users][graph_cap_rows][deg]: rows of a user's graph are rows of that user's segment
  const void* queries;  // [nq][E]
  const int32_t* query_users;  // [nq] or nullptr (user 0)
  const int32_t* graph_rows;   // [n_users]: rows each user's graph covers
  const int32_t* emb_fact_id;  // [n_users][seg_capacity] row -> fact id, or nullptr when the row is the id
  int64_t seg_capacity, graph_cap_rows;
  int32_t n_users, emb_dim, deg;
  int32_t k, list_len, parents, n_entry, max_iters;
  uint32_t table_mask;  // visited table: table_mask + 1 slots (a power of two, at least twice the rows ever scored)
  int32_t* out_ids;     // [nq][k]
  float* out_scores;    // [nq][k] or nullptr
  int32_t* out_counters;  // [nq][2] or nullptr: steps taken, rows scored
  const uint32_t* removed_bits;  // one bit per row, or nullptr: removed rows walk along but are passed over in the result
};

// key of a list entry: order key of the score, then lower row first, lowest bit = not yet expanded
__device__ __forceinline__ unsigned long long ann_key(float score, int32_t row, bool unexpanded) {
  return ((unsigned long long)order_key(score) << 32) | ((unsigned long long)(0x7fffffffu - (uint32_t)row) << 1) |
         (unexpanded ? 1ull : 0ull);
}
__device__ __forceinline__ int32_t ann_key_row(unsigned long long key) {
  return (int32_t)(0x7fffffffu - (uint32_t)((key & 0xffffffffull) >> 1));
}

// Scores of two rows at once (two rows' loads in flight per warp) against the query held in shared memory as
// fp32; lane layout and summation order of score_rows.  All lanes return both sums.
template <typename T>
__device__ __forceinline__ void ann_score_pair(const T* seg, int E, const float* s_q, int64_t r0, int64_t r1, bool has1, float& s0,
                                               float& s1) {
  constexpr int VEC = 16 / sizeof(T);
  const int lane = threadIdx.x & 31;
  const int nvec = E / VEC;
  const uint4* p0 = reinterpret_cast<const uint4*>(seg + r0 * E);
  const uint4* p1 = reinterpret_cast<const uint4*>(seg + (has1 ? r1 : r0) * E);
  float a0 = 0.f, a1 = 0.f;
  for (int v0 = 0; v0 < nvec; v0 += 128) {
    uint4 x[4], y[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int v = v0 + u * 32 + lane;
      if (v < nvec) {
        x[u] = __ldg(p0 + v);
        y[u] = __ldg(p1 + v);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int v = v0 + u * 32 + lane;
      if (v < nvec) {
        const float* qs = s_q + v * VEC;
        if (sizeof(T) == 2) {
          float f[8], g[8];
          unpack8(x[u], f);
          unpack8(y[u], g);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            a0 = fmaf(f[i], qs[i], a0);
            a1 = fmaf(g[i], qs[i], a1);
          }
        } else {
          const float* f = reinterpret_cast<const float*>(&x[u]);
          const float* g = reinterpret_cast<const float*>(&y[u]);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            a0 = fmaf(f[i], qs[i], a0);
            a1 = fmaf(g[i], qs[i], a1);
          }
        }
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    a0 += __shfl_xor_sync(0xffffffffu, a0, o);
    a1 += __shfl_xor_sync(0xffffffffu, a1, o);
  }
  s0 = a0 + 0.0f;  // -0 -> +0
  s1 = a1 + 0.0f;
}

struct AnnShared {
  unsigned long long list[kAnnMaxList];
  unsigned long long merged[kAnnMaxList + kAnnMaxCand];
  unsigned long long surv[kAnnMaxCand];  // candidates that can enter the list
  int32_t cand[kAnnMaxCand];
  int32_t parent[32];
  uint32_t warp_cnt[32];
  uint32_t n_cand, n_parent, n_surv, len, n_scored, done, steps;
};

// One thread-block CLUSTER per query (1, 2, 4 or 8 CTAs of 1024 threads; the host picks the size so that a small
// batch still spreads over the GPU).  The CTA of rank 0 owns the search state (list, visited table, candidates) and
// takes every decision; all CTAs of the cluster score the step's candidates, reading the candidate rows from and
// writing the keys into rank 0's shared memory through the cluster's distributed shared memory.  What this buys: a
// step scores up to 512 rows of 2 KiB, and one SM alone pulls only about 43 GB/s from memory, which made a
// single-CTA step 12-14 us; eight SMs bring the same rows in about 1.5 us.
// Dynamic shared memory: the query as fp32 (emb_dim floats), then the visited table (used in rank 0 only).
template <typename T>
__global__ void __launch_bounds__(kAnnThreads, 1) ann_search_kernel(const AnnParams p) {
  namespace cg = cooperative_groups;
  extern __shared__ __align__(16) unsigned char dyn[];
  __shared__ AnnShared sm;
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned crank = cluster.block_rank(), csize = cluster.num_blocks();
  const bool master = crank == 0;
  AnnShared* const m = cluster.map_shared_rank(&sm, 0);  // the state lives in rank 0
  float* s_q = reinterpret_cast<float*>(dyn);
  uint32_t* table = reinterpret_cast<uint32_t*>(dyn + (size_t)p.emb_dim * sizeof(float));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int q = blockIdx.x / csize;
  const int user_in = p.query_users ? p.query_users[q] : 0;
  const bool user_ok = user_in >= 0 && user_in < p.n_users;
  const int user = user_ok ? user_in : 0;
  const int E = p.emb_dim, n = user_ok ? p.graph_rows[user] : 0, L = p.list_len;
  const T* seg = reinterpret_cast<const T*>(p.emb) + (int64_t)user * p.seg_capacity * E;
  const int32_t* graph = p.graph + (int64_t)user * p.graph_cap_rows * p.deg;
  const int64_t row_base = (int64_t)user * p.seg_capacity;  // of this user's rows in the per-row tables
  const T* qv = reinterpret_cast<const T*>(p.queries) + (int64_t)q * E;

  for (int i = tid; i < E; i += kAnnThreads) s_q[i] = (float)qv[i];
  if (master) {
    for (uint32_t i = tid; i <= p.table_mask; i += kAnnThreads) table[i] = kAnnEmpty;
    if (tid == 0) {
      sm.n_cand = 0;
      sm.len = 0;
      sm.n_scored = 0;
      sm.done = n > 0 ? 0u : 1u;
      sm.steps = 0;
    }
  }
  __syncthreads();

  // (rank 0) a row joins V at most once: the thread that claims its slot lists it as a candidate
  auto visit = [&](int32_t row) {
    uint32_t slot = ((uint32_t)row * 2654435761u) & p.table_mask;
    for (uint32_t probe = 0; probe <= p.table_mask; ++probe) {
      const uint32_t old = atomicCAS(&table[slot], kAnnEmpty, (uint32_t)row);
      if (old == kAnnEmpty) {
        const uint32_t c = atomicAdd(&sm.n_cand, 1u);
        if (c < (uint32_t)kAnnMaxCand) sm.cand[c] = row;
        return;
      }
      if (old == (uint32_t)row) return;
      slot = (slot + 1) & p.table_mask;
    }
  };

  if (master && n > 0) {
    if (tid < p.n_entry) visit((int32_t)(((unsigned long long)(tid + 1) * 2654435761ull) % (unsigned long long)n));
  }
  for (;;) {
    cluster.sync();  // rank 0's candidate list (or its decision that the search is over) is complete
    if (m->done) break;
    // ---- every CTA: score its share of the candidates into rank 0's merge array ----
    {
      const int n_cand = min((int)m->n_cand, kAnnMaxCand);
      const int len = (int)m->len;
      const int gw = (int)crank * (kAnnThreads / 32) + warp, n_warps = (int)csize * (kAnnThreads / 32);
      // one row per warp while the warps of the cluster suffice, else two rows in flight per warp
      const int per = n_cand <= n_warps ? 1 : 2;
      for (int c = per * gw; c < n_cand; c += per * n_warps) {
        const bool has1 = per == 2 && c + 1 < n_cand;
        const int32_t r0 = m->cand[c], r1 = has1 ? m->cand[c + 1] : r0;
        float s0, s1;
        ann_score_pair<T>(seg, E, s_q, r0, r1, has1, s0, s1);
        if (lane == 0) {
          m->merged[len + c] = ann_key(s0, r0, true);
          if (has1) m->merged[len + c + 1] = ann_key(s1, r1, true);
        }
      }
    }
    cluster.sync();  // all keys have arrived in rank 0
    if (!master) continue;
    // ---- rank 0: merge, then choose the next parents and collect their unseen neighbours ----
    {
      const int n_cand = min((int)sm.n_cand, kAnnMaxCand);
      const int len = (int)sm.len;
      const int total = len + n_cand;
      // A full list admits only candidates above its last entry: those survivors are compacted first (their
      // order does not matter), so that the ranking below costs a few comparisons per entry once the search has
      // converged.  The list is sorted, the survivors are not: rank of a list entry = its index + the survivors
      // above it; rank of a survivor = the list entries above it (binary search) + the survivors above it.
      const unsigned long long floor_key = len == L ? sm.list[len - 1] : 0ull;
      if (tid == 0) sm.n_surv = 0;
      __syncthreads();
      if (tid >= len && tid < total) {
        const unsigned long long key = sm.merged[tid];
        if (key > floor_key) sm.surv[atomicAdd(&sm.n_surv, 1u)] = key;
      }
      __syncthreads();
      const int n_surv = (int)sm.n_surv;
      const int total_s = len + n_surv;
      unsigned long long mine = 0;
      int rank = 0;
      if (tid < len) {
        mine = sm.list[tid];
        rank = tid;
      } else if (tid < total_s) {
        mine = sm.surv[tid - len];
        int lo = 0, hi = len;  // first index whose key is below mine
        while (lo < hi) {
          const int mid = (lo + hi) >> 1;
          if (sm.list[mid] > mine) lo = mid + 1; else hi = mid;
        }
        rank = lo;
      }
      if (tid < total_s) {
        for (int j = 0; j < n_surv; ++j) rank += sm.surv[j] > mine;
      }
      __syncthreads();  // every thread has read its list entry before the list is overwritten
      if (tid < total_s && rank < L) sm.list[rank] = mine;
      __syncthreads();
      const int new_len = min(total_s, L);
      if (tid == 0) {
        sm.len = (uint32_t)new_len;
        sm.n_scored += (uint32_t)n_cand;
        sm.n_cand = 0;
      }
      // the first `parents` unexpanded entries, in list order
      const bool unexp = tid < new_len && (sm.list[tid] & 1ull);
      const uint32_t ballot = __ballot_sync(0xffffffffu, unexp);
      if (lane == 0) sm.warp_cnt[warp] = __popc(ballot);
      __syncthreads();
      uint32_t before = 0, all = 0;
      for (int w = 0; w < kAnnMaxList / 32; ++w) {
        const uint32_t c = sm.warp_cnt[w];
        before += w < warp ? c : 0u;
        all += c;
      }
      const bool stop = all == 0 || (int)sm.steps >= p.max_iters;  // the same in every thread
      if (stop) {
        if (tid == 0) sm.done = 1;
      } else {
        const uint32_t prank = before + __popc(ballot & ((1u << lane) - 1u));
        if (unexp && prank < (uint32_t)p.parents) {
          sm.parent[prank] = ann_key_row(sm.list[tid]);
          sm.list[tid] &= ~1ull;
        }
        __syncthreads();
        const int n_slots = (int)min(all, (uint32_t)p.parents) * p.deg;
        if (tid < n_slots) {
          const int32_t nb = __ldg(graph + (int64_t)sm.parent[tid / p.deg] * p.deg + tid % p.deg);
          if (nb >= 0 && nb < n) visit(nb);
        }
        if (tid == 0) sm.steps += 1;
      }
    }
  }
  cluster.sync();  // nobody leaves while another CTA may still read rank 0's shared memory
  if (!master) return;
  const int len = (int)sm.len;
  auto id_of = [&](int32_t row) { return p.emb_fact_id ? __ldg(p.emb_fact_id + row_base + row) : row; };
  if (p.removed_bits == nullptr) {
    for (int r = tid; r < p.k; r += kAnnThreads) {
      const bool ok = r < len;
      const unsigned long long key = ok ? sm.list[r] : 0ull;
      p.out_ids[(int64_t)q * p.k + r] = ok ? id_of(ann_key_row(key)) : -1;
      if (p.out_scores) p.out_scores[(int64_t)q * p.k + r] = ok ? key_score((uint32_t)(key >> 32)) : 0.f;
    }
  } else {
    // the list entries that have not been removed, in list order (the list holds at most 256 entries: 8 warps)
    const unsigned long long key = tid < len ? sm.list[tid] : 0ull;
    const int32_t row = ann_key_row(key);
    const int64_t grow = row_base + row;
    const bool keep = tid < len && !((__ldg(p.removed_bits + (grow >> 5)) >> (grow & 31)) & 1u);
    const uint32_t ballot = __ballot_sync(0xffffffffu, keep);
    if (lane == 0) sm.warp_cnt[warp] = __popc(ballot);
    __syncthreads();
    uint32_t before = 0, all = 0;
    for (int w = 0; w < kAnnMaxList / 32; ++w) {
      const uint32_t c = sm.warp_cnt[w];
      before += w < warp ? c : 0u;
      all += c;
    }
    const uint32_t pos = before + __popc(ballot & ((1u << lane) - 1u));
    if (keep && pos < (uint32_t)p.k) {
      p.out_ids[(int64_t)q * p.k + pos] = id_of(row);
      if (p.out_scores) p.out_scores[(int64_t)q * p.k + pos] = key_score((uint32_t)(key >> 32));
    }
    for (int r = (int)all + tid; r < p.k; r += kAnnThreads) {
      p.out_ids[(int64_t)q * p.k + r] = -1;
      if (p.out_scores) p.out_scores[(int64_t)q * p.k + r] = 0.f;
    }
  }
  if (p.out_counters && tid == 0) {
    p.out_counters[2 * q] = (int32_t)sm.steps;
    p.out_counters[2 * q + 1] = (int32_t)sm.n_scored;
  }
}

// Graph rows of a batch of `nb` consecutive rows starting at `row0` from their top-(deg + 1) lists (exact retrieval
// with the rows as queries): the row itself is dropped wherever it ranks (rows with duplicates need not rank first),
// the first deg others stay, -1 pads.
__global__ void graph_rows_kernel(const int32_t* topk, int k1, int32_t* graph, int deg, int64_t row0, int nb) {
  const int r = blockIdx.x * blockDim.y + threadIdx.y;  // one warp per row
  if (r >= nb) return;
  const int lane = threadIdx.x;
  const int32_t self = (int32_t)(row0 + r);
  const int32_t* src = topk + (int64_t)r * k1;
  int32_t* dst = graph + (row0 + r) * deg;
  int written = 0;
  for (int base = 0; base < k1; base += 32) {
    const int j = base + lane;
    const int32_t id = j < k1 ? src[j] : -1;
    const bool keep = id >= 0 && id != self;
    const uint32_t ballot = __ballot_sync(0xffffffffu, keep);
    const int pos = written + __popc(ballot & ((1u << lane) - 1u));
    if (keep && pos < deg) dst[pos] = id;
    written += __popc(ballot);
  }
  for (int j = min(written, deg) + lane; j < deg; j += 32) dst[j] = -1;
}

// ---- growing the graph for appended rows ------------------------------------------------------------------------
// Rule (the oracle states it the same way): a new row gets its exact list over all rows, like any row of a fresh
// graph (the build code above does that); an OLD row nb is offered every new row that lists nb among its own
// neighbours, and keeps the best `deg` of (old list + offers) by inner product with nb, best first, ties to the
// lower row.  Rows are processed in batches; after each batch two kernels apply the batch's offers.
constexpr int kAppendMaxPairs = 4096;   // (old row, new row) offers of one batch: batch rows * degree
constexpr int kAppendMaxOffers = 64;    // new rows of one batch (each offers itself to an old row at most once)
constexpr int kAppendWarps = 8;

// One CTA: the batch's offers as keys (old row << 32 | new row), sorted ascending, so that the offers to one old row
// form a run; *n_pairs = their number.  Neighbours that are new rows themselves get no offer (their lists are exact).
__global__ void __launch_bounds__(1024) append_pairs_kernel(const int32_t* graph, int deg, int64_t row0, int nb_rows, int64_t n_old,
                                                            unsigned long long* pairs, int* n_pairs) {
  __shared__ unsigned long long keys[kAppendMaxPairs];
  __shared__ int s_count;
  const int tid = threadIdx.x;
  if (tid == 0) s_count = 0;
  __syncthreads();
  const int total = nb_rows * deg;
  int mine = 0;
  for (int t = tid; t < kAppendMaxPairs; t += 1024) {
    unsigned long long key = 0ull;  // sorts last in a descending sort of inverted keys
    if (t < total) {
      const int64_t r = row0 + t / deg;
      const int32_t nbr = graph[r * deg + t % deg];
      if (nbr >= 0 && nbr < n_old) {
        key = ~(((unsigned long long)(uint32_t)nbr << 32) | (unsigned long long)(uint32_t)r);
        ++mine;
      }
    }
    keys[t] = key;
  }
  if (mine) atomicAdd(&s_count, mine);
  __syncthreads();
  bitonic_sort_desc<1024>(keys, kAppendMaxPairs);  // descending in the inverted keys = ascending in (old row, new row)
  for (int t = tid; t < kAppendMaxPairs; t += 1024) pairs[t] = ~keys[t];
  if (tid == 0) *n_pairs = s_count;
}

// One warp per run of offers to the same old row nb: scores of the old list and of the offers against row nb (the
// fp32 sums of the retrieval kernels), ranking by counting, best `deg` written back.
template <typename T>
__global__ void __launch_bounds__(kAppendWarps * 32) append_update_kernel(const RetrieveParams p, int32_t* graph, int deg, int64_t n_rows,
                                                                          const unsigned long long* pairs, const int* n_pairs) {
  __shared__ unsigned long long s_key[kAppendWarps][256 + kAppendMaxOffers];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int i = blockIdx.x * kAppendWarps + warp;
  const int n = *n_pairs;
  if (i >= n) return;
  const unsigned long long first = pairs[i];
  const int32_t nb = (int32_t)(first >> 32);
  if (i > 0 && (int32_t)(pairs[i - 1] >> 32) == nb) return;  // not the start of a run
  int run = 1;
  while (i + run < n && (int32_t)(pairs[i + run] >> 32) == nb && run < kAppendMaxOffers) ++run;
  const T* seg = reinterpret_cast<const T*>(p.emb);
  unsigned long long* key = s_key[warp];
  int32_t* list = graph + (int64_t)nb * deg;
  // candidates: the valid old entries, then the offers
  int n_cand = 0;
  for (int j = 0; j < deg + run; ++j) {
    const int32_t c = j < deg ? list[j] : (int32_t)(pairs[i + j - deg] & 0xffffffffull);
    if (j < deg && (c < 0 || c >= n_rows)) continue;  // (the list may hold new rows accepted from earlier batches)
    const float sc = score_one_row<T>(p, nb, seg, c) + 0.0f;  // "query" = row nb (p.queries is the embedding matrix)
    if (lane == 0) key[n_cand] = ((unsigned long long)order_key(sc) << 32) | (unsigned long long)(0xffffffffu - (uint32_t)c);
    ++n_cand;
  }
  __syncwarp();
  for (int c = lane; c < n_cand; c += 32) {
    const unsigned long long mine = key[c];
    int rank = 0;
    for (int j = 0; j < n_cand; ++j) rank += key[j] > mine;
    if (rank < deg) list[rank] = (int32_t)(0xffffffffu - (uint32_t)(mine & 0xffffffffull));
  }
  for (int j = n_cand + lane; j < deg; j += 32) list[j] = -1;
}

}  // namespace ms
