// Exact retrieval: inner-product scoring of query embeddings against every fact of the query's user
// (R2) and top-k selection with "higher score first, equal scores: lower fact id first" (R3).
// Paper: Sec. 3.2 (top-k search by embedding similarity returning fact ids; inner product, Sec. 6.1).
#pragma once
#include "common.cuh"
#include "inject.cuh"

namespace ms {

struct RetrieveParams {
  const void* emb;             // [n_users][seg_capacity][E]
  const int32_t* emb_fact_id;  // [n_users][seg_capacity] fact id of each row
  const int32_t* user_count;   // [n_users] rows in use
  int64_t seg_capacity;
  int32_t n_users, emb_dim;
  const void* queries;         // [nq][E]
  const int32_t* query_users;  // [nq] or NULL
  int32_t nq, k;
  float* scores;               // scratch [nq][score_stride]
  int64_t score_stride;
  int32_t* out_ids;
  float* out_scores;
  const uint32_t* removed_bits;  // one bit per row (row index user * seg_capacity + slot), or nullptr: nothing was ever removed
  int32_t return_rows;           // 1: results are rows of the segment instead of fact ids (graph building)
};

// A removed row scores minus infinity, so it sorts behind every row that is left; results that would carry that
// score are written as "no fact" (id -1, score 0).
__device__ __forceinline__ bool row_removed(const RetrieveParams& p, int user, int64_t row) {
  if (p.removed_bits == nullptr) return false;
  const int64_t g = (int64_t)user * p.seg_capacity + row;
  return (__ldg(p.removed_bits + (g >> 5)) >> (g & 31)) & 1u;
}
constexpr uint32_t kRemovedKey = 0x007fffffu;  // order_key(-infinity)

constexpr int kScoreThreads = 256;
constexpr int kScoreWarps = kScoreThreads / 32;
constexpr int kTopkThreads = 1024;
constexpr int kTopkMaxK = 2048;
constexpr int kFusedMaxRows = 8192;  // largest segment whose top-k runs inside the scoring kernel
// CTA size of the one-launch scoring + top-k (+ plan) kernels.  The last CTA of a query does the selection and the
// planning alone.  Few queries: 512 threads (two CTAs per SM; they find room on an SM sooner than a CTA that needs all
// of it, and their barriers are cheaper), 1024 threads when the planning has many tokens to lay out (k above
// kFusedPlanBigK) or the segment is too long for the 512-thread selection.  Many queries: 256 threads fill the GPU better.
constexpr int kFusedThreadsFew = 512, kFusedThreadsBig = 1024, kFusedThreadsMany = 256, kFusedFewQueries = 8, kFusedPlanBigK = 32;
static_assert(2 * kTopkMaxK * sizeof(int32_t) <= kTopkMaxK * sizeof(unsigned long long), "plan arrays reuse the candidate buffer");

__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
  const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 t = __half22float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

// acc + x[0] y[0] + ... + x[7] y[7] for the 8 fp16 values of two 16-byte vectors, added in index order with the
// mixed-precision FMA of this architecture (fma.rn.f32.f16: fp16 factors, fp32 addend and result, the exact product
// rounded once with the sum) - bit for bit what fmaf gives on the converted values, without the sixteen conversions.
__device__ __forceinline__ float dot8_f16(const uint4& x, const uint4& y, float acc) {
  const uint32_t* xw = reinterpret_cast<const uint32_t*>(&x);
  const uint32_t* yw = reinterpret_cast<const uint32_t*>(&y);
#pragma unroll
  for (int w = 0; w < 4; ++w)
    asm("{\n\t"
        ".reg .b16 xl, xh, yl, yh;\n\t"
        "mov.b32 {xl, xh}, %1;\n\t"
        "mov.b32 {yl, yh}, %2;\n\t"
        "fma.rn.f32.f16 %0, xl, yl, %0;\n\t"
        "fma.rn.f32.f16 %0, xh, yh, %0;\n\t"
        "}"
        : "+f"(acc)
        : "r"(xw[w]), "r"(yw[w]));
  return acc;
}

// fp32 score -> unsigned key that orders like the float
__device__ __forceinline__ uint32_t order_key(float s) {
  uint32_t u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_score(uint32_t kx) {
  uint32_t u = (kx & 0x80000000u) ? (kx & 0x7fffffffu) : ~kx;
  return __uint_as_float(u);
}

// ------------------------------------------------------------------------------------------------
// Scoring on CUDA cores: one warp per embedding row, 16-byte loads, fp32 accumulation.
// The summation order of a row depends only on the lane layout, never on which warp or CTA handles
// it, so identical rows get bit-identical scores (needed for the id tie rule).
// ------------------------------------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ void score_rows(const RetrieveParams& p, const float* s_q, int q, int user, int n, int64_t row0,
                                           int rows_per_cta) {
  constexpr int VEC = 16 / sizeof(T);  // elements per 16-byte vector
  const int E = p.emb_dim;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const T* seg = reinterpret_cast<const T*>(p.emb) + (int64_t)user * p.seg_capacity * E;
  const int64_t row_end = min(row0 + rows_per_cta, (int64_t)n);
  const int nvec = E / VEC;
  for (int64_t row = row0 + warp; row < row_end; row += kScoreWarps) {
    const uint4* rp = reinterpret_cast<const uint4*>(seg + row * E);
    float acc = 0.f;
    for (int v0 = 0; v0 < nvec; v0 += 128) {  // up to four vectors in flight per lane
      uint4 x[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + u * 32 + lane;
        if (v < nvec) x[u] = __ldg(rp + v);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + u * 32 + lane;
        if (v < nvec) {
          const float* qs = s_q + v * VEC;
          if (sizeof(T) == 2) {
            float f[8];
            unpack8(x[u], f);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc = fmaf(f[i], qs[i], acc);
          } else {
            const float* f = reinterpret_cast<const float*>(&x[u]);
#pragma unroll
            for (int i = 0; i < 4; ++i) acc = fmaf(f[i], qs[i], acc);
          }
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) p.scores[(int64_t)q * p.score_stride + row] = row_removed(p, user, row) ? -INFINITY : acc + 0.0f;  // -0 -> +0
  }
}

// Two rows at once (both rows' loads in flight together), each with the lane layout and summation order of
// score_rows; all lanes return both sums.
template <typename T>
__device__ __forceinline__ void score_two_rows(const RetrieveParams& p, int q, const T* seg, int64_t row0, int64_t row1, float& s0,
                                               float& s1) {
  constexpr int VEC = 16 / sizeof(T);
  const int E = p.emb_dim;
  const int lane = threadIdx.x & 31;
  const uint4* qp = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(p.queries) + (int64_t)q * E);
  const uint4* r0 = reinterpret_cast<const uint4*>(seg + row0 * E);
  const uint4* r1 = reinterpret_cast<const uint4*>(seg + row1 * E);
  const int nvec = E / VEC;
  float a0 = 0.f, a1 = 0.f;
  for (int v0 = 0; v0 < nvec; v0 += 128) {
    uint4 x[4], z[4], y[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int v = v0 + u * 32 + lane;
      if (v < nvec) {
        x[u] = __ldg(r0 + v);
        z[u] = __ldg(r1 + v);
        y[u] = __ldg(qp + v);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int v = v0 + u * 32 + lane;
      if (v < nvec) {
        if (sizeof(T) == 2) {
          a0 = dot8_f16(x[u], y[u], a0);
          a1 = dot8_f16(z[u], y[u], a1);
        } else {
          const float* f = reinterpret_cast<const float*>(&x[u]);
          const float* h = reinterpret_cast<const float*>(&z[u]);
          const float* g = reinterpret_cast<const float*>(&y[u]);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            a0 = fmaf(f[i], g[i], a0);
            a1 = fmaf(h[i], g[i], a1);
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
  s0 = a0;
  s1 = a1;
}

// The same scoring with the query read straight from global memory (through L1) next to the row, so that one
// memory round trip serves both and no shared-memory staging or barrier is needed.  Same lane layout and
// summation order as score_rows.
template <typename T, int WARPS>
__device__ __forceinline__ void score_rows_direct(const RetrieveParams& p, int q, int user, int n, int64_t row0, int rows_per_cta) {
  constexpr int VEC = 16 / sizeof(T);
  const int E = p.emb_dim;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const T* seg = reinterpret_cast<const T*>(p.emb) + (int64_t)user * p.seg_capacity * E;
  const uint4* qp = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(p.queries) + (int64_t)q * E);
  const int64_t row_end = min(row0 + rows_per_cta, (int64_t)n);
  const int nvec = E / VEC;
  int64_t row = row0 + warp;
  if constexpr (WARPS <= 8) {
    // small CTAs (many queries in flight): two rows per warp at a time, which keeps about 128 KB of loads in flight
    // per SM; the 1024-thread CTAs of the few-query case have no registers for that
    for (; row + WARPS < row_end; row += 2 * WARPS) {
      float s0, s1;
      score_two_rows<T>(p, q, seg, row, row + WARPS, s0, s1);
      if (lane == 0) {
        p.scores[(int64_t)q * p.score_stride + row] = row_removed(p, user, row) ? -INFINITY : s0 + 0.0f;
        p.scores[(int64_t)q * p.score_stride + row + WARPS] = row_removed(p, user, row + WARPS) ? -INFINITY : s1 + 0.0f;
      }
    }
  }
  for (; row < row_end; row += WARPS) {
    const uint4* rp = reinterpret_cast<const uint4*>(seg + row * E);
    float acc = 0.f;
    for (int v0 = 0; v0 < nvec; v0 += 128) {
      uint4 x[4], y[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + u * 32 + lane;
        if (v < nvec) {
          x[u] = __ldg(rp + v);
          y[u] = __ldg(qp + v);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + u * 32 + lane;
        if (v < nvec) {
          if (sizeof(T) == 2) {
            acc = dot8_f16(x[u], y[u], acc);
          } else {
            const float* f = reinterpret_cast<const float*>(&x[u]);
            const float* g = reinterpret_cast<const float*>(&y[u]);
#pragma unroll
            for (int i = 0; i < 4; ++i) acc = fmaf(f[i], g[i], acc);
          }
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) p.scores[(int64_t)q * p.score_stride + row] = row_removed(p, user, row) ? -INFINITY : acc + 0.0f;  // -0 -> +0
  }
}

// Bitonic network over P (a power of two) 64-bit keys in shared memory, largest first.
template <int THREADS>
__device__ __forceinline__ void bitonic_sort_desc(unsigned long long* cand, int P) {
  const int tid = threadIdx.x;
  for (int size = 2; size <= P; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int t = tid; t < P / 2; t += THREADS) {
        const int lo = 2 * t - (t & (stride - 1));
        const int hi = lo + stride;
        const bool desc = (lo & size) == 0;
        const unsigned long long a = cand[lo], b = cand[hi];
        if ((a < b) == desc) {
          cand[lo] = b;
          cand[hi] = a;
        }
      }
      __syncthreads();
    }
  }
}

// What a selected index stands for: the index itself, a row taken from an index->row map (candidate lists), and/or
// the fact id of that row.  Both maps are optional.
struct IdMap {
  const int32_t* idx_to_row;  // or nullptr: the index is the row
  const int32_t* row_ids;     // or nullptr: the row is the id
  int32_t* mirror = nullptr;  // optional copy of the result ids (by rank) in shared memory, for a consumer in the same CTA
  __device__ __forceinline__ int32_t operator()(uint32_t idx) const {
    int32_t row = idx_to_row ? idx_to_row[idx] : (int32_t)idx;
    return (row >= 0 && row_ids) ? row_ids[row] : row;
  }
};

// Ranks 0..k-1: fact id and fp32 score of the sorted candidates, -1 / 0 beyond `take`.
template <int THREADS>
__device__ __forceinline__ void write_topk(const unsigned long long* cand, int take, int k, const IdMap ids,
                                           int32_t* out_ids, float* out_scores) {
  for (int r = threadIdx.x; r < k; r += THREADS) {
    int32_t id = -1;
    float s = 0.f;
    if (r < take) {
      const unsigned long long c = cand[r];
      if ((uint32_t)(c >> 32) != kRemovedKey) {  // (a removed row that made the list because too few rows are left)
        id = ids(0xffffffffu - (uint32_t)(c & 0xffffffffull));
        s = key_score((uint32_t)(c >> 32));
      }
    }
    out_ids[r] = id;
    if (ids.mirror) ids.mirror[r] = id;
    if (out_scores) out_scores[r] = s;
  }
}

// Sampled bucket choice of topk_block: sample size and shape, and the shortest list it is used for.
constexpr int kSampleSize = 4096;
constexpr int kSampleChunks = 64;
constexpr int kSampleMinN = 65536;

struct TopkShared {
  uint32_t hist[256];
  unsigned long long cand[kTopkMaxK];
  uint32_t warp_cnt[32];
  uint32_t warp_min[32], warp_max[32];
  uint32_t prefix, krem, ngt, eq_base;
  uint32_t kmin, kmax, bucket, n_cand;
};

// ------------------------------------------------------------------------------------------------
// Top-k of one query by one CTA of THREADS threads.  Radix select (4 passes of 8 bits, most significant
// first) finds the k-th largest score key T; everything above T is taken, rows equal to T are taken lowest
// row first (rows of a user are in fact-id order), and the k survivors are sorted by a bitonic network on
// the 64-bit key (score key << 32) | ~row.  `keys` (shared memory, optional) holds the n order keys;
// without it they are recomputed from the scores in global memory on every pass.
// ------------------------------------------------------------------------------------------------
// Visits keys i = tid, tid + THREADS, ... < n, eight at a time: the eight loads are issued before any is used, so
// that a pass over keys in global memory is not a chain of dependent round trips.
template <int THREADS, class KeyAt, class Visit>
__device__ __forceinline__ void for_each_key(int n, KeyAt key_at, Visit visit) {
  const int tid = threadIdx.x;
  for (int base = tid; base < n; base += THREADS * 8) {
    decltype(key_at(0)) kx[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = base + u * THREADS;
      if (i < n) kx[u] = key_at(i);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = base + u * THREADS;
      if (i < n) visit(i, kx[u]);
    }
  }
}

// 256 buckets linear in the score VALUE over [s_lo, s_hi] (linear in the key would be logarithmic in the value and
// put a whole octave of top scores into one bucket); monotone in the score; scores above s_hi land in bucket 255.
struct LinearBuckets {
  float s_lo, scale;
  __device__ __forceinline__ static LinearBuckets over(float lo, float hi) { return {lo, 255.5f / fmaxf(hi - lo, 1e-30f)}; }
  __device__ __forceinline__ uint32_t of(float sv) const {  // of a score sv >= s_lo
    return min(255u, (uint32_t)((sv - s_lo) * scale));
  }
};

// Block-wide minimum and maximum of per-thread keys -> sm.kmin, sm.kmax (visible to all threads on return);
// also clears the histogram.
template <int THREADS>
__device__ __forceinline__ void block_min_max(TopkShared& sm, uint32_t lo, uint32_t hi) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, o));
  }
  if (lane == 0) {
    sm.warp_min[warp] = lo;
    sm.warp_max[warp] = hi;
  }
  for (int b = tid; b < 256; b += THREADS) sm.hist[b] = 0;
  __syncthreads();
  if (warp == 0) {
    lo = lane < THREADS / 32 ? sm.warp_min[lane] : 0xffffffffu;
    hi = lane < THREADS / 32 ? sm.warp_max[lane] : 0u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if (lane == 0) {
      sm.kmin = lo;
      sm.kmax = hi;
    }
  }
  __syncthreads();
}

// Warp 0: the highest bucket B with at least `target` histogram entries in buckets >= B -> sm.bucket, and that
// count -> sm.n_cand.  Nothing is written when the whole histogram holds fewer than `target` entries.
__device__ __forceinline__ void find_rank_bucket(TopkShared& sm, uint32_t target) {
  const int lane = threadIdx.x & 31;
  if (threadIdx.x >= 32) return;
  uint32_t c[8], sum = 0;
#pragma unroll
  for (int b = 0; b < 8; ++b) {
    c[b] = sm.hist[8 * lane + b];
    sum += c[b];
  }
  uint32_t incl = sum;  // buckets of this lane and of all higher lanes
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_down_sync(0xffffffffu, incl, o);
    if (lane + o < 32) incl += y;
  }
  uint32_t above = incl - sum;
  if (above < target && incl >= target) {
    int b = 7;
    for (; b > 0; --b) {
      if (above + c[b] >= target) break;
      above += c[b];
    }
    sm.bucket = 8 * lane + b;
    sm.n_cand = above + c[b];
  }
}

// The n_cand (>= min(n, k), <= kTopkMaxK) candidates in `cand` (shared memory), distinct 64-bit keys, are ranked and the best k
// written out.  Few candidates: the rank of a candidate is the number of larger ones, no sorting network.
template <int THREADS>
__device__ __forceinline__ void rank_candidates(unsigned long long* cand, uint32_t n_cand, int k, int take, const IdMap ids,
                                                int32_t* out_ids, float* out_scores) {
  const int tid = threadIdx.x;
  if (n_cand * 4 <= (uint32_t)THREADS) {
    // four lanes share a candidate and split the comparisons
    const uint32_t ci = (uint32_t)tid >> 2, part = (uint32_t)tid & 3u;
    const unsigned long long mine = ci < n_cand ? cand[ci] : 0ull;
    uint32_t rank = 0;
    for (uint32_t jj = part; jj < n_cand; jj += 4) rank += cand[jj] > mine;
    rank += __shfl_xor_sync(0xffffffffu, rank, 1);
    rank += __shfl_xor_sync(0xffffffffu, rank, 2);
    if (ci < n_cand && part == 0 && rank < (uint32_t)k) {
      const bool gone = (uint32_t)(mine >> 32) == kRemovedKey;
      const int32_t id = gone ? -1 : ids(0xffffffffu - (uint32_t)(mine & 0xffffffffull));
      out_ids[rank] = id;
      if (ids.mirror) ids.mirror[rank] = id;
      if (out_scores) out_scores[rank] = gone ? 0.f : key_score((uint32_t)(mine >> 32));
    }
    return;
  }
  if (n_cand <= (uint32_t)THREADS) {
    if (tid < (int)n_cand) {
      const unsigned long long mine = cand[tid];
      uint32_t rank = 0;
      for (uint32_t jj = 0; jj < n_cand; ++jj) rank += cand[jj] > mine;
      if (rank < (uint32_t)k) {
        const bool gone = (uint32_t)(mine >> 32) == kRemovedKey;
        const int32_t id = gone ? -1 : ids(0xffffffffu - (uint32_t)(mine & 0xffffffffull));
        out_ids[rank] = id;
        if (ids.mirror) ids.mirror[rank] = id;
        if (out_scores) out_scores[rank] = gone ? 0.f : key_score((uint32_t)(mine >> 32));
      }
    }
    return;
  }
  int P2 = 1;
  while (P2 < (int)n_cand) P2 <<= 1;
  for (int i = (int)n_cand + tid; i < P2; i += THREADS) cand[i] = 0ull;
  __syncthreads();
  bitonic_sort_desc<THREADS>(cand, P2);
  write_topk<THREADS>(cand, take, k, ids, out_ids, out_scores);
}

// A visit of (index, score) over fp32 scores in global memory, read as 16-byte vectors, UNROLL vectors per thread in flight: a
// long score list (a hundred thousand group maxima per query) is swept by ONE CTA, whose speed is set by the bytes
// it keeps in flight.  `sc` must be 16-byte aligned.  The visiting order differs from for_each_key; callers depend
// on the set of (index, key) pairs only.
template <int THREADS, int UNROLL, class Visit>
__device__ __forceinline__ void for_each_score_vec4(const float* sc, int n, Visit visit) {
  const int tid = threadIdx.x;
  const int n4 = n >> 2;
  const float4* v = reinterpret_cast<const float4*>(sc);
  for (int base = tid; base < n4; base += THREADS * UNROLL) {
    float4 x[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int i = base + u * THREADS;
      if (i < n4) x[u] = __ldcg(v + i);
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int i = base + u * THREADS;
      if (i < n4) {
        visit(4 * i + 0, x[u].x);
        visit(4 * i + 1, x[u].y);
        visit(4 * i + 2, x[u].z);
        visit(4 * i + 3, x[u].w);
      }
    }
  }
  const int i = 4 * n4 + tid;
  if (i < n) visit(i, __ldcg(sc + i));
}

// Second selection level for a candidate set that is several times larger than k (ranking by counting is
// quadratic): the same bucket search over the candidates' own score range keeps those in or above the bucket of
// the k-th largest.  n_cand <= kTopkMaxK / 2 candidates in sm.cand[0..n_cand); the survivors (at least k) go to
// sm.cand[kTopkMaxK / 2 ...) and their number is returned (0: the candidates' scores are all equal, nothing moved).
template <int THREADS>
__device__ __forceinline__ uint32_t refine_candidates(TopkShared& sm, uint32_t n_cand, int k) {
  const int tid = threadIdx.x;
  uint32_t lo = 0xffffffffu, hi = 0u;
  for (uint32_t j = tid; j < n_cand; j += THREADS) {
    const uint32_t kx = (uint32_t)(sm.cand[j] >> 32);
    lo = min(lo, kx);
    hi = max(hi, kx);
  }
  block_min_max<THREADS>(sm, lo, hi);
  const float smin = key_score(sm.kmin), smax = key_score(sm.kmax);
  if (!(smax > smin)) return 0u;
  LinearBuckets bk{0.f, 0.f};
  for (int attempt = 0; attempt < 2; ++attempt) {
    bk = LinearBuckets::over(attempt == 0 ? smin + 0.5f * (smax - smin) : smin, smax);
    if (attempt) {
      for (int b = tid; b < 256; b += THREADS) sm.hist[b] = 0;
    }
    if (tid == 0) sm.n_cand = 0xffffffffu;
    __syncthreads();
    for (uint32_t j = tid; j < n_cand; j += THREADS) {
      const float sv = key_score((uint32_t)(sm.cand[j] >> 32));
      if (sv >= bk.s_lo) atomicAdd(&sm.hist[bk.of(sv)], 1u);
    }
    __syncthreads();
    find_rank_bucket(sm, (uint32_t)k);
    __syncthreads();
    if (sm.n_cand != 0xffffffffu) break;
  }
  const uint32_t B = sm.bucket, n2 = sm.n_cand;
  if (tid == 0) sm.ngt = 0;
  __syncthreads();
  for (uint32_t j = tid; j < n_cand; j += THREADS) {
    const unsigned long long c = sm.cand[j];
    const float sv = key_score((uint32_t)(c >> 32));
    if (sv >= bk.s_lo && bk.of(sv) >= B) sm.cand[kTopkMaxK / 2 + atomicAdd(&sm.ngt, 1u)] = c;
  }
  __syncthreads();
  return n2;
}

// Top-k of a LONG fp32 score list in global memory (n >= kSampleMinN, 16-byte aligned) with one sweep of the list:
// the buckets and the candidate threshold come from kSampleSize scores taken in kSampleChunks evenly spaced runs,
// aiming at about 4.5 k candidates; the sweep gathers every score in or above the threshold bucket and counts
// them.  Returns true (the same value in every thread) when the gathered set held at least k and at most
// kTopkMaxK candidates and the result has been written; false when the sample was unrepresentative or unlucky (or
// the list too long for the candidate array), in which case nothing has been written and the caller runs the exact
// selection: a bad sample costs time, never correctness.
template <int THREADS>
__device__ bool topk_sampled(TopkShared& sm, const float* sc, int n, int k, const IdMap ids, int32_t* out_ids,
                             float* out_scores) {
  static_assert(kSampleSize * sizeof(float) <= sizeof(sm.cand), "the sample lives in the candidate array");
  const int tid = threadIdx.x;
  const uint32_t sample_rank = max(12u, (uint32_t)((4.5f * (float)k * (float)kSampleSize) / (float)n) + 1u);
  if ((float)sample_rank * (float)n / (float)kSampleSize > 0.5f * (float)kTopkMaxK) return false;
  float* samp = reinterpret_cast<float*>(sm.cand);
  constexpr int kRun = kSampleSize / kSampleChunks;
  const int64_t stride = n / kSampleChunks;
  float flo = INFINITY, fhi = -INFINITY;
  for (int j = tid; j < kSampleSize; j += THREADS) {
    const float sv = __ldcg(sc + (int64_t)(j / kRun) * stride + (j % kRun));
    samp[j] = sv;
    if (sv > -INFINITY) {  // removed rows score minus infinity: they take no part in the bucket layout
      flo = fminf(flo, sv);
      fhi = fmaxf(fhi, sv);
    }
  }
  block_min_max<THREADS>(sm, order_key(flo), order_key(fhi));
  const float smin = key_score(sm.kmin), smax = key_score(sm.kmax);
  if (!(smax > smin)) return false;
  LinearBuckets bk{0.f, 0.f};
  for (int attempt = 0; attempt < 2; ++attempt) {  // upper half of the sample's range first, as in topk_block
    bk = LinearBuckets::over(attempt == 0 ? smin + 0.5f * (smax - smin) : smin, smax);
    if (attempt) {
      for (int b = tid; b < 256; b += THREADS) sm.hist[b] = 0;
    }
    if (tid == 0) sm.n_cand = 0xffffffffu;
    __syncthreads();
    for (int j = tid; j < kSampleSize; j += THREADS) {
      const float sv = samp[j];
      if (sv >= bk.s_lo) atomicAdd(&sm.hist[bk.of(sv)], 1u);
    }
    __syncthreads();
    find_rank_bucket(sm, sample_rank);
    __syncthreads();
    if (sm.n_cand != 0xffffffffu) break;
  }
  if (sm.n_cand == 0xffffffffu) return false;
  const uint32_t B = sm.bucket;
  if (tid == 0) sm.ngt = 0;
  __syncthreads();  // the sample has been read by everyone: the candidates may overwrite it
  for_each_score_vec4<THREADS, 8>(sc, n, [&](int i, float sv) {
    if (sv >= bk.s_lo && bk.of(sv) >= B) {
      const uint32_t slot = atomicAdd(&sm.ngt, 1u);
      if (slot < (uint32_t)kTopkMaxK)
        sm.cand[slot] = ((unsigned long long)order_key(sv) << 32) | (uint32_t)(0xffffffffu - (uint32_t)i);
    }
  });
  __syncthreads();
  const uint32_t n_cand = sm.ngt;
  __syncthreads();  // everyone has read the count before a later selection resets it
  if (n_cand < (uint32_t)k || n_cand > (uint32_t)kTopkMaxK) return false;
  if (n_cand > 2u * (uint32_t)k && n_cand <= (uint32_t)kTopkMaxK / 2) {
    const uint32_t n2 = refine_candidates<THREADS>(sm, n_cand, k);
    if (n2) {
      rank_candidates<THREADS>(sm.cand + kTopkMaxK / 2, n2, k, k, ids, out_ids, out_scores);
      return true;
    }
  }
  rank_candidates<THREADS>(sm.cand, n_cand, k, k, ids, out_ids, out_scores);
  return true;
}

// LONG = false leaves out the code for long lists in global memory (vector sweeps, sampled bucket choice): the fused
// kernels, whose keys sit in shared memory, stay small.
template <int THREADS, bool LONG = true>
__device__ void topk_block(TopkShared& sm, const float* sc, const uint32_t* keys, int n, int k, const IdMap ids,
                           int32_t* out_ids, float* out_scores, bool have_minmax = false, uint32_t my_lo = 0xffffffffu,
                           uint32_t my_hi = 0u) {
  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const int take = min(n, k);
  auto key_at = [&](int i) -> uint32_t { return keys ? keys[i] : order_key(__ldcg(sc + i)); };
  // The fast path below works on the SCORES (a key converts back without loss): most elements then cost one
  // comparison per pass.  Long lists in global memory are swept with vector loads.
  auto score_at = [&](int i) -> float { return keys ? key_score(keys[i]) : __ldcg(sc + i); };
  const bool vec = LONG && keys == nullptr && n >= THREADS * 16 && (reinterpret_cast<uintptr_t>(sc) & 15) == 0;
  auto sweep = [&](auto visit) {
    if constexpr (LONG) {
      if (vec) {
        for_each_score_vec4<THREADS, 4>(sc, n, visit);
        return;
      }
    }
    for_each_key<THREADS>(n, score_at, visit);
  };

  // ---- sampled path: long lists in global memory, bucket choice from a sample, ONE sweep of the list ------
  if constexpr (LONG) {
    if (n > k && vec && !have_minmax && n >= kSampleMinN) {
      if (topk_sampled<THREADS>(sm, sc, n, k, ids, out_ids, out_scores)) return;
    }
  }

  // ---- fast path: one histogram over 256 LINEAR buckets of the score range -------------------------------
  // Scores of unit-norm embeddings share sign and exponent, so the leading radix digits of almost all keys
  // coincide; buckets that are linear in the score value spread them.  Every score in or above the bucket B
  // that holds the k-th largest becomes a candidate (their number is k plus part of one bucket); the 64-bit
  // keys order them exactly, ties by row.  If the candidates do not fit (massive ties) the radix path runs.
  if (n > k) {
    uint32_t lo = my_lo, hi = my_hi;
    if (!have_minmax) {
      float flo = INFINITY, fhi = -INFINITY;
      sweep([&](int, float sv) {
        if (sv > -INFINITY) {  // removed rows score minus infinity: they take no part in the bucket layout
          flo = fminf(flo, sv);
          fhi = fmaxf(fhi, sv);
        }
      });
      if (flo <= fhi) {  // this thread saw at least one score
        lo = order_key(flo);
        hi = order_key(fhi);
      }
    }
    block_min_max<THREADS>(sm, lo, hi);  // -> sm.kmin, sm.kmax; clears sm.hist
    if (sm.kmin > sm.kmax) {  // no score at all took part: every row of the segment has been removed
      for (int r = tid; r < k; r += THREADS) {
        out_ids[r] = -1;
        if (ids.mirror) ids.mirror[r] = -1;
        if (out_scores) out_scores[r] = 0.f;
      }
      return;
    }
    const uint32_t range = sm.kmax - sm.kmin;
    const float smin = key_score(sm.kmin), smax = key_score(sm.kmax);
    // With k much smaller than n only the upper part of the value range can hold the k-th largest, so the first
    // attempt histograms the upper half alone (twice the resolution and a fraction of the shared-memory atomics);
    // if fewer than k scores live there the whole range is used.
    LinearBuckets bk{0.f, 0.f};
    for (int attempt = 0; attempt < 2; ++attempt) {
      bk = LinearBuckets::over(attempt == 0 ? smin + 0.5f * (smax - smin) : smin, smax);
      if (attempt) {
        for (int b = tid; b < 256; b += THREADS) sm.hist[b] = 0;
      }
      if (tid == 0) sm.n_cand = 0xffffffffu;
      __syncthreads();
      sweep([&](int, float sv) {
        if (sv >= bk.s_lo) atomicAdd(&sm.hist[bk.of(sv)], 1u);
      });
      __syncthreads();
      find_rank_bucket(sm, (uint32_t)k);
      __syncthreads();
      if (sm.n_cand != 0xffffffffu) break;  // the k-th largest lies in the histogrammed range
    }
    if (range != 0 && sm.n_cand <= (uint32_t)kTopkMaxK) {
      const uint32_t B = sm.bucket, n_cand = sm.n_cand;
      if (tid == 0) sm.ngt = 0;
      __syncthreads();
      sweep([&](int i, float sv) {
        if (sv >= bk.s_lo && bk.of(sv) >= B) {  // a score below the histogrammed range is never a candidate
          const uint32_t slot = atomicAdd(&sm.ngt, 1u);
          if (slot < (uint32_t)kTopkMaxK)
            sm.cand[slot] = ((unsigned long long)order_key(sv) << 32) | (uint32_t)(0xffffffffu - (uint32_t)i);
        }
      });
      __syncthreads();
      rank_candidates<THREADS>(sm.cand, n_cand, k, take, ids, out_ids, out_scores);
      return;
    }
  }

  uint32_t T = 0;        // threshold key
  uint32_t need_eq = 0;  // how many rows with key == T to take
  if (n > k) {
    if (tid == 0) {
      sm.prefix = 0;
      sm.krem = (uint32_t)k;
    }
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int b = tid; b < 256; b += THREADS) sm.hist[b] = 0;
      __syncthreads();
      const uint32_t prefix = sm.prefix;
      const uint32_t himask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
      for (int i = tid; i < n; i += THREADS) {
        const uint32_t kx = key_at(i);
        if ((kx & himask) == prefix) atomicAdd(&sm.hist[(kx >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (warp == 0) {
        // lane l owns buckets 8l..8l+7; find the bucket b with count(> b) < krem <= count(>= b)
        uint32_t c[8], sum = 0;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
          c[b] = sm.hist[8 * lane + b];
          sum += c[b];
        }
        uint32_t incl = sum;  // buckets of this lane and of all higher lanes
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t y = __shfl_down_sync(0xffffffffu, incl, o);
          if (lane + o < 32) incl += y;
        }
        const uint32_t krem = sm.krem;
        uint32_t above = incl - sum;
        if (above < krem && incl >= krem) {
          int b = 7;
          for (; b > 0; --b) {
            if (above + c[b] >= krem) break;
            above += c[b];
          }
          sm.prefix = prefix | ((uint32_t)(8 * lane + b) << shift);
          sm.krem = krem - above;
        }
      }
      __syncthreads();
    }
    T = sm.prefix;
    need_eq = sm.krem;
  }
  if (tid == 0) {
    sm.ngt = 0;
    sm.eq_base = 0;
  }
  int P = 1;  // sort width: next power of two >= take
  while (P < take) P <<= 1;
  for (int i = tid; i < P; i += THREADS) sm.cand[i] = 0ull;  // padding keys are the smallest
  __syncthreads();

  if (n <= k) {
    for (int i = tid; i < n; i += THREADS)
      sm.cand[i] = ((unsigned long long)key_at(i) << 32) | (uint32_t)(0xffffffffu - (uint32_t)i);
  } else {
    const uint32_t n_gt = (uint32_t)k - need_eq;
    // rows above the threshold: order does not matter here, they are sorted afterwards;
    // rows equal to the threshold: ordered compaction, lowest rows first, the first need_eq are kept
    for (int base = 0; base < n; base += THREADS) {
      const int i = base + tid;
      uint32_t kx = 0;
      bool gt = false, eq = false;
      if (i < n) {
        kx = key_at(i);
        gt = kx > T;
        eq = kx == T;
      }
      if (gt) {
        const uint32_t slot = atomicAdd(&sm.ngt, 1u);
        if (slot < n_gt) sm.cand[slot] = ((unsigned long long)kx << 32) | (uint32_t)(0xffffffffu - (uint32_t)i);
      }
      const uint32_t bal = __ballot_sync(0xffffffffu, eq);
      if (__syncthreads_or(eq)) {
        if (lane == 0) sm.warp_cnt[warp] = __popc(bal);
        __syncthreads();
        uint32_t before = sm.eq_base;
        for (int w = 0; w < warp; ++w) before += sm.warp_cnt[w];
        if (eq) {
          const uint32_t rank = before + __popc(bal & ((1u << lane) - 1u));
          if (rank < need_eq) sm.cand[n_gt + rank] = ((unsigned long long)kx << 32) | (uint32_t)(0xffffffffu - (uint32_t)i);
        }
        __syncthreads();
        if (tid == 0) {
          uint32_t tot = 0;
          for (int w = 0; w < THREADS / 32; ++w) tot += sm.warp_cnt[w];
          sm.eq_base += tot;
        }
        __syncthreads();
      }
    }
  }
  __syncthreads();

  bitonic_sort_desc<THREADS>(sm.cand, P);
  write_topk<THREADS>(sm.cand, take, k, ids, out_ids, out_scores);
}

// ------------------------------------------------------------------------------------------------
// Selection for the fused kernels (short segments, moderate k): a threshold from the warps' own best keys instead of
// a block-wide histogram.  The n keys sit in registers, key i with thread i mod THREADS.  Every warp pulls out the
// VALUES of its t = ceil(k / warps) + 1 best keys (a warp-wide maximum per key: one redux instruction, no shared
// memory, no block barrier).  The k-th largest of those warps * t values is a lower bound of the k-th largest key
// of the whole segment (the k-th largest of a subset never exceeds the k-th largest of the set), and a tight one:
// for rows spread evenly over the warps, about 1.1 k keys reach it.  Every key at or above the bound becomes a
// candidate, and the candidates are ranked exactly by counting on the 64-bit keys (score, then lower row).  Three
// block barriers; nothing depends on the distribution of the scores.  More candidates than threads (massive ties,
// or the best rows all in a few warps) is the caller's cue to run topk_block instead.
// ------------------------------------------------------------------------------------------------
constexpr int kExtractMaxK = 256;   // largest k served this way
constexpr int kExtractMaxKpl = 8;   // keys per thread held in registers
struct ExtractShared {
  uint32_t sub[32 * 32];               // [warp][t]: the values of the warp's t best keys (0: the warp has fewer)
  int32_t plan_len[kExtractMaxK + 1];  // planning entries (placement order): length and source token of each
  int32_t plan_src[kExtractMaxK + 1];
  uint32_t bound;                      // the lower bound of the k-th largest key
  uint32_t n_cand;
};

__host__ __device__ __forceinline__ int extract_rounds(int k, int n_warps) { return (k + n_warps - 1) / n_warps + 1; }

// All THREADS threads call.  Returns true (the same in every thread) when the candidates fit one per thread: then every
// rank < min(n, k) is held by exactly one thread, which gets it in my_rank together with the key in my_key (score key
// in the upper half, 0xffffffff - row in the lower); the other threads get my_rank = -1.  When n < k the ranks from n
// on have no key.  Returns false otherwise; s_keys holds the n order keys for the fallback either way.
// `cand` is shared memory for THREADS 64-bit keys.
// key_at(i): the order key of place i < n, or 0 for an empty place (no finite score has key 0).
template <int THREADS, int KPL, class KeyAt>
__device__ __forceinline__ bool topk_extract_keys(ExtractShared& es, unsigned long long* cand, KeyAt key_at, uint32_t* s_keys, int n, int k,
                                                  int& my_rank, unsigned long long& my_key) {
  constexpr int NW = THREADS / 32;
  constexpr unsigned kFull = 0xffffffffu;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t = extract_rounds(k, NW);
  uint32_t key[KPL];
#pragma unroll
  for (int j = 0; j < KPL; ++j) {
    const int i = j * THREADS + tid;
    key[j] = i < n ? key_at(i) : 0u;
  }
  if (s_keys != nullptr) {  // (the caller's fallback wants them)
#pragma unroll
    for (int j = 0; j < KPL; ++j) {
      const int i = j * THREADS + tid;
      if (i < n) s_keys[i] = key[j];
    }
  }
  if (tid == 0) {
    es.bound = 0u;
    es.n_cand = 0u;
  }
  // the t largest DISTINCT values of this warp, largest first: lane r ends up with the r-th.  (Equal keys count once
  // here; a bound taken from distinct values, each held by at least one key, is still a lower bound.)
  uint32_t mine = 0u, prev = 0xffffffffu;
  for (int r = 0; r < t; ++r) {
    uint32_t hb = 0u;
#pragma unroll
    for (int j = 0; j < KPL; ++j) hb = max(hb, key[j] < prev ? key[j] : 0u);
    prev = __reduce_max_sync(kFull, hb);
    if (prev == 0u) break;  // the warp has no smaller value left (uniform)
    if (lane == r) mine = prev;
  }
  if (lane < t) es.sub[warp * t + lane] = mine;
  __syncwarp();
  __syncthreads();

  // the k-th largest of the warps' values: rank by counting, G lanes per value (equal values of different warps are
  // told apart by their place, so ranks are distinct)
  const int S = NW * t;
  int g_shift = 3;
  while (g_shift > 0 && (S << g_shift) > THREADS) --g_shift;
  {
    const int vi = tid >> g_shift, part = tid & ((1 << g_shift) - 1);
    const uint32_t v = vi < S ? es.sub[vi] : 0u;
    uint32_t rank = 0;
    if (vi < S)
      for (int j = part; j < S; j += 1 << g_shift) {
        const uint32_t o = es.sub[j];
        rank += (o > v) || (o == v && j < vi);
      }
    for (int o = 1; o < (1 << g_shift); o <<= 1) rank += __shfl_xor_sync(kFull, rank, o);
    if (vi < S && part == 0 && rank == (uint32_t)k - 1u) es.bound = v;  // stays 0 when fewer than k values exist: every key is a candidate
  }
  __syncwarp();
  __syncthreads();

  // candidates: every key at or above the bound, as 64-bit keys (score key, then lower row first)
  const uint32_t bound = es.bound;
#pragma unroll
  for (int j = 0; j < KPL; ++j) {
    const bool in = key[j] != 0u && key[j] >= bound;
    const unsigned votes = __ballot_sync(kFull, in);
    if (votes) {
      uint32_t base = 0;
      if (lane == 0) base = atomicAdd(&es.n_cand, (uint32_t)__popc(votes));
      base = __shfl_sync(kFull, base, 0);
      const uint32_t slot = base + (uint32_t)__popc(votes & ((1u << lane) - 1u));
      if (in && slot < (uint32_t)THREADS)
        cand[slot] = ((unsigned long long)key[j] << 32) | (uint32_t)(0xffffffffu - (uint32_t)(j * THREADS + tid));
    }
  }
  __syncwarp();
  __syncthreads();
  const uint32_t C = es.n_cand;
  my_rank = -1;
  my_key = 0ull;
  if (C > (uint32_t)THREADS) return false;
  if (C * 4u <= (uint32_t)THREADS) {
    // four lanes share a candidate and split the comparisons
    const uint32_t ci = (uint32_t)tid >> 2, part = (uint32_t)tid & 3u;
    const unsigned long long me = ci < C ? cand[ci] : 0ull;
    uint32_t rank = 0;
    for (uint32_t jj = part; jj < C; jj += 4) rank += cand[jj] > me;
    rank += __shfl_xor_sync(kFull, rank, 1);
    rank += __shfl_xor_sync(kFull, rank, 2);
    if (ci < C && part == 0 && rank < (uint32_t)k) {
      my_rank = (int)rank;
      my_key = me;
    }
  } else if (tid < (int)C) {
    const unsigned long long me = cand[tid];
    uint32_t rank = 0;
    for (uint32_t jj = 0; jj < C; ++jj) rank += cand[jj] > me;
    if (rank < (uint32_t)k) {
      my_rank = (int)rank;
      my_key = me;
    }
  }
  __syncwarp();
  return true;
}

template <int THREADS, int KPL>
__device__ __forceinline__ bool topk_extract(ExtractShared& es, unsigned long long* cand, const float* __restrict__ sc, uint32_t* s_keys,
                                             int n, int k, int& my_rank, unsigned long long& my_key) {
  return topk_extract_keys<THREADS, KPL>(es, cand, [&](int i) { return order_key(__ldcg(sc + i)); }, s_keys, n, k, my_rank, my_key);
}

// Scoring only (large segments): grid = (row groups, nq); dynamic shared memory holds the query as fp32.
template <typename T>
__global__ void __launch_bounds__(kScoreThreads) score_rows_kernel(const RetrieveParams p, int rows_per_cta) {
  extern __shared__ float s_q[];
  const int q = blockIdx.y;
  const int user = p.query_users ? p.query_users[q] : 0;
  const bool user_ok = user >= 0 && user < p.n_users;
  const int n = user_ok ? p.user_count[user] : 0;
  const int64_t row0 = (int64_t)blockIdx.x * rows_per_cta;
  if (row0 >= n) return;
  const T* qv = reinterpret_cast<const T*>(p.queries) + (int64_t)q * p.emb_dim;
  for (int d = threadIdx.x; d < p.emb_dim; d += kScoreThreads) s_q[d] = (float)qv[d];
  __syncthreads();
  score_rows<T>(p, s_q, q, user, n, row0, rows_per_cta);
}

// Top-k only (large segments): one CTA per query, keys recomputed from global scores.
__global__ void __launch_bounds__(kTopkThreads, 1) topk_kernel(const RetrieveParams p) {
  __shared__ TopkShared sm;
  const int q = blockIdx.x;
  const int user = p.query_users ? p.query_users[q] : 0;
  const bool user_ok = user >= 0 && user < p.n_users;
  const int n = user_ok ? p.user_count[user] : 0;
  topk_block<kTopkThreads>(sm, p.scores + (int64_t)q * p.score_stride, nullptr, n, p.k,
                           IdMap{nullptr, p.return_rows ? nullptr : p.emb_fact_id + (int64_t)(user_ok ? user : 0) * p.seg_capacity},
                           p.out_ids + (int64_t)q * p.k, p.out_scores ? p.out_scores + (int64_t)q * p.k : nullptr);
}

// Body of the fused scoring + top-k kernels below (PLAN: the last CTA of a query also plans its injection).
// early (PLAN only): the kernel was launched as a programmatic dependent and has NOT yet waited for the preceding grid;
// everything up to the selection reads only the store and the caller's inputs and writes only this library's scratch,
// and the wait comes right before the first write that a preceding kernel could still be concerned with.
template <typename T, int THREADS, bool PLAN>
__device__ __forceinline__ void score_topk_body(const RetrieveParams& p, int rows_per_cta, uint32_t* tickets, int keys_capacity,
                                                int n_host, const InjectParams* ip, bool early = false) {
  extern __shared__ uint32_t s_keys[];
  __shared__ TopkShared sm;
  __shared__ ExtractShared es;
  __shared__ PlanShared ps;
  __shared__ int32_t s_ids[PLAN ? kTopkMaxK : 1];  // the selected ids by rank, for the planning that follows in this CTA
  __shared__ int s_last;
  const int q = blockIdx.y;
  int user = 0, n = n_host;
  bool user_ok = true;
  if (n_host < 0) {
    user = p.query_users ? p.query_users[q] : 0;
    user_ok = user >= 0 && user < p.n_users;
    n = user_ok ? min(p.user_count[user], keys_capacity) : 0;
  }
  const int64_t row0 = (int64_t)blockIdx.x * rows_per_cta;
  if (row0 < n) score_rows_direct<T, THREADS / 32>(p, q, user, n, row0, rows_per_cta);
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();  // this CTA's scores are visible before its ticket is
    const uint32_t t = atomicAdd(&tickets[q], 1u);
    s_last = t == gridDim.x - 1;
    if (s_last) tickets[q] = 0;  // ready for the next call (calls on one store are ordered on the device)
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (PLAN) plan_prefetch<THREADS>(*ip, q, ps);  // in flight while the ids are being selected
  const float* sc = p.scores + (int64_t)q * p.score_stride;
  // with a single user segment facts are numbered in row order: the row is the fact id
  const int32_t* row_ids = (p.n_users == 1 || p.return_rows) ? nullptr : p.emb_fact_id + (int64_t)(user_ok ? user : 0) * p.seg_capacity;
  int32_t* out_ids = p.out_ids + (int64_t)q * p.k;
  float* out_scores = p.out_scores ? p.out_scores + (int64_t)q * p.k : nullptr;
  const int k = p.k;

  // ---- fast selection: a threshold from the warps' own best keys (see topk_extract) -------------------------
  bool done = false;
  const bool plan_fast = PLAN && k + (ip->prefix_len > 0 ? 1 : 0) <= kExtractMaxK + 1;
  if (k <= kExtractMaxK && n <= THREADS * kExtractMaxKpl && extract_rounds(k, THREADS / 32) <= 32 && (!PLAN || plan_fast)) {
    const int has_prefix = PLAN ? (ip->prefix_len > 0) : 0;
    if (PLAN) {
      // planning entries default to "nothing" (ranks beyond the segment); a fact's entry is filled in the moment
      // its rank is known, so the fact-table reads overlap one another and nothing waits for the id list
      for (int j = threadIdx.x; j < k + has_prefix; j += THREADS) {
        es.plan_len[j] = 0;
        es.plan_src[j] = 0;
      }
      if (threadIdx.x == 0) ps.status = 0;
    }
    auto pad = [&](int rank) {
      out_ids[rank] = -1;
      if (out_scores) out_scores[rank] = 0.f;
    };
    int my_rank = -1;
    unsigned long long my_key = 0ull;
    if (n <= THREADS) done = topk_extract<THREADS, 1>(es, sm.cand, sc, s_keys, n, k, my_rank, my_key);
    else if (n <= 2 * THREADS) done = topk_extract<THREADS, 2>(es, sm.cand, sc, s_keys, n, k, my_rank, my_key);
    else if (n <= 4 * THREADS) done = topk_extract<THREADS, 4>(es, sm.cand, sc, s_keys, n, k, my_rank, my_key);
    else done = topk_extract<THREADS, 8>(es, sm.cand, sc, s_keys, n, k, my_rank, my_key);
    if (done) {
      // the thread that holds a rank resolves the fact (store data only) ...
      int32_t id = -1;
      const bool gone = (uint32_t)(my_key >> 32) == kRemovedKey;  // a removed row that ranks because too few rows are left
      if (my_rank >= 0 && !gone) {
        const uint32_t row = 0xffffffffu - (uint32_t)my_key;
        id = row_ids ? row_ids[row] : (int32_t)row;
        if (PLAN) {
          const int j = has_prefix + ((ip->flags & 1u) ? (k - 1 - my_rank) : my_rank);
          const FactRec f = ip->facts[id];
          if (!f.resident) {
            atomicOr(&ps.status, 2 /*MS_REQ_NOT_RESIDENT*/);
          } else {
            es.plan_len[j] = f.n_tokens;
            es.plan_src[j] = f.resident == 2 ? (f.tok_off | kHostTierBit) : f.tok_off;
          }
        }
      }
      // ... and only then come the first writes outside this library's scratch
      if (PLAN && early) grid_dependency_wait();
      if (my_rank >= 0) {
        out_ids[my_rank] = id;
        if (out_scores) out_scores[my_rank] = gone ? 0.f : key_score((uint32_t)(my_key >> 32));
      }
      for (int r = n + (int)threadIdx.x; r < k; r += THREADS) pad(r);  // a segment shorter than k: the other ranks are empty
      if (PLAN) {
        __syncwarp();  // only some lanes resolved a fact: together again before the barrier
        __syncthreads();
        plan_request<THREADS, true, true>(*ip, q, es.plan_len, es.plan_src, ps, nullptr);
      }
      return;
    }
  } else {
    for (int i = threadIdx.x; i < n; i += THREADS) s_keys[i] = order_key(__ldcg(sc + i));
  }
  __syncthreads();
  if (PLAN && early) grid_dependency_wait();

  // ---- general selection (large k, long segments, or more candidates than threads) --------------------------
  topk_block<THREADS, false>(sm, sc, s_keys, n, k, IdMap{nullptr, row_ids, PLAN ? s_ids : nullptr}, out_ids, out_scores);
  if (PLAN) {
    // the ids of query q are request q's fact list: plan it right here (steps I1-I3), in the shared memory the
    // selection no longer needs, so that the copy kernel can follow without a separate planning launch
    __syncthreads();
    int32_t* s_begin = reinterpret_cast<int32_t*>(sm.cand);
    plan_request<THREADS, true>(*ip, q, s_begin, s_begin + kTopkMaxK, ps, s_ids);
  }
}

// Scoring + top-k in ONE launch for segments of at most kFusedMaxRows rows: grid = (row groups, nq).
// The CTA that finishes a query's scores last (a wait-free ticket) selects and sorts that query's top-k from
// keys held in shared memory (dynamic shared memory: keys_capacity uint32 keys).  n_host >= 0 is the row count
// of user 0 known to the host (no per-query users): it saves the dependent load of the device-side count.
template <typename T, int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS >= 1024 ? 1 : THREADS >= 512 ? 2 : 4) score_topk_fused_kernel(const RetrieveParams p, int rows_per_cta,
                                                                         uint32_t* tickets, int keys_capacity, int n_host) {
  grid_dependency_wait();    // launched as a programmatic dependent: nothing is touched before the preceding grid is done
  grid_launch_dependents();  // a kernel that follows as a programmatic dependent may be placed while this one drains
  score_topk_body<T, THREADS, false>(p, rows_per_cta, tickets, keys_capacity, n_host, nullptr);
}

// The same, and the last CTA of a query goes on to plan that query's injection request (memstore_retrieve_inject).
// early != 0 (the caller vouches that the queries, users, start positions and block tables were complete before the
// preceding work of the stream began): the scoring and the selection do not wait for the preceding grid - when that is
// this library's copy kernel, they run on the SMs it vacates while it drains - and only the last CTA of a query waits,
// right before it writes the ids and the plan.
template <typename T, int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS >= 1024 ? 1 : THREADS >= 512 ? 2 : 4) score_topk_plan_kernel(const RetrieveParams p, int rows_per_cta,
                                                                        uint32_t* tickets, int keys_capacity, int n_host,
                                                                        const __grid_constant__ InjectParams ip, int early) {
  if (!early) grid_dependency_wait();  // launched as a programmatic dependent: nothing is touched before the preceding grid is done
  grid_launch_dependents();  // the copy kernel may be scheduled early; it waits for this grid before reading the plan
  score_topk_body<T, THREADS, true>(p, rows_per_cta, tickets, keys_capacity, n_host, &ip, early != 0);
}

// ---- tensor-core path, steps 2 and 3 (step 1 is score_gemm_groupmax_kernel) -------------------------------------

// Step 2: per query, the k2 groups with the largest group maximum, written in ASCENDING group order (so that the
// candidate rows of step 3 are in row order and "lower index first" among equal scores means "lower fact id first").
__global__ void __launch_bounds__(kTopkThreads, 1) select_groups_kernel(const float* gmax, int64_t gmax_stride, int n_groups, int k2,
                                                                    int32_t* sel /*[nq][k2]*/, float* next_best /*[nq]*/) {
  __shared__ TopkShared sm;
  __shared__ int32_t s_sel[512];
  __shared__ float s_val[512];
  grid_dependency_wait();  // every kernel of this chain is a programmatic dependent of the one before it
  grid_launch_dependents();
  const int q = blockIdx.x;
  int32_t* out = sel + (int64_t)q * k2;
  // one group more than asked for: its maximum is the best score the filter saw among the rows that will NOT be
  // rescored, which the rescoring step compares with the k-th exact score it finds
  topk_block<kTopkThreads>(sm, gmax + (int64_t)q * gmax_stride, nullptr, n_groups, k2 + 1, IdMap{nullptr, nullptr}, s_sel, s_val);
  __syncthreads();
  if (threadIdx.x == 0) next_best[q] = n_groups > k2 ? s_val[k2] : -INFINITY;
  // order the chosen group indices ascending by counting (k2 <= 512 distinct indices; -1 padding, present only when
  // the segment has fewer than k2 groups, counts as the largest value and keeps its relative order)
  for (int i = threadIdx.x; i < k2; i += kTopkThreads) {
    const uint32_t mine = (uint32_t)s_sel[i];
    int rank = 0;
    for (int j = 0; j < k2; ++j) {
      const uint32_t other = (uint32_t)s_sel[j];
      rank += (other < mine) || (other == mine && j < i);
    }
    out[rank] = (int32_t)mine;
  }
}

// One row's score with the lane layout and summation order of score_rows (all lanes return the sum).
template <typename T>
__device__ __forceinline__ float score_one_row(const RetrieveParams& p, int q, const T* seg, int64_t row) {
  constexpr int VEC = 16 / sizeof(T);
  const int E = p.emb_dim;
  const int lane = threadIdx.x & 31;
  const uint4* qp = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(p.queries) + (int64_t)q * E);
  const uint4* rp = reinterpret_cast<const uint4*>(seg + row * E);
  const int nvec = E / VEC;
  float acc = 0.f;
  for (int v0 = 0; v0 < nvec; v0 += 128) {
    uint4 x[4], y[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int v = v0 + u * 32 + lane;
      if (v < nvec) {
        x[u] = __ldg(rp + v);
        y[u] = __ldg(qp + v);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int v = v0 + u * 32 + lane;
      if (v < nvec) {
        if (sizeof(T) == 2) {
          acc = dot8_f16(x[u], y[u], acc);
        } else {
          const float* f = reinterpret_cast<const float*>(&x[u]);
          const float* g = reinterpret_cast<const float*>(&y[u]);
#pragma unroll
          for (int i = 0; i < 4; ++i) acc = fmaf(f[i], g[i], acc);
        }
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  return acc;
}

constexpr float kTcFilterRounding = 1e-5f;  // tensor-core fp32 accumulation against the fixed-order CUDA-core sum, times max(1, |score|)
// The exact scores of the rows of the chosen groups: candidate c of the query is row sel[c / 8] * 8 + c % 8 (sel: the
// query's k2 groups in ascending order, -1 padded).  The calling warp takes the groups first, first + step, ...; two rows
// in flight at a time.  cs / cr: the query's candidate scores and rows ([k2 * 8], cr = -1 for an absent row).
template <typename T>
__device__ __forceinline__ void rescore_groups(const RetrieveParams& p, int q, const int32_t* sel, int k2, int n_rows, float* cs, int32_t* cr,
                                               int first, int step) {
  const int lane = threadIdx.x & 31;
  const T* seg = reinterpret_cast<const T*>(p.emb);  // user 0
  for (int g_idx = first; g_idx < k2; g_idx += step) {
    const int32_t g = sel[g_idx];
    for (int r = 0; r < 8; r += 2) {
      const int64_t row = (int64_t)g * 8 + r;
      const bool ok0 = g >= 0 && row < n_rows, ok1 = g >= 0 && row + 1 < n_rows;
      float s0 = -INFINITY, s1 = -INFINITY;
      if (ok1) {
        score_two_rows<T>(p, q, seg, row, row + 1, s0, s1);
        s0 += 0.0f;
        s1 += 0.0f;
      } else if (ok0) {
        s0 = score_one_row<T>(p, q, seg, row) + 0.0f;
      }
      // a removed row stays a candidate (the valid candidates must remain a prefix) with the score of a removed row
      if (ok0 && row_removed(p, 0, row)) s0 = -INFINITY;
      if (ok1 && row_removed(p, 0, row + 1)) s1 = -INFINITY;
      if (lane == 0) {
        cs[g_idx * 8 + r] = s0;
        cr[g_idx * 8 + r] = ok0 ? (int32_t)row : -1;
        cs[g_idx * 8 + r + 1] = s1;
        cr[g_idx * 8 + r + 1] = ok1 ? (int32_t)(row + 1) : -1;
      }
    }
  }
}

// The top-k of a query's rescored candidates (all THREADS threads of the CTA call, after the candidates have been
// written and made visible), and the margin check: when the k-th exact score does not beat `best_unscored` (the
// filter's best score among the rows that were not rescored) by more than the filter's rounding, a row outside the
// selected groups may belong to the top-k: redo[q] is raised and kth[q] tells the fix-up kernel which exact score a row
// must reach.  s_keys: shared memory for n_cand keys.
template <int THREADS>
__device__ __forceinline__ void rescore_select(const RetrieveParams& p, int q, TopkShared& sm, uint32_t* s_keys, const float* cs,
                                               const int32_t* cr, int n_cand, float* scores_out, float best_unscored, int* redo, float* kth) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // Candidates are in ascending row order with every absent one (padding group, row beyond the segment) at the
  // end, so the valid candidates are a prefix: count them and select among those only.
  int mine = 0;
  for (int i = threadIdx.x; i < n_cand; i += THREADS) mine += __ldcg(cr + i) >= 0;
  mine = __reduce_add_sync(0xffffffffu, mine);
  if (lane == 0) sm.warp_cnt[warp] = (uint32_t)mine;
  __syncthreads();
  int n_valid = 0;
  for (int w = 0; w < THREADS / 32; ++w) n_valid += (int)sm.warp_cnt[w];
  uint32_t lo = 0xffffffffu, hi = 0u;
  for (int i = threadIdx.x; i < n_valid; i += THREADS) {
    const uint32_t kx = order_key(__ldcg(cs + i));
    s_keys[i] = kx;
    if (kx != kRemovedKey) {
      lo = min(lo, kx);
      hi = max(hi, kx);
    }
  }
  __syncthreads();
  topk_block<THREADS, false>(sm, cs, s_keys, n_valid, p.k, IdMap{cr, p.return_rows ? nullptr : p.emb_fact_id}, p.out_ids + (int64_t)q * p.k,
                             scores_out + (int64_t)q * p.k, true, lo, hi);
  __syncthreads();
  if (threadIdx.x == 0) {
    int again = 0;
    float need = 0.f;
    if (n_valid >= p.k) {
      need = __ldcg(scores_out + (int64_t)q * p.k + p.k - 1);
      again = best_unscored >= need - kTcFilterRounding * fmaxf(1.f, fabsf(need));
    }
    redo[q] = again;
    kth[q] = need;
  }
}

// Step 3: grid = (groups of the query / warps per CTA, nq); a warp rescores one chosen group, the last CTA of a query
// (wait-free ticket) selects.  Dynamic shared memory: k2 * 8 uint32 keys.  `scores_out` ([nq][k], never NULL) receives
// the exact scores by rank.
template <typename T>
__global__ void __launch_bounds__(kScoreThreads) rescore_topk_kernel(const RetrieveParams p, const int32_t* sel, int k2, int n_rows,
                                                                     float* cand_scores, int32_t* cand_rows, uint32_t* tickets,
                                                                     float* scores_out, const float* next_best, int* redo, float* kth) {
  extern __shared__ uint32_t s_keys[];
  __shared__ TopkShared sm;
  __shared__ int s_last;
  grid_dependency_wait();
  grid_launch_dependents();
  const int q = blockIdx.y;
  const int n_cand = k2 * 8;
  float* cs = cand_scores + (int64_t)q * n_cand;
  int32_t* cr = cand_rows + (int64_t)q * n_cand;
  rescore_groups<T>(p, q, sel + (int64_t)q * k2, k2, n_rows, cs, cr, (int)blockIdx.x * kScoreWarps + (int)(threadIdx.x >> 5),
                    (int)gridDim.x * kScoreWarps);
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const uint32_t t = atomicAdd(&tickets[q], 1u);
    s_last = t == gridDim.x - 1;
    if (s_last) tickets[q] = 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  rescore_select<kScoreThreads>(p, q, sm, s_keys, cs, cr, n_cand, scores_out, next_best[q], redo, kth);
}

// Steps 2 and 3 in one launch when the filter kernel listed candidate rows (see score_gemm.cuh); grid = (kListCtas, nq).
// The candidates of a query sit in one segment of `seg` places per epilogue warp of the filter kernel, cand_cnt[q][segment]
// of them used, each (order key of the filter score << 32) | row.  EVERY CTA of a query gathers the used places into a
// dense list and takes the k2 candidates with the best filter scores (the same work in each: the list is a few hundred
// entries and nothing has to be exchanged); then the CTAs share the exact rescoring of those rows - the CUDA-core
// routine of the other kernels, a warp per two rows, so that the k2 scattered 2 KiB reads of a query come from several
// SMs at once - and the CTA that finishes last (a wait-free ticket) ranks them by (exact score, lower row first) and
// writes the top-k.  The margin check is that of rescore_topk_kernel; the best filter score among the rows that were
// NOT rescored is the (k2+1)-th candidate's or the highest threshold the filter applied (every row it did not list
// scored below that), whichever is larger.
// Fewer than k2 candidates in all, a warp that found more than its segment holds, a list longer than kListMaxRows, or
// more candidates tied at the cut than the selection ranks: the list is unusable and CTA 0 alone serves the query from
// the group maxima (the bodies of select_groups_kernel and rescore_topk_kernel: slower, about 0.1 ms, and rare).  The
// histogram and the threshold record of the query are left zeroed for the next call.  Dynamic shared memory: k2g * 8
// uint32 keys.
constexpr int kListThreads = 512;
constexpr int kListCtas = 4;
constexpr int kListMaxRows = 2048;
constexpr int kListMaxK2 = 288;  // rows rescored per query: the largest k of the filter path (256) and the margin
constexpr int kCandMaxSegs = 1024;
template <typename T>
__global__ void __launch_bounds__(kListThreads, 1)
    list_topk_kernel(const RetrieveParams p, const unsigned long long* cand, int n_seg, int seg, const uint32_t* cand_cnt, uint32_t* thr_used,
                     uint32_t* hist, int hist_words, uint32_t* calib, int k2, float* exact /*[nq][k2]*/, uint32_t* tickets, float* scores_out, int* redo,
                     float* kth, unsigned long long* list_stats /*served, rows listed, fallbacks*/, const float* gmax, int64_t gmax_stride,
                     int n_groups, int k2g, int n_rows, float* cand_scores /*[nq][k2g * 8]*/, int32_t* cand_rows, uint32_t* raw,
                     int raw_stride, int n_raw) {
  extern __shared__ uint32_t s_dyn[];
  __shared__ ExtractShared es;
  __shared__ TopkShared sm;  // (the group selection of an unusable list; its candidate array also serves the row selection)
  __shared__ uint16_t s_list[kListMaxRows];  // the used places, segment by segment
  __shared__ int32_t s_rows[512];            // the chosen rows by filter rank (or the chosen groups)
  __shared__ float s_val[512];               // their exact scores (or the groups' maxima)
  __shared__ unsigned long long s_key[kListMaxK2];
  __shared__ uint32_t s_wtot[kListThreads / 32];
  __shared__ float s_next, s_kth;
  __shared__ int s_last;
  constexpr unsigned kFull = 0xffffffffu;
  grid_dependency_wait();
  grid_launch_dependents();
  const int q = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    s_next = -INFINITY;
    s_kth = 0.f;
  }
  // ---- the used places of all segments, densely (block-wide exclusive scan of the segments' counts)
  uint32_t n = 0;
  int overrun = 0;
  for (int c0 = 0; c0 < n_seg; c0 += kListThreads) {
    const int i = c0 + tid;
    uint32_t c = i < n_seg ? cand_cnt[(size_t)q * n_seg + i] : 0u;
    overrun |= c > (uint32_t)seg;
    c = min(c, (uint32_t)seg);
    uint32_t incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(kFull, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) s_wtot[warp] = incl;
    __syncthreads();
    uint32_t before = 0, total = 0;
    for (int w = 0; w < kListThreads / 32; ++w) {
      const uint32_t t = s_wtot[w];
      before += w < warp ? t : 0u;
      total += t;
    }
    const uint32_t at = n + before + incl - c;
    for (uint32_t j = 0; j < c; ++j)
      if (at + j < (uint32_t)kListMaxRows) s_list[at + j] = (uint16_t)(i * seg + (int)j);
    n += total;
    __syncthreads();
  }
  overrun = __syncthreads_or(overrun);
  if (blockIdx.x == 0) {  // clean for the next call (only this kernel's CTA 0 of the query touches the histogram)
    uint4* hq = reinterpret_cast<uint4*>(hist + (size_t)q * hist_words);  // hist_words is a multiple of 4
    for (int i = tid; i < hist_words / 4; i += kListThreads) hq[i] = make_uint4(0u, 0u, 0u, 0u);
    for (int i = tid; i < n_raw; i += kListThreads) raw[(size_t)q * raw_stride + i] = 0xffffffffu;  // the calibration table: empty
    if (tid < 4) calib[(size_t)q * 4 + tid] = 0u;
  }
  const int n_places = n_seg * seg;
  bool ok = !overrun && n >= (uint32_t)k2 && n <= (uint32_t)kListMaxRows && k2 <= kListMaxK2 && n_places <= 65536;
  int my_rank = -1;
  unsigned long long my_key = 0ull;
  const unsigned long long* mine = cand + (size_t)q * n_places;
  if (ok) {
    auto key_at = [&](int i) { return (uint32_t)(__ldcg(mine + s_list[i]) >> 32); };
    if (n <= (uint32_t)kListThreads) ok = topk_extract_keys<kListThreads, 1>(es, sm.cand, key_at, nullptr, (int)n, k2 + 1, my_rank, my_key);
    else if (n <= 2u * kListThreads) ok = topk_extract_keys<kListThreads, 2>(es, sm.cand, key_at, nullptr, (int)n, k2 + 1, my_rank, my_key);
    else ok = topk_extract_keys<kListThreads, 4>(es, sm.cand, key_at, nullptr, (int)n, k2 + 1, my_rank, my_key);
  }
  if (!ok) {
    // ---- the list is unusable: CTA 0 serves the query from the group maxima
    if (blockIdx.x != 0) return;
    __syncthreads();
    topk_block<kListThreads>(sm, gmax + (int64_t)q * gmax_stride, nullptr, n_groups, k2g + 1, IdMap{nullptr, nullptr}, s_rows, s_val);
    __syncthreads();
    const float best_unscored = n_groups > k2g ? s_val[k2g] : -INFINITY;
    if (tid == 0) {
      atomicAdd(list_stats + 2, 1ull);
      thr_used[q] = 0u;
    }
    __syncthreads();
    int32_t* groups = reinterpret_cast<int32_t*>(s_val);  // the chosen groups in ascending order (by counting, as select_groups_kernel)
    for (int i = tid; i < k2g; i += kListThreads) {
      const uint32_t me = (uint32_t)s_rows[i];
      int rank = 0;
      for (int j = 0; j < k2g; ++j) {
        const uint32_t other = (uint32_t)s_rows[j];
        rank += (other < me) || (other == me && j < i);
      }
      groups[rank] = (int32_t)me;
    }
    __syncthreads();
    float* cs = cand_scores + (int64_t)q * k2g * 8;
    int32_t* cr = cand_rows + (int64_t)q * k2g * 8;
    rescore_groups<T>(p, q, groups, k2g, n_rows, cs, cr, warp, kListThreads / 32);
    __syncthreads();
    rescore_select<kListThreads>(p, q, sm, s_dyn, cs, cr, k2g * 8, scores_out, best_unscored, redo, kth);
    return;
  }
  if (my_rank >= 0) {
    if (my_rank < k2) s_rows[my_rank] = (int32_t)(uint32_t)__ldcg(mine + s_list[0xffffffffu - (uint32_t)my_key]);
    else s_next = key_score((uint32_t)(my_key >> 32));
  }
  __syncwarp();
  __syncthreads();
  // ---- exact scores: this CTA takes the ranks blockIdx.x, blockIdx.x + kListCtas, ...; a warp two of them at a time
  const T* seg_rows = reinterpret_cast<const T*>(p.emb);  // user 0
  float* ex = exact + (int64_t)q * k2;
  constexpr int kWarps = kListThreads / 32;
  for (int j = warp; (int)blockIdx.x + kListCtas * j < k2; j += 2 * kWarps) {
    const int ra = (int)blockIdx.x + kListCtas * j, rb = ra + kListCtas * kWarps;
    float s0, s1 = 0.f;
    if (rb < k2) score_two_rows<T>(p, q, seg_rows, (int64_t)s_rows[ra], (int64_t)s_rows[rb], s0, s1);
    else s0 = score_one_row<T>(p, q, seg_rows, (int64_t)s_rows[ra]);
    if (lane == 0) {
      ex[ra] = s0 + 0.0f;
      if (rb < k2) ex[rb] = s1 + 0.0f;
    }
  }
  __syncwarp();
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    const uint32_t t = atomicAdd(&tickets[q], 1u);
    s_last = t == gridDim.x - 1;
    if (s_last) tickets[q] = 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (tid < k2) {
    const float sc = __ldcg(ex + tid);
    s_val[tid] = sc;
    s_key[tid] = ((unsigned long long)order_key(sc) << 32) | (0xffffffffu - (uint32_t)s_rows[tid]);
  }
  const uint32_t tk = thr_used[q];
  __syncthreads();
  // ---- rank by counting, two lanes per candidate when the threads allow (the rows are distinct, so the keys are)
  {
    const int per = 2 * k2 <= kListThreads ? 2 : 1;
    const int ci = per == 2 ? tid >> 1 : tid, part = per == 2 ? tid & 1 : 0;
    const unsigned long long me = ci < k2 ? s_key[ci] : 0ull;
    uint32_t rank = 0;
    if (ci < k2)
      for (int j = part; j < k2; j += per) rank += s_key[j] > me;
    if (per == 2) rank += __shfl_xor_sync(kFull, rank, 1);
    if (ci < k2 && part == 0 && rank < (uint32_t)p.k) {
      const int32_t row = s_rows[ci];
      p.out_ids[(int64_t)q * p.k + rank] = (p.return_rows || p.emb_fact_id == nullptr) ? row : p.emb_fact_id[row];
      scores_out[(int64_t)q * p.k + rank] = s_val[ci];
      if (rank == (uint32_t)p.k - 1u) s_kth = s_val[ci];
    }
  }
  __syncwarp();
  __syncthreads();
  if (tid == 0) {
    const float need = s_kth;
    const float nb = fmaxf(s_next, tk ? key_score(tk) : -INFINITY);
    atomicAdd(list_stats, 1ull);
    atomicAdd(list_stats + 1, (unsigned long long)n);
    thr_used[q] = 0u;
    redo[q] = nb >= need - kTcFilterRounding * fmaxf(1.f, fabsf(need));
    kth[q] = need;
  }
}

// Fix-up of the tensor-core path for the queries whose margin check failed (rare: more groups than the margin within
// rounding of the k-th score - near-duplicate rows spread over many groups).  Launched after every rescoring; CTAs of
// queries that passed leave at once.  For a flagged query every row of the segment is scored exactly (the CUDA-core
// routine of the other kernels) and the rows that reach kth[q] - every row of the true top-k does - are collected as
// 64-bit keys; the last CTA of the query sorts them and writes the top-k.  More collected rows than `cap` (thousands
// of rows within rounding of one another) leave the filter's answer in place and raise *overflow.
constexpr int kFixupCap = 4096;
template <typename T>
__global__ void __launch_bounds__(kScoreThreads) tc_fixup_kernel(const RetrieveParams p, int n_rows, int rows_per_cta, int* redo, const float* kth,
                                                                 uint32_t* counts, unsigned long long* keys /*[nq][kFixupCap]*/,
                                                                 uint32_t* tickets, float* scores_out, int* overflow, uint32_t* n_fixups) {
  extern __shared__ unsigned long long s_fix[];  // kFixupCap keys
  __shared__ int s_last;
  grid_dependency_wait();
  const int q = blockIdx.y;
  if (!redo[q]) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const T* seg = reinterpret_cast<const T*>(p.emb);  // user 0
  const float need = kth[q];
  const int64_t row0 = (int64_t)blockIdx.x * rows_per_cta, row_end = min(row0 + rows_per_cta, (int64_t)n_rows);
  unsigned long long* mine = keys + (int64_t)q * kFixupCap;
  for (int64_t row = row0 + 2 * warp; row < row_end; row += 2 * kScoreWarps) {
    float s0, s1 = -INFINITY;
    if (row + 1 < row_end) {
      score_two_rows<T>(p, q, seg, row, row + 1, s0, s1);
      s1 += 0.0f;
    } else {
      s0 = score_one_row<T>(p, q, seg, row);
    }
    s0 += 0.0f;
    if (row_removed(p, 0, row)) s0 = -INFINITY;
    if (row + 1 < row_end && row_removed(p, 0, row + 1)) s1 = -INFINITY;
    if (lane == 0) {
      if (s0 >= need) {
        const uint32_t slot = atomicAdd(&counts[q], 1u);
        if (slot < (uint32_t)kFixupCap) mine[slot] = ((unsigned long long)order_key(s0) << 32) | (uint32_t)(0xffffffffu - (uint32_t)row);
      }
      if (s1 >= need) {
        const uint32_t slot = atomicAdd(&counts[q], 1u);
        if (slot < (uint32_t)kFixupCap) mine[slot] = ((unsigned long long)order_key(s1) << 32) | (uint32_t)(0xffffffffu - (uint32_t)(row + 1));
      }
    }
  }
  __syncwarp();
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const uint32_t t = atomicAdd(&tickets[q], 1u);
    s_last = t == gridDim.x - 1;
    if (s_last) tickets[q] = 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const uint32_t n = __ldcg(&counts[q]);
  __syncthreads();
  if (threadIdx.x == 0) {
    counts[q] = 0;
    redo[q] = 0;
    atomicAdd(n_fixups, 1u);
    if (n > (uint32_t)kFixupCap) atomicExch(overflow, 1);
  }
  if (n > (uint32_t)kFixupCap || n < (uint32_t)p.k) return;  // (fewer than k cannot happen: the k rescored rows reach kth)
  int P2 = 1;
  while (P2 < (int)n) P2 <<= 1;
  for (int i = threadIdx.x; i < P2; i += kScoreThreads) s_fix[i] = i < (int)n ? __ldcg(mine + i) : 0ull;
  __syncthreads();
  bitonic_sort_desc<kScoreThreads>(s_fix, P2);
  write_topk<kScoreThreads>(s_fix, p.k, p.k, IdMap{nullptr, p.return_rows ? nullptr : p.emb_fact_id}, p.out_ids + (int64_t)q * p.k,
                            scores_out + (int64_t)q * p.k);
}

}  // namespace ms
