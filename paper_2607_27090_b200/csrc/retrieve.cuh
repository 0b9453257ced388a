// Exact retrieval: inner-product scoring of query embeddings against every fact of the query's user
// (R2) and top-k selection with "higher score first, equal scores: lower fact id first" (R3).
// Paper: Sec. 3.2 (top-k search by embedding similarity returning fact ids; inner product, Sec. 6.1).
#pragma once
#include "common.cuh"

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
};

constexpr int kScoreThreads = 256;
constexpr int kScoreWarps = kScoreThreads / 32;

__device__ __forceinline__ void unpack8(const uint4& v, float* f, const __half*) {
  const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 t = __half22float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

// ------------------------------------------------------------------------------------------------
// Scoring on CUDA cores: one warp per embedding row, 16-byte loads, fp32 accumulation.
// The summation order of a row depends only on the lane layout, never on which warp or CTA handles
// it, so identical rows get bit-identical scores (needed for the id tie rule).
// grid = (row groups, nq); dynamic shared memory holds the query as fp32.
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kScoreThreads) score_rows_kernel(const RetrieveParams p, int rows_per_cta) {
  extern __shared__ float s_q[];
  constexpr int VEC = 16 / sizeof(T);  // elements per 16-byte vector
  const int q = blockIdx.y;
  const int user = p.query_users ? p.query_users[q] : 0;
  const bool user_ok = user >= 0 && user < p.n_users;
  const int n = user_ok ? p.user_count[user] : 0;
  const int64_t row0 = (int64_t)blockIdx.x * rows_per_cta;
  if (row0 >= n) return;
  const int E = p.emb_dim;
  const T* qv = reinterpret_cast<const T*>(p.queries) + (int64_t)q * E;
  for (int d = threadIdx.x; d < E; d += kScoreThreads) s_q[d] = (float)qv[d];
  __syncthreads();

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
            unpack8(x[u], f, (const __half*)nullptr);
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
    if (lane == 0) p.scores[(int64_t)q * p.score_stride + row] = acc + 0.0f;  // -0 -> +0
  }
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

constexpr int kTopkThreads = 1024;
constexpr int kTopkMaxK = 2048;

// ------------------------------------------------------------------------------------------------
// Top-k: one CTA per query.  Radix select (4 passes of 8 bits, most significant first) finds the
// k-th largest score key T; everything above T is taken, rows equal to T are taken lowest row first
// (rows of a user are in fact-id order), and the k survivors are sorted by a bitonic network on the
// 64-bit key (score key << 32) | ~row.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTopkThreads) topk_kernel(const RetrieveParams p) {
  __shared__ uint32_t s_hist[256];
  __shared__ unsigned long long s_cand[kTopkMaxK];
  __shared__ uint32_t s_prefix, s_krem, s_ngt, s_warp_cnt[kTopkThreads / 32], s_eq_base;

  const int q = blockIdx.x;
  const int tid = threadIdx.x;
  const int user = p.query_users ? p.query_users[q] : 0;
  const bool user_ok = user >= 0 && user < p.n_users;
  const int n = user_ok ? p.user_count[user] : 0;
  const int k = p.k;
  const float* sc = p.scores + (int64_t)q * p.score_stride;
  const int take = min(n, k);

  uint32_t T = 0;        // threshold key
  uint32_t need_eq = 0;  // how many rows with key == T to take
  if (n > k) {
    if (tid == 0) {
      s_prefix = 0;
      s_krem = (uint32_t)k;
    }
    for (int shift = 24; shift >= 0; shift -= 8) {
      if (tid < 256) s_hist[tid] = 0;
      __syncthreads();
      const uint32_t prefix = s_prefix;
      const uint32_t himask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
      for (int i = tid; i < n; i += kTopkThreads) {
        const uint32_t kx = order_key(sc[i]);
        if ((kx & himask) == prefix) atomicAdd(&s_hist[(kx >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (tid == 0) {
        // walk buckets from the top: find b with count(> b) < krem <= count(>= b)
        uint32_t krem = s_krem, above = 0;
        int b = 255;
        for (; b > 0; --b) {
          if (above + s_hist[b] >= krem) break;
          above += s_hist[b];
        }
        s_prefix = prefix | ((uint32_t)b << shift);
        s_krem = krem - above;
      }
      __syncthreads();
    }
    T = s_prefix;
    need_eq = s_krem;
  }
  if (tid == 0) {
    s_ngt = 0;
    s_eq_base = 0;
  }
  for (int i = tid; i < kTopkMaxK; i += kTopkThreads) s_cand[i] = 0ull;
  __syncthreads();

  if (n <= k) {
    for (int i = tid; i < n; i += kTopkThreads)
      s_cand[i] = ((unsigned long long)order_key(sc[i]) << 32) | (uint32_t)(0xffffffffu - (uint32_t)i);
  } else {
    const uint32_t n_gt = (uint32_t)k - need_eq;
    // rows above the threshold: order does not matter, they are sorted afterwards
    // rows equal to the threshold: ordered compaction, lowest rows first, stop after need_eq
    const int lane = tid & 31, warp = tid >> 5;
    for (int base = 0; base < n; base += kTopkThreads) {
      const int i = base + tid;
      uint32_t kx = 0;
      bool gt = false, eq = false;
      if (i < n) {
        kx = order_key(sc[i]);
        gt = kx > T;
        eq = kx == T;
      }
      if (gt) {
        const uint32_t slot = atomicAdd(&s_ngt, 1u);
        if (slot < n_gt) s_cand[slot] = ((unsigned long long)kx << 32) | (uint32_t)(0xffffffffu - (uint32_t)i);
      }
      const uint32_t bal = __ballot_sync(0xffffffffu, eq);
      if (__syncthreads_or(eq)) {
        if (lane == 0) s_warp_cnt[warp] = __popc(bal);
        __syncthreads();
        uint32_t before = s_eq_base;
        for (int w = 0; w < warp; ++w) before += s_warp_cnt[w];
        if (eq) {
          const uint32_t rank = before + __popc(bal & ((1u << lane) - 1u));
          if (rank < need_eq) s_cand[n_gt + rank] = ((unsigned long long)kx << 32) | (uint32_t)(0xffffffffu - (uint32_t)i);
        }
        __syncthreads();
        if (tid == 0) {
          uint32_t tot = 0;
          for (int w = 0; w < kTopkThreads / 32; ++w) tot += s_warp_cnt[w];
          s_eq_base += tot;
        }
        __syncthreads();
      }
    }
  }
  __syncthreads();

  // bitonic sort, descending, over the next power of two >= take (padding keys are 0 = smallest)
  int P = 1;
  while (P < take) P <<= 1;
  for (int size = 2; size <= P; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int t = tid; t < P / 2; t += kTopkThreads) {
        const int lo = 2 * t - (t & (stride - 1));
        const int hi = lo + stride;
        const bool desc = (lo & size) == 0;
        const unsigned long long a = s_cand[lo], b = s_cand[hi];
        if ((a < b) == desc) {
          s_cand[lo] = b;
          s_cand[hi] = a;
        }
      }
      __syncthreads();
    }
  }

  const int32_t* row_ids = p.emb_fact_id + (int64_t)(user_ok ? user : 0) * p.seg_capacity;
  for (int r = tid; r < k; r += kTopkThreads) {
    int32_t id = -1;
    float s = 0.f;
    if (r < take) {
      const unsigned long long c = s_cand[r];
      const uint32_t row = 0xffffffffu - (uint32_t)(c & 0xffffffffull);
      id = row_ids[row];
      s = key_score((uint32_t)(c >> 32));
    }
    p.out_ids[(int64_t)q * k + r] = id;
    if (p.out_scores) p.out_scores[(int64_t)q * k + r] = s;
  }
}

}  // namespace ms
