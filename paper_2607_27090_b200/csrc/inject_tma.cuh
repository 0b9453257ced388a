// Injection copy kernel, bulk-async (TMA) staged version for sm_100a (steps I4 + I5).
//
// One persistent CTA per SM runs three roles over a ring of shared-memory stages:
//   warp 0       producer : cp.async.bulk global -> shared of the K and V rows of a stage, completion on an mbarrier
//   warp 1       V store  : cp.async.bulk shared -> global of the V rows (V never enters a register)
//   warps 2..9   K rotate : read K rows from shared memory, RoPE in fp32, 16-byte stores into the cache
// A stage holds the rows of up to 8 tokens of one tile for one layer (at most 16 KiB of K and 16 KiB of V).
// Work is claimed dynamically in chunks of a few consecutive layers of one sub-tile (one atomic ticket each), so
// the position-dependent cos/sin of a thread are computed once per chunk and reused over heads and layers.
//
// Every wait on an mbarrier is bounded; on a time-out the kernel raises MS_REQ_KERNEL_TIMEOUT in every
// request's status word, stops issuing work and leaves.  All copies are plain CTA-local bulk copies.
#pragma once
#include "inject.cuh"

namespace ms {

constexpr int kTmaStages = 6;
constexpr int kTmaAreaBytes = 16384;  // K area and V area of one stage
constexpr int kTmaConsumerWarps = 8;
constexpr int kTmaThreads = (2 + kTmaConsumerWarps) * 32;
constexpr uint32_t kSpinLimit = 1u << 22;  // x >= 64 ns: about a quarter of a second

struct __align__(16) StageMeta {
  int64_t dst_off[kTileTokens];
  int32_t pos0;      // position of token 0 of the stage
  uint32_t valid;    // bit t: token t present
  int32_t layer;
  uint32_t tsub;     // tile * n_sub + sub (changes when positions change)
};

constexpr size_t kTmaSmemBytes = (size_t)kTmaStages * 2 * kTmaAreaBytes + kTmaStages * sizeof(StageMeta) + 2 * kTmaStages * 8 + 16;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("{ .reg .b64 st; mbarrier.arrive.shared::cta.b64 st, [%0]; }" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
// Bounded wait for the phase with the given parity.  Returns false on time-out or when another role gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, uint32_t limit = kSpinLimit) {
  const uint32_t addr = smem_u32(bar);
  for (uint32_t spin = 0; spin < limit; ++spin) {
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok)
        : "r"(addr), "r"(parity)
        : "memory");
    if (ok) return true;
    if (spin > 32) {
      if (*abort_flag) return false;
      __nanosleep(64);
    }
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          smem_u32(smem_dst)),
      "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}

// ts = tokens per stage (8, 4, 2 or 1, with ts * row bytes <= kTmaAreaBytes); v_rows: 1 = a token's V row is
// contiguous in the cache (head_stride == head_dim), 0 = store head by head.
template <int STYLE>
__global__ void __launch_bounds__(kTmaThreads, 1) inject_copy_tma_kernel(const InjectParams p, const int ts, const int v_rows) {
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* const stages = smem;
  StageMeta* const meta = reinterpret_cast<StageMeta*>(smem + (size_t)kTmaStages * 2 * kTmaAreaBytes);
  uint64_t* const full = reinterpret_cast<uint64_t*>(meta + kTmaStages);
  uint64_t* const empty = full + kTmaStages;
  volatile int* const abort_flag = reinterpret_cast<volatile int*>(empty + kTmaStages);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int D = p.head_dim, H = p.n_heads, L = p.n_layers;
  const int row_bytes = H * D * 2;
  const uint32_t limit = p.spin_limit ? p.spin_limit : kSpinLimit;  // (a test shortens the waits, see memstore_test_hooks)

  if (threadIdx.x == 0) {
    for (int s = 0; s < kTmaStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], kTmaConsumerWarps + 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  grid_dependency_wait();  // tile descriptors come from the plan kernel

  const uint32_t n_tiles = min(p.ctrl->n_tiles, p.tiles_capacity);
  const int n_sub = kTileTokens / ts;
  const uint32_t n_ts = n_tiles * n_sub;
  // Work is handed out dynamically in chunks = (sub-tile, group of `lg` consecutive layers): SMs do not all get the
  // same memory service rate, and equal static shares leave the fast ones idle at the end.  A chunk is one atomic
  // ticket; its stages share positions, so a consumer thread computes its cos/sin once per chunk.
  const int lg = p.layers_per_item;
  const uint32_t n_lg = (uint32_t)((L + lg - 1) / lg);
  const uint32_t n_chunks = n_ts * n_lg;

  if (warp == 0 && p.mute_producer) {
    // test aid: this role issues nothing at all (no copy is ever in flight), so the other roles' waits run out
  } else if (warp == 0) {
    // ---------------------------------------------------------------- producer
    // Lanes 0..7 hold token t of the stage for K, lanes 8..15 the same tokens for V.  Rows that follow one
    // another in the arena (tokens of one fact) are fetched by ONE bulk copy issued by the first lane of the run.
    const uint64_t pol = policy_evict_first();
    const int t = lane & 7;
    const bool is_k = lane < 8, is_v = lane >= 8 && lane < 16;
    auto ticket = [&]() -> uint32_t {
      uint32_t c = 0;
      if (lane == 0) c = atomicAdd(&p.ctrl->work_next, 1u);
      return c;  // only lane 0's value is meaningful until broadcast
    };
    // two tickets and one descriptor are always in flight, so neither latency is exposed
    uint32_t c0 = __shfl_sync(0xffffffffu, ticket(), 0);
    uint32_t c1_raw = ticket();
    int32_t src_n = -1, pos0_n = 0;
    int64_t dst_n = 0;
    auto load_desc = [&](uint32_t chunk) {
      src_n = -1;
      if (chunk < n_chunks) {
        const uint32_t tsub = chunk / n_lg;
        const TileDesc* d = p.tiles + tsub / n_sub;
        const int sub = tsub % n_sub;
        if (lane < 16 && t < ts) {
          src_n = d->src_tok[sub * ts + t];
          dst_n = d->dst_off[sub * ts + t];
        }
        pos0_n = d->pos0 + sub * ts;
      }
    };
    load_desc(c0);
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    while (ok && c0 < n_chunks) {
      // promote the prefetched descriptor, start the next ticket and the next descriptor
      const int32_t src = src_n, pos0 = pos0_n;
      const int64_t dst = dst_n;
      const uint32_t c1 = __shfl_sync(0xffffffffu, c1_raw, 0);
      c1_raw = ticket();
      load_desc(c1);
      const int l0 = (int)(c0 % n_lg) * lg, l1 = min(l0 + lg, L);
      const uint32_t valid = __ballot_sync(0xffffffffu, is_k && src >= 0);
      // run starts: a valid token whose predecessor is absent or not the previous arena token
      const int32_t prev_src = __shfl_up_sync(0xffffffffu, src, 1);
      const bool start = src >= 0 && (t == 0 || prev_src < 0 || prev_src + 1 != src);
      const uint32_t starts = __ballot_sync(0xffffffffu, is_k && start);
      // rows in the run that begins at t: up to the next start or the next absent token
      const uint32_t stop = (starts | (~valid & 0xffu)) >> (t + 1);
      const int to_next = stop ? __ffs((int)stop) : (8 - t);
      const uint32_t run_rows = (start && (is_k || is_v)) ? (uint32_t)min(to_next, 8 - t) : 0u;
      for (int layer = l0; layer < l1; ++layer) {
        ok = mbar_wait(&empty[s], ph ^ 1u, abort_flag, limit);
        if (!ok) break;
        if (is_k) meta[s].dst_off[t] = dst;
        if (lane == 0) {
          meta[s].pos0 = pos0;
          meta[s].valid = valid;
          meta[s].layer = layer;
          meta[s].tsub = c0;  // consumers recompute cos/sin when this changes
        }
        __syncwarp();  // every lane's part of meta[s] is written before the barrier can complete
        if (lane == 0) mbar_arrive_expect_tx(&full[s], (uint32_t)__popc(valid) * 2u * (uint32_t)row_bytes);
        __syncwarp();  // the expected byte count is registered before any copy can complete
        if (run_rows) {
          const __nv_bfloat16* g = (is_k ? p.k_arena : p.v_arena) + ((int64_t)layer * p.arena_tokens + src) * (int64_t)(H * D);
          uint8_t* sdst = stages + (size_t)s * 2 * kTmaAreaBytes + (is_k ? 0 : kTmaAreaBytes) + (size_t)t * row_bytes;
          bulk_load(sdst, g, run_rows * (uint32_t)row_bytes, &full[s], pol);
        }
        if (++s == kTmaStages) {
          s = 0;
          ph ^= 1u;
        }
      }
      c0 = c1;
    }
    // end marker: a stage with layer = -1 tells the other roles that no more work will come
    if (ok && mbar_wait(&empty[s], ph ^ 1u, abort_flag, limit)) {
      if (lane == 0) {
        meta[s].layer = -1;
        meta[s].valid = 0;
        mbar_arrive_expect_tx(&full[s], 0u);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- V store
    // Lane t < 8 owns token t.  Rows that follow one another in the cache (same block, token_stride == row)
    // leave in ONE bulk store issued by the first lane of the run.
    int prev = -1;
    int s = 0;
    uint32_t ph = 0;
    const int t = lane & 7;
    for (;;) {
      if (!mbar_wait(&full[s], ph, abort_flag, limit)) break;
      const int layer = meta[s].layer;
      if (layer < 0) break;
      const uint32_t valid = meta[s].valid;
      const int64_t lbase = (int64_t)layer * p.layer_stride;
      const uint8_t* vsm = stages + (size_t)s * 2 * kTmaAreaBytes + kTmaAreaBytes;
      if (v_rows) {
        const bool ok = lane < 8 && ((valid >> t) & 1u);
        const int64_t d = meta[s].dst_off[t];
        const int64_t prev_d = __shfl_up_sync(0xffffffffu, d, 1);
        const bool prev_ok = __shfl_up_sync(0xffffffffu, (int)ok, 1) != 0;
        const bool start = ok && (t == 0 || !prev_ok || prev_d + (int64_t)(H * D) != d);
        const uint32_t starts = __ballot_sync(0xffffffffu, start);
        if (start) {
          const uint32_t stop = (starts | (~valid & 0xffu)) >> (t + 1);
          const int rows = min(stop ? __ffs((int)stop) : (8 - t), 8 - t);
          bulk_store(p.v_cache + lbase + d, vsm + (size_t)t * row_bytes, (uint32_t)(rows * row_bytes));
        }
      } else {
        for (int u = lane; u < ts * H; u += 32) {
          const int tt = u / H, h = u % H;
          if ((valid >> tt) & 1u)
            bulk_store(p.v_cache + lbase + meta[s].dst_off[tt] + (int64_t)h * p.head_stride,
                       vsm + (size_t)tt * row_bytes + (size_t)h * D * 2, (uint32_t)(D * 2));
        }
      }
      bulk_commit();
      bulk_wait_read<1>();  // the stores of the previous stage have finished reading shared memory
      __syncwarp();
      if (lane == 0 && prev >= 0) mbar_arrive(&empty[prev]);
      prev = s;
      if (++s == kTmaStages) {
        s = 0;
        ph ^= 1u;
      }
    }
    bulk_wait_all();
    __syncwarp();
    if (lane == 0 && prev >= 0) mbar_arrive(&empty[prev]);
  } else {
    // ---------------------------------------------------------------- K rotate + store
    const int ctid = threadIdx.x - 64;
    const int tpt = (kTmaConsumerWarps * 32) / ts;  // threads per token (a power of two >= 32)
    const int t = ctid / tpt, l = ctid % tpt;
    const int G = D >> 4, g_shift = 31 - __clz(G);  // frequency octets per head (a power of two)
    const int j = l & (G - 1);                      // octet of every unit of this thread (G divides tpt)
    const int n_units = H * G;
    const int offA = STYLE == 0 ? 8 * j : 16 * j;
    const int offB = STYLE == 0 ? D / 2 + 8 * j : 16 * j + 8;
    float f8[8], sn[8], cs[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) f8[q] = p.inv_freq[8 * j + q];
    uint32_t cur = 0xffffffffu;
    int s = 0;
    uint32_t ph = 0;
    for (;;) {
      if (!mbar_wait(&full[s], ph, abort_flag, limit)) break;
      const StageMeta& mt = meta[s];
      if (mt.layer < 0) break;
      if (mt.tsub != cur) {
        cur = mt.tsub;
        const float posf = (float)(mt.pos0 + t);
#pragma unroll
        for (int q = 0; q < 8; ++q) rope_sincos(posf, f8[q], sn[q], cs[q]);
      }
      if ((mt.valid >> t) & 1u) {
        const uint8_t* ksm = stages + (size_t)s * 2 * kTmaAreaBytes + (size_t)t * row_bytes;
        __nv_bfloat16* kd = p.k_cache + (int64_t)mt.layer * p.layer_stride + mt.dst_off[t];
        for (int u = l; u < n_units; u += tpt) {
          const int h = u >> g_shift;
          uint4 a = *reinterpret_cast<const uint4*>(ksm + (size_t)(h * D + offA) * 2);
          uint4 b = *reinterpret_cast<const uint4*>(ksm + (size_t)(h * D + offB) * 2);
          rotate_unit<STYLE>(a, b, sn, cs);
          __nv_bfloat16* o = kd + (int64_t)h * p.head_stride;
          st_stream(reinterpret_cast<uint4*>(o + offA), a);
          st_stream(reinterpret_cast<uint4*>(o + offB), b);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
      if (++s == kTmaStages) {
        s = 0;
        ph ^= 1u;
      }
    }
  }

  __syncthreads();
  if (*abort_flag) {
    // give copies that may still be in flight time to land before the shared memory is released
    for (int w = 0; w < 4096; ++w) __nanosleep(256);
    if (p.out_status)
      for (int r = threadIdx.x; r < p.nreq; r += blockDim.x) atomicOr(&p.out_status[r], 32 /*MS_REQ_KERNEL_TIMEOUT*/);
  }
}

}  // namespace ms
