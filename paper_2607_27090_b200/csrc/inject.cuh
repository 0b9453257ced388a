// Chunked-RoPE injection kernels: a small plan kernel (ids -> positions -> slots) followed by a
// persistent gather / rotate / scatter kernel.  Paper: Sec. 3.3 (composition), Theorem 2 (chunked RoPE),
// Sec. 5.2 (position policy), Sec. 2.2 and 3.4 (paged blocks, slot mapping).
#pragma once
#include "common.cuh"

namespace ms {

struct InjectParams {
  // store
  const FactRec* facts;
  int32_t n_facts;
  const __nv_bfloat16* k_arena;  // [L][arena_tokens][H][D]
  const __nv_bfloat16* v_arena;
  int64_t arena_tokens;
  const __nv_bfloat16* k_host;  // pinned host arena as seen from the device, [L][host_tokens][H][D], or nullptr
  const __nv_bfloat16* v_host;
  int64_t host_tokens;
  const float* inv_freq;  // [D/2]
  int32_t n_layers, n_heads, head_dim, rope_style;
  int32_t rotary_dim;  // first coordinates of a head that rotate (a multiple of 16, <= head_dim)
  int32_t max_position;
  // request
  const int32_t* fact_ids;  // [nreq][k]
  int32_t nreq, k;
  int32_t prefix_src, prefix_len;  // instruction prefix placed before the facts (arena token, length); length 0 = none
  const int32_t* start_pos;
  const int32_t* block_tables;
  int32_t max_blocks;
  uint32_t flags;
  // cache
  __nv_bfloat16* k_cache;
  __nv_bfloat16* v_cache;
  int64_t layer_stride, block_stride, token_stride, head_stride, num_blocks;
  int32_t block_size;
  float k_scale, v_scale;  // 8-bit cache: per-tensor scales of K and V (the cache holds value / scale)
  float k_recip, v_recip;  // their reciprocals, correctly rounded to fp32 (computed by the host in double)
  // outputs
  int32_t* out_n_tokens;
  int32_t* out_status;
  int64_t* out_slot_mapping;
  int64_t slot_stride;
  // scratch
  TileDesc* tiles;
  uint32_t tiles_capacity;
  InjectCtrl* ctrl;  // control block of the store (see InjectCtrl)
  int32_t layers_per_item;
  // composition cache (nullptr / 0: none)
  CcSlot* cc_slots;
  __nv_bfloat16* cc_k;  // [L][cc_tokens][H][D] rotated keys of the cached segments, slot s at tokens s * cc_slot_tokens ...
  __nv_bfloat16* cc_v;
  int64_t cc_tokens;
  int32_t cc_n_slots, cc_slot_tokens;
  uint32_t cc_epoch, cc_call;  // current epoch of the store; number of this injection call (for the least-recently-used choice)
  int32_t cc_fill_all;         // 0: only requests that name a host-tier fact are recorded; 1: every eligible request
  uint32_t* cc_counters;       // [0] hits, [1] fills
  uint32_t spin_limit;    // 0: the default bound of the staged kernel's waits; else a test's shorter bound
  int32_t mute_producer;  // test aid: the staged kernel's producer role issues nothing
  // memstore_serve_host with MS_SERVE_EARLY_RETURN (one request): a word of pinned host memory, through its device
  // address, that takes host_seq once the request's ids, token count and status - which the kernels write into pinned
  // host memory too - are final; nullptr otherwise
  uint32_t* host_flag;
  uint32_t host_seq;
  int32_t host_flag_in_copy;  // 1: the direct copy kernel raises the flag when it starts (the planning kernel is then spared the
                              // system-wide fence at its end, which the copy kernel would have to wait out); 0: the planning does
};

constexpr int kPlanThreads = 256;      // planning CTA when a call holds more requests than the GPU has SMs
constexpr int kPlanMaxParts = 16;       // CTAs that plan one long request together
constexpr int kPlanThreadsWide = 1024;  // otherwise: the tile descriptors are laid out one token per thread and pass
constexpr int kPlanMaxK = 4096;  // facts per request held in shared memory by the plan kernel

// ------------------------------------------------------------------------------------------------
// Plan kernel: one CTA per request.
//   I1 fact resolution (id -> arena offset, length), I2 exclusive scan of lengths (b_i, m),
//   I3 slot = block_table[pos / bs] * bs + pos % bs, validation, tile descriptors.
// ------------------------------------------------------------------------------------------------
// Shared memory of one planning CTA: s_begin / s_src hold one entry per fact of the request plus one for the
// instruction prefix (the caller sizes them).
constexpr int kPlanTableCache = 2048;  // block-table entries of a request kept in shared memory
struct PlanShared {
  int32_t table[kPlanTableCache];
  int32_t scan[32];  // one partial sum per warp (up to 1024 threads)
  int32_t carry, status;
  uint32_t tile_base;
  uint32_t cc_hash_lo, cc_hash_hi;  // composition cache: hash of the request's key; slot that may hold it; slot to record into
  int32_t cc_cand, cc_victim;
};

// What planning request r needs and what does not depend on the request's ids, fetched ahead of time (all THREADS
// threads call; plan_request<THREADS, true> completes it): the block-table row goes to shared memory with asynchronous
// copies, and the head of the fact table is pulled towards the SM, so that a caller with other work to do first (the
// retrieval kernel selects the ids in the meantime) finds both at hand.
template <int THREADS>
__device__ __forceinline__ void plan_prefetch(const InjectParams& p, const int r, PlanShared& ps) {
  const int tid = threadIdx.x;
  const int32_t* table_row = p.block_tables + (int64_t)r * p.max_blocks;
  const int n_cached = min(p.max_blocks, kPlanTableCache);
  for (int i = tid; i < n_cached; i += THREADS)
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(&ps.table[i])), "l"(table_row + i)
                 : "memory");
  asm volatile("cp.async.commit_group;" ::: "memory");
  const int n_lines = min((p.n_facts * (int)sizeof(FactRec) + 127) / 128, THREADS);
  if (tid < n_lines) asm volatile("prefetch.global.L1 [%0];" ::"l"(reinterpret_cast<const char*>(p.facts) + (size_t)tid * 128));
}

// Plans request r with the THREADS threads of the calling CTA (all of them must call).  PREFETCHED: plan_prefetch has
// been called for this request by the same threads.  PREFILLED: the caller has resolved the facts already - s_begin[j]
// holds the LENGTH and s_src[j] the source token of entry j (placement order, entry 0 left for the prefix when there
// is one), data errors of the lookup are in ps.status, and a block barrier separates those writes from this call.
// parts > 1 (a call of ONE long request without a composition cache): `parts` CTAs plan the request together.  Each
// resolves the facts and scans the lengths itself (cheap), they share the per-token work - every CTA takes every
// parts-th pass of THREADS tokens - and the last one to finish (a ticket in the control block, whose `acc` word gathers
// the status bits meanwhile) writes the token count, the status and the tile count.
template <int THREADS, bool PREFETCHED = false, bool PREFILLED = false>
__device__ __forceinline__ void plan_request(const InjectParams& p, const int r, int32_t* s_begin, int32_t* s_src, PlanShared& ps,
                                             const int32_t* ids_smem = nullptr, const uint32_t part = 0, const uint32_t parts = 1) {
  int32_t* const s_scan = ps.scan;
  int32_t& s_carry = ps.carry;
  int32_t& s_status = ps.status;
  uint32_t& s_tile_base = ps.tile_base;
  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const int32_t start = p.start_pos[r];  // issued first: its latency hides behind the scan
  if (tid == 0) {
    s_carry = 0;
    if (!PREFILLED) s_status = 0;
  }
  // the request's block-table row goes to shared memory in one coalesced sweep: the per-token lookups below would
  // otherwise be a chain of dependent global loads
  const int32_t* table_row = p.block_tables + (int64_t)r * p.max_blocks;
  const int n_cached = min(p.max_blocks, kPlanTableCache);
  if constexpr (PREFETCHED) {
    asm volatile("cp.async.wait_all;" ::: "memory");
  } else {
    for (int i = tid; i < n_cached; i += THREADS) ps.table[i] = table_row[i];
  }
  __syncthreads();

  // lengths of the entries in placement order (the instruction prefix, if any, then the facts), exclusive scan in
  // chunks of THREADS
  // ids_smem: the request's id list in shared memory, when its producer ran in this CTA (the same values as in
  // p.fact_ids; it saves a round trip to global memory)
  const int32_t* ids = ids_smem ? ids_smem : p.fact_ids + (int64_t)r * p.k;
  const int has_prefix = p.prefix_len > 0;
  const int n_entries = p.k + has_prefix;
  // length and source token of entry j of the placement list (nothing for an absent, unknown or non-resident fact)
  auto entry = [&](int j, int32_t& len, int32_t& src) {
    len = 0;
    src = 0;
    if (j < has_prefix) {
      len = p.prefix_len;
      src = p.prefix_src;
    } else if (PREFILLED) {
      if (j < n_entries) {
        len = s_begin[j];
        src = s_src[j];
      }
    } else if (j < n_entries) {
      const int jf = j - has_prefix;
      const int32_t id = ids[(p.flags & 1u) ? (p.k - 1 - jf) : jf];
      if (id >= 0) {
        if (id >= p.n_facts) {
          atomicOr(&s_status, 1 /*MS_REQ_BAD_FACT_ID*/);
        } else {
          const FactRec f = p.facts[id];
          if (!f.resident) {
            atomicOr(&s_status, 2 /*MS_REQ_NOT_RESIDENT*/);
          } else {
            len = f.n_tokens;
            src = f.resident == 2 ? (f.tok_off | kHostTierBit) : f.tok_off;
          }
        }
      }
    }
  };
  int32_t m;
  int names_host_fact = 0;  // some placed fact lives in the host tier (the same value in every thread)
  if (n_entries <= THREADS) {
    // at most one entry per thread: one barrier, then every warp combines the warps' totals by a shuffle scan
    const int j = tid;
    int32_t len, src;
    entry(j, len, src);
    int32_t x = len;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int32_t y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (lane == 31) s_scan[warp] = x;
    __syncwarp();
    __syncthreads();
    int32_t tot = lane < THREADS / 32 ? s_scan[lane] : 0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int32_t y = __shfl_up_sync(0xffffffffu, tot, o);
      if (lane >= o) tot += y;
    }
    const int32_t below = __shfl_sync(0xffffffffu, tot, warp > 0 ? warp - 1 : 0);
    m = __shfl_sync(0xffffffffu, tot, 31);
    if (j < n_entries) {
      s_begin[j] = (warp > 0 ? below : 0) + x - len;
      s_src[j] = src;
    }
    __syncwarp();
    names_host_fact = __syncthreads_or(len > 0 && (src & kHostTierBit) != 0);
  } else {
    // longer lists: chunks of THREADS entries with a running carry
    for (int base = 0; base < n_entries; base += THREADS) {
      const int j = base + tid;
      int32_t len, src;
      entry(j, len, src);
      int32_t x = len;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int32_t y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += y;
      }
      if (lane == 31) s_scan[warp] = x;
      __syncwarp();
      __syncthreads();
      int32_t warp_off = 0;
      for (int w = 0; w < warp; ++w) warp_off += s_scan[w];
      const int32_t carry = s_carry;
      if (j < n_entries) {
        s_begin[j] = carry + warp_off + x - len;
        s_src[j] = src;
      }
      __syncthreads();
      if (tid == THREADS - 1) s_carry = carry + warp_off + x;
      __syncwarp();
      names_host_fact |= __syncthreads_or(len > 0 && (src & kHostTierBit) != 0);
    }
    m = s_carry;
  }
  // A start position that is negative, or at or beyond the position bound, places no token at all: no tile is made
  // (the divisions and the block-table lookups below assume 0 <= pos), the request gets a status bit, and the slot
  // mapping lists every composed token as skipped.
  const bool bad_start = start < 0 || start >= p.max_position;
  if (bad_start && m > 0) {
    if (tid == 0) atomicOr(&s_status, start < 0 ? 64 /*MS_REQ_BAD_START*/ : 16 /*MS_REQ_POSITION_OVERFLOW*/);
    if (p.out_slot_mapping)
      for (int64_t q = (int64_t)part * THREADS + tid; q < min((int64_t)m, p.slot_stride); q += (int64_t)parts * THREADS)
        p.out_slot_mapping[(int64_t)r * p.slot_stride + q] = -1;
  }
  // ---- composition cache: has this very request been composed before, or should it be recorded now? ------------
  int32_t hit_base = -1, fill_base = kNoFill;
  if (p.cc_slots != nullptr && m > 0 && !bad_start && m <= p.cc_slot_tokens && p.k <= kCcMaxK && p.k > 0) {
    const int32_t* key_ids = p.fact_ids + (int64_t)r * p.k;  // the list as the caller (or the retrieval) wrote it
    const int32_t key_flags = (int32_t)(p.flags & 3u);
    if (tid == 0) {
      ps.cc_hash_lo = 0x9e3779b9u * (uint32_t)(p.k + 1) ^ (uint32_t)start * 0x85ebca6bu ^ (uint32_t)key_flags;
      ps.cc_hash_hi = 0xc2b2ae35u * (uint32_t)(p.prefix_src + 3) ^ (uint32_t)p.prefix_len;
      ps.cc_cand = -1;
      ps.cc_victim = -1;
    }
    __syncthreads();
    for (int t = tid; t < p.k; t += THREADS) {
      uint32_t h = (uint32_t)key_ids[t] * 0x9e3779b1u + (uint32_t)t * 0x7feb352du;
      h ^= h >> 15;
      h *= 0x846ca68bu;
      h ^= h >> 16;
      atomicXor(&ps.cc_hash_lo, h);
      atomicAdd(&ps.cc_hash_hi, h * 0x2c1b3c6du + 1u);
    }
    __syncwarp();
    __syncthreads();
    if (warp == 0) {
      // lane l looks at slots l and l + 32: same key fields and hash?  otherwise, how long ago was it used?
      uint32_t best_age = 0xffffffffu;
      int best_slot = -1, match = -1;
      for (int sl = lane; sl < p.cc_n_slots; sl += 32) {
        const CcSlot& c = p.cc_slots[sl];
        const bool live = c.epoch == p.cc_epoch;
        if (live && c.hash_lo == ps.cc_hash_lo && c.hash_hi == ps.cc_hash_hi && c.k == p.k && c.start == start && c.flags == key_flags &&
            c.prefix_src == p.prefix_src && c.prefix_len == p.prefix_len && c.m == m && match < 0)
          match = sl;
        const uint32_t age = live ? c.last_use + 1u : 0u;  // empty slots first, then the least recently used
        if (age < best_age) {
          best_age = age;
          best_slot = sl;
        }
      }
      const unsigned found = __ballot_sync(0xffffffffu, match >= 0);
      if (found) {
        const int src_lane = __ffs(found) - 1;
        const int sl = __shfl_sync(0xffffffffu, match, src_lane);
        if (lane == 0) ps.cc_cand = sl;
      }
      const uint32_t oldest = __reduce_min_sync(0xffffffffu, best_age);
      const unsigned who = __ballot_sync(0xffffffffu, best_age == oldest && best_slot >= 0);
      if (who) {
        const int sl = __shfl_sync(0xffffffffu, best_slot, __ffs(who) - 1);
        if (lane == 0) ps.cc_victim = sl;
      }
    }
    __syncwarp();
    __syncthreads();
    const int cand = ps.cc_cand;
    int same = 0;
    if (cand >= 0) {  // equal hashes: compare the id lists themselves
      bool eq = true;
      for (int t = tid; t < p.k; t += THREADS) eq = eq && p.cc_slots[cand].ids[t] == key_ids[t];
      __syncwarp();
      same = __syncthreads_and(eq);
    }
    if (same) {
      hit_base = cand * p.cc_slot_tokens;
      if (tid == 0) {
        p.cc_slots[cand].last_use = p.cc_call;
        atomicAdd(&p.cc_counters[0], 1u);
      }
    } else if (p.nreq == 1 && s_status == 0 && ps.cc_victim >= 0 && (p.cc_fill_all || names_host_fact)) {
      // record this request (single-request calls only: one planning CTA, so slots are never claimed concurrently)
      const int v = ps.cc_victim;
      fill_base = v * p.cc_slot_tokens;
      CcSlot& c = p.cc_slots[v];
      for (int t = tid; t < p.k; t += THREADS) c.ids[t] = key_ids[t];
      if (tid == 0) {
        c.hash_lo = ps.cc_hash_lo;
        c.hash_hi = ps.cc_hash_hi;
        c.k = p.k;
        c.start = start;
        c.flags = key_flags;
        c.prefix_src = p.prefix_src;
        c.prefix_len = p.prefix_len;
        c.m = m;
        c.epoch = p.cc_epoch;
        c.last_use = p.cc_call;
        atomicAdd(&p.cc_counters[1], 1u);
      }
    }
  }
  const int32_t first_tile_pos = bad_start ? 0 : (start / kTileTokens) * kTileTokens;
  const uint32_t n_tiles = (m > 0 && !bad_start) ? (uint32_t)((start - first_tile_pos + m + kTileTokens - 1) / kTileTokens) : 0u;
  uint32_t tile_base = 0;
  if (p.nreq > 1) {  // (a single request owns the whole tile list: no ticket needed)
    if (tid == 0) s_tile_base = n_tiles ? atomicAdd(&p.ctrl->acc, n_tiles) : 0u;
    __syncthreads();
    tile_base = s_tile_base;
  }

  const int bs = p.block_size;
  const int bs_shift = (bs & (bs - 1)) == 0 ? 31 - __clz(bs) : -1;  // block sizes are powers of two in practice
  for (uint32_t e = part * THREADS + tid; e < n_tiles * kTileTokens; e += parts * THREADS) {
    const uint32_t t = e / kTileTokens, ln = e % kTileTokens;
    const int32_t pos = first_tile_pos + (int32_t)e;
    const int32_t q = pos - start;  // index in the composed segment
    int32_t src_tok = -1;
    int64_t dst = 0, slot = -1;
    if (q >= 0 && q < m) {
      // the fact that owns composed token q is the LAST i with b_i <= q: entries of length zero (skipped,
      // unknown or non-resident ids) share their b_i with the next placed fact, and trailing ones have b_i = m > q
      int lo = 0, hi = n_entries - 1;
      while (lo < hi) {
        int mid = (lo + hi + 1) >> 1;
        if (s_begin[mid] <= q) lo = mid; else hi = mid - 1;
      }
      const int i = lo;
      int32_t st = 0;
      if (pos >= p.max_position) {
        st = 16;  // MS_REQ_POSITION_OVERFLOW
      } else {
        const int32_t bi = bs_shift >= 0 ? pos >> bs_shift : pos / bs;
        const int32_t in_block = bs_shift >= 0 ? (pos & (bs - 1)) : pos - bi * bs;
        if (bi >= p.max_blocks) {
          st = 4;  // MS_REQ_BLOCK_TABLE_SHORT
        } else {
          const int32_t blk = bi < n_cached ? ps.table[bi] : table_row[bi];
          if (blk < 0 || blk >= p.num_blocks) {
            st = 8;  // MS_REQ_BAD_BLOCK_ID
          } else {
            src_tok = hit_base >= 0 ? (kCacheTierBit | (hit_base + q)) : s_src[i] + (q - s_begin[i]);
            dst = (int64_t)blk * p.block_stride + (int64_t)in_block * p.token_stride;
            slot = (int64_t)blk * bs + in_block;
          }
        }
      }
      if (st) atomicOr(&s_status, st);
      if (p.out_slot_mapping && q < p.slot_stride) p.out_slot_mapping[(int64_t)r * p.slot_stride + q] = slot;
    }
    if (tile_base + t < p.tiles_capacity) {
      TileDesc* d = p.tiles + tile_base + t;
      if (ln == 0) {
        const int32_t pos0 = first_tile_pos + (int32_t)(t * kTileTokens);
        d->pos0 = pos0;
        d->fill_tok0 = fill_base == kNoFill ? kNoFill : fill_base + (pos0 - start);
      }
      d->src_tok[ln] = src_tok;
      d->dst_off[ln] = dst;
    }
  }
  __syncwarp();
  __syncthreads();
  if (tid == 0 && parts > 1) {
    // one request planned by several CTAs: the last of them publishes
    if (s_status) atomicOr(&p.ctrl->acc, (uint32_t)s_status);
    __threadfence();  // this CTA's descriptors and status bits are visible before its arrival is
    if (atomicAdd(&p.ctrl->planned, 1u) == parts - 1u) {
      __threadfence();
      const int32_t st_all = (int32_t)atomicExch(&p.ctrl->acc, 0u);
      if (p.out_n_tokens) p.out_n_tokens[r] = m;
      if (p.out_status) p.out_status[r] = st_all;
      if (p.host_flag != nullptr && !p.host_flag_in_copy) {
        __threadfence_system();
        *reinterpret_cast<volatile uint32_t*>(p.host_flag) = p.host_seq;
      }
      p.ctrl->n_tiles = n_tiles;
      p.ctrl->work_next = 0;
      p.ctrl->planned = 0;
    }
  } else if (tid == 0) {
    if (p.out_n_tokens) p.out_n_tokens[r] = m;
    if (p.out_status) p.out_status[r] = s_status;
    if (p.host_flag != nullptr && !p.host_flag_in_copy) {
      // the ids (written before the barriers above, by this CTA or an earlier kernel) and the two words above reach the
      // host before the flag does
      __threadfence_system();
      *reinterpret_cast<volatile uint32_t*>(p.host_flag) = p.host_seq;
    }
    // the last planning CTA of the call hands the control block to the copy kernel and leaves it clean
    if (p.nreq == 1) {
      p.ctrl->n_tiles = n_tiles;
      p.ctrl->work_next = 0;
    } else {
      __threadfence();  // this CTA's claim on `acc` is visible before its arrival is
      if (atomicAdd(&p.ctrl->planned, 1u) == (uint32_t)p.nreq - 1u) {
        __threadfence();
        p.ctrl->n_tiles = atomicExch(&p.ctrl->acc, 0u);
        p.ctrl->work_next = 0;
        p.ctrl->planned = 0;
      }
    }
  }
}

template <int THREADS>
__global__ void __launch_bounds__(THREADS) inject_plan_kernel(const InjectParams p) {
  __shared__ int32_t s_begin[kPlanMaxK];  // b_i: first composed token of placed fact i
  __shared__ int32_t s_src[kPlanMaxK];    // arena token of the fact's first token
  __shared__ PlanShared ps;
  grid_dependency_wait();    // launched as a programmatic dependent (of the previous call's copy kernel, typically)
  grid_launch_dependents();  // the copy kernel may start its prologue now; it waits before reading the plan
  plan_request<THREADS>(p, blockIdx.x, s_begin, s_src, ps, nullptr, blockIdx.y, gridDim.y);
}

// ------------------------------------------------------------------------------------------------
// RoPE angle: pos * inv_freq formed EXACTLY as hi + lo, reduced by 2*pi with a three-constant
// Cody-Waite scheme (each fma step is exact up to the last), then sin/cos of the reduced argument.
// Naive fp32 pos*inv_freq is off by up to 0.5 rad-ulp of a 2^24-sized angle and is not usable.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void rope_sincos(float posf, float inv_freq, float& s, float& c) {
  const float hi = __fmul_rn(posf, inv_freq);
  const float lo = __fmaf_rn(posf, inv_freq, -hi);
  const float n = (hi * 0.15915494309189535f + 12582912.f) - 12582912.f;  // round to nearest integer, |x| < 2^22
  float r = __fmaf_rn(n, -6.28125f, hi);                  // exact
  r = __fmaf_rn(n, -0.0019350051879882812f, r);           // exact
  r = __fmaf_rn(n, -3.019916050561733e-07f, r);           // one rounding
  r += lo;
  if (r > 3.14159274f) r -= 6.28318548f;
  if (r < -3.14159274f) r += 6.28318548f;
  __sincosf(r, &s, &c);
}

__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);  // .x = lo (low half), .y = hi
  return *reinterpret_cast<uint32_t*>(&v);
}

// Rotate one unit = two 16-byte vectors a, b of one head (8 frequencies sn[], cs[]).
//   half-split : a = x[8j .. 8j+7], b = x[D/2+8j ..]; pair i is (a_i, b_i)
//   interleaved: a = x[16j .. 16j+7] = pairs 8j..8j+3, b = x[16j+8 ..] = pairs 8j+4..8j+7
template <int STYLE>
__device__ __forceinline__ void rotate_unit(uint4& a, uint4& b, const float* sn, const float* cs) {
  uint32_t* aw = reinterpret_cast<uint32_t*>(&a);
  uint32_t* bw = reinterpret_cast<uint32_t*>(&b);
  if (STYLE == 0) {
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      float x1l = bf16lo(aw[w]), x1h = bf16hi(aw[w]);
      float x2l = bf16lo(bw[w]), x2h = bf16hi(bw[w]);
      float y1l = x1l * cs[2 * w] - x2l * sn[2 * w];
      float y2l = x2l * cs[2 * w] + x1l * sn[2 * w];
      float y1h = x1h * cs[2 * w + 1] - x2h * sn[2 * w + 1];
      float y2h = x2h * cs[2 * w + 1] + x1h * sn[2 * w + 1];
      aw[w] = pack_bf16(y1l, y1h);
      bw[w] = pack_bf16(y2l, y2h);
    }
  } else {
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      float x1 = bf16lo(aw[w]), x2 = bf16hi(aw[w]);
      aw[w] = pack_bf16(x1 * cs[w] - x2 * sn[w], x2 * cs[w] + x1 * sn[w]);
      float z1 = bf16lo(bw[w]), z2 = bf16hi(bw[w]);
      bw[w] = pack_bf16(z1 * cs[4 + w] - z2 * sn[4 + w], z2 * cs[4 + w] + z1 * sn[4 + w]);
    }
  }
}

// Eight fp32 values -> eight e4m3 bytes (round to nearest even, saturating), lowest address first.
__device__ __forceinline__ uint2 pack_e4m3x8(const float* f) {
  uint32_t w[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(f[4 * h], f[4 * h + 1]), __NV_SATFINITE, __NV_E4M3);
    const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(f[4 * h + 2], f[4 * h + 3]), __NV_SATFINITE, __NV_E4M3);
    w[h] = lo | (hi << 16);
  }
  return make_uint2(w[0], w[1]);
}

// x / s rounded to nearest in fp32, as IEEE division gives it, from the correctly rounded reciprocal r = RN(1 / s) that
// the host supplies: two residual corrections with fused multiply-adds (q <- q + (x - q s) r; the residuals are
// exact).  After the first the quotient is faithful, after the second it is the correctly rounded one (Markstein's
// theorem on division with a correctly rounded reciprocal; it excludes divisors whose significand is all ones, for
// which the host asks for the hardware division instead).  Quotients far outside what an e4m3 cache can hold skip the
// corrections (they saturate or vanish whatever their last bit), which also keeps infinities out of the residuals.
template <bool HW_DIV>
__device__ __forceinline__ float div_by_scale(float x, float s, float r) {
  if (HW_DIV) return __fdiv_rn(x, s);
  const float q0 = __fmul_rn(x, r);
  const float q1 = __fmaf_rn(__fmaf_rn(-q0, s, x), r, q0);
  const float q2 = __fmaf_rn(__fmaf_rn(-q1, s, x), r, q1);
  const float a = fabsf(q0);
  return (a < 1e30f && a > 1e-30f) ? q2 : q0;
}

// Two quotients at once with the packed fp32 instructions of this architecture (mul / fma .f32x2: each half is the
// IEEE operation of the scalar instruction, so the results are those of div_by_scale bit for bit, in half the
// instructions).
__device__ __forceinline__ unsigned long long pack_f32x2(float a, float b) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void div_by_scale_x2(float x0, float x1, float s, float r, float& o0, float& o1) {
  const unsigned long long X = pack_f32x2(x0, x1), NS = pack_f32x2(-s, -s), R = pack_f32x2(r, r);
  unsigned long long Q0, T, Q1, Q2;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(Q0) : "l"(X), "l"(R));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(T) : "l"(Q0), "l"(NS), "l"(X));  // x - q0 s, exactly
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(Q1) : "l"(T), "l"(R), "l"(Q0));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(T) : "l"(Q1), "l"(NS), "l"(X));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(Q2) : "l"(T), "l"(R), "l"(Q1));
  float a0, a1, b0, b1;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(Q0));
  asm("mov.b64 {%0, %1}, %2;" : "=f"(b0), "=f"(b1) : "l"(Q2));
  const float m0 = fabsf(a0), m1 = fabsf(a1);
  o0 = (m0 < 1e30f && m0 > 1e-30f) ? b0 : a0;
  o1 = (m1 < 1e30f && m1 > 1e-30f) ? b1 : a1;
}

// The 8 bf16 values of a 16-byte vector divided by `scale` in fp32: the arithmetic of the serving engines' own 8-bit
// cache write (they divide the bf16 key or value by the per-tensor scale in fp32 and round once to e4m3).
template <bool HW_DIV>
__device__ __forceinline__ void scaled_floats(const uint4& a, float scale, float recip, float* f) {
  const uint32_t* aw = reinterpret_cast<const uint32_t*>(&a);
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    if (HW_DIV) {
      f[2 * w] = div_by_scale<true>(bf16lo(aw[w]), scale, recip);
      f[2 * w + 1] = div_by_scale<true>(bf16hi(aw[w]), scale, recip);
    } else {
      div_by_scale_x2(bf16lo(aw[w]), bf16hi(aw[w]), scale, recip, f[2 * w], f[2 * w + 1]);
    }
  }
}

constexpr int kCopyThreads = 256;
constexpr int kThreadsPerToken = kCopyThreads / kTileTokens;  // 32
constexpr int kUnitsPerThread = 2;
constexpr int kUnitsPerPart = kThreadsPerToken * kUnitsPerThread;  // units of a token row served by one CTA

// ------------------------------------------------------------------------------------------------
// Copy kernel (I4 + I5): ONE CTA per work item = (tile of 8 tokens, layer, row part), no shared memory.
// The grid is the host's estimate of the item count (the real tile count is only known on the device); CTAs
// beyond the real count return at once and a low estimate makes some CTAs take a second item.  The hardware CTA scheduler keeps every SM full and balances SMs that get unequal memory
// service, and with 768 resident threads per SM each holding eight 16-byte loads, about 96 KB per SM are in
// flight: measured on B200 this plain structure sustains the copy rate of the device, and a persistent
// shared-memory ring fed by bulk copies does not (see inject_tma.cuh).
//
// 32 threads serve one token; a thread owns up to two units of the token's row, a unit being (head, frequency
// octet): two 16-byte vectors of K (rotated) and the same two of V (copied).  32 and 64 are multiples of D/16, so
// both units of a thread share the frequency octet: its 8 cos/sin pairs are computed once, while the loads fly.
// ------------------------------------------------------------------------------------------------
//
// Variants: when only the first R < D coordinates rotate, octets j >= R/16 of a head are plain copies (for both pair
// styles their two vectors are the 32 contiguous bytes at element 16 j).  FP8 = true writes an 8-bit e4m3 cache: the
// bf16 key (rotated and rounded exactly as for a bf16 cache) and the bf16 value are divided by the per-tensor scale in
// fp32 and rounded once to e4m3, so the cache is byte for byte what an engine's own cache write would make of the
// bf16 cache contents; a thread then stores two 8-byte vectors per row.
// FP8: 0 = bf16 cache, 1 = 8-bit cache, 2 = 8-bit cache with the hardware division (see div_by_scale)
template <int STYLE, int FP8>
__global__ void __launch_bounds__(kCopyThreads, 3) inject_copy_kernel(const InjectParams p) {
  const int tid = threadIdx.x;
  const int tk = tid >> 5;  // token of the tile
  const int l = tid & 31;
  const int D = p.head_dim;
  const int G = D >> 4, g_shift = 31 - __clz(G);  // frequency octets per head (a power of two, at most 16)
  const int n_units = p.n_heads << g_shift;
  const int j = l & (G - 1);
  const int R = p.rotary_dim;
  const bool rotates = 16 * j < R;
  // element offsets of this thread's two vectors inside a head
  const int offA = (STYLE == 0 && rotates) ? 8 * j : 16 * j;
  const int offB = (STYLE == 0 && rotates) ? R / 2 + 8 * j : 16 * j + 8;
  const int u0 = blockIdx.y * kUnitsPerPart + l;
  if (u0 >= n_units) return;

  grid_dependency_wait();  // tile descriptors come from the plan kernel
  // A kernel launched after this one as a programmatic dependent (the next request's retrieval) may be placed on the
  // SMs once every CTA of this grid has got this far; it waits for this grid's completion before it does anything.
  grid_launch_dependents();

  if (p.host_flag != nullptr && p.host_flag_in_copy && blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) {
    // early return of memstore_serve_host: the planning grid is complete, so the request's ids, token count and status
    // are final; they reach the host before the flag does
    __threadfence_system();
    *reinterpret_cast<volatile uint32_t*>(p.host_flag) = p.host_seq;
  }
  const uint32_t n_tiles = min(p.ctrl->n_tiles, p.tiles_capacity);
  const uint32_t n_items = n_tiles * (uint32_t)p.n_layers;
  // items in (layer, tile) order: CTAs that run together stream neighbouring rows of one layer.  The grid is the
  // host's ESTIMATE of the item count: CTAs beyond the real count leave at once, and if the estimate was low the
  // first CTAs take a second item.
  for (uint32_t item = blockIdx.x; item < n_items; item += gridDim.x) {
    const uint32_t layer = item / n_tiles;
    const uint32_t tile = item - layer * n_tiles;
    const TileDesc* d = p.tiles + tile;
    const int32_t src = d->src_tok[tk];
    if (src < 0) continue;
    const int64_t dst = d->dst_off[tk];
    const int32_t pos = d->pos0 + tk;

    // source rows: the HBM arena, (host tier) the pinned host arena read straight over PCIe, or a segment composed
    // earlier and kept in the composition cache, whose keys are rotated already
    const bool host = (src & kHostTierBit) != 0, cached = (src & kCacheTierBit) != 0;
    const int64_t tier_tokens = cached ? p.cc_tokens : host ? p.host_tokens : p.arena_tokens;
    const int64_t src_row = ((int64_t)layer * tier_tokens + (src & ~(kHostTierBit | kCacheTierBit))) * (int64_t)(p.n_heads * D);
    const __nv_bfloat16* ks = (cached ? p.cc_k : host ? p.k_host : p.k_arena) + src_row;
    const __nv_bfloat16* vs = (cached ? p.cc_v : host ? p.v_host : p.v_arena) + src_row;
    const bool rotate_now = rotates && !cached;
    // a request that is being recorded: the composed rows go to the composition cache as well
    const int32_t fill0 = d->fill_tok0;
    const int64_t dbase = (int64_t)layer * p.layer_stride + dst;
    uint4 ka[kUnitsPerThread], kb[kUnitsPerThread], va[kUnitsPerThread], vb[kUnitsPerThread];
#pragma unroll
    for (int u = 0; u < kUnitsPerThread; ++u) {
      const int unit = u0 + u * kThreadsPerToken;
      if (unit < n_units) {
        const int h = unit >> g_shift;
        ka[u] = ld_stream(reinterpret_cast<const uint4*>(ks + h * D + offA));
        kb[u] = ld_stream(reinterpret_cast<const uint4*>(ks + h * D + offB));
        va[u] = ld_stream(reinterpret_cast<const uint4*>(vs + h * D + offA));
        vb[u] = ld_stream(reinterpret_cast<const uint4*>(vs + h * D + offB));
      }
    }
    // cos/sin of (pos, 8 frequencies), evaluated while the loads are in flight
    float sn[8], cs[8];
    const float posf = (float)pos;
    if (rotate_now) {
#pragma unroll
      for (int i = 0; i < 8; ++i) rope_sincos(posf, __ldg(p.inv_freq + 8 * j + i), sn[i], cs[i]);
    }
#pragma unroll
    for (int u = 0; u < kUnitsPerThread; ++u) {
      const int unit = u0 + u * kThreadsPerToken;
      if (unit < n_units) {
        const int h = unit >> g_shift;
        if (rotate_now) rotate_unit<STYLE>(ka[u], kb[u], sn, cs);
        if (fill0 != kNoFill) {
          const int64_t fill_row = ((int64_t)layer * p.cc_tokens + (fill0 + tk)) * (int64_t)(p.n_heads * D);
          __nv_bfloat16* ck = p.cc_k + fill_row + h * D;
          __nv_bfloat16* cv = p.cc_v + fill_row + h * D;
          st_stream(reinterpret_cast<uint4*>(ck + offA), ka[u]);
          st_stream(reinterpret_cast<uint4*>(ck + offB), kb[u]);
          st_stream(reinterpret_cast<uint4*>(cv + offA), va[u]);
          st_stream(reinterpret_cast<uint4*>(cv + offB), vb[u]);
        }
        if (!FP8) {
          __nv_bfloat16* kd = p.k_cache + dbase + (int64_t)h * p.head_stride;
          st_stream(reinterpret_cast<uint4*>(kd + offA), ka[u]);
          st_stream(reinterpret_cast<uint4*>(kd + offB), kb[u]);
          __nv_bfloat16* vd = p.v_cache + dbase + (int64_t)h * p.head_stride;
          st_stream(reinterpret_cast<uint4*>(vd + offA), va[u]);
          st_stream(reinterpret_cast<uint4*>(vd + offB), vb[u]);
        } else {
          float fa[8], fb[8];
          scaled_floats<FP8 == 2>(ka[u], p.k_scale, p.k_recip, fa);
          scaled_floats<FP8 == 2>(kb[u], p.k_scale, p.k_recip, fb);
          uint8_t* kd = reinterpret_cast<uint8_t*>(p.k_cache) + dbase + (int64_t)h * p.head_stride;
          st_stream8(reinterpret_cast<uint2*>(kd + offA), pack_e4m3x8(fa));
          st_stream8(reinterpret_cast<uint2*>(kd + offB), pack_e4m3x8(fb));
          scaled_floats<FP8 == 2>(va[u], p.v_scale, p.v_recip, fa);
          scaled_floats<FP8 == 2>(vb[u], p.v_scale, p.v_recip, fb);
          uint8_t* vd = reinterpret_cast<uint8_t*>(p.v_cache) + dbase + (int64_t)h * p.head_stride;
          st_stream8(reinterpret_cast<uint2*>(vd + offA), pack_e4m3x8(fa));
          st_stream8(reinterpret_cast<uint2*>(vd + offB), pack_e4m3x8(fb));
        }
      }
    }
  }
}

}  // namespace ms
