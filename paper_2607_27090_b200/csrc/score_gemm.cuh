// Batched scoring on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), sm_100a only.  Step R2 for many
// queries that search ONE segment (Sec. 3.2: inner-product search; here 64 queries x 1M facts is a dense
// [facts x E] x [E x queries] contraction, the one place on the path that is GEMM-shaped).
//
// The kernel does not write the score matrix.  It is a FILTER: for every group of 8 consecutive embedding rows
// and every query it writes the largest score of the group (fp32), 1/8 of a score matrix.  A later step picks the
// best groups per query and rescores their rows with the exact CUDA-core routine, so tensor-core rounding never
// decides a rank; it only has to keep every top-k row inside a selected group.
//
// With candidate emission on (GemmParams::hist) the kernel ALSO hands the later steps a short list of candidate ROWS per
// query, so that they need not sweep the group maxima nor rescore whole groups.  Every row whose score reaches the
// query's current THRESHOLD is appended to the query's list (row, filter score).  A threshold is valid when at least k2
// rows of the segment score at or above it (then no row below it is among the k2 best), and thresholds only rise:
//  - the first two tiles of every CTA are computed before any threshold exists; their accumulators stay PARKED in tensor
//    memory, and every epilogue warp only writes the best score of its 32 rows per query to a global table;
//  - when all CTAs have done so (the table is filled with a pattern that is no score between calls, so an entry is its
//    own arrival flag; every CTA is resident, one per SM), the seventh warp of CTA q CALIBRATES query q: the exact
//    k2-th largest of the table's values (a search on the order-preserving keys, two bits at a time, in registers) is the
//    first threshold, and the span from it to the largest value fixes 256 LINEAR buckets for the
//    query's histogram - linear in the score and as wide as the query's own top region, so that the resolution does
//    not depend on the magnitude of the scores (buckets over the bits of the floats resolve 6 %: useless when all the
//    best scores lie within 1 % of one another);
//  - from then on a warp that lists rows for a query also counts the best of them in the query's histogram
//    (fire-and-forget atomics: one per level), and the seventh warp of every CTA keeps reading the histograms (two loads
//    of one line per query) and raises the CTA's 64 thresholds in shared memory to the lower edge of the bucket at which
//    the count from the top reaches k2.  A stale threshold only lets more rows through.
// The epilogue warps never wait for global memory: a warp appends to its OWN segment of every query's list
// ([query][CTA][warp][cand_seg] places, counted in registers) and publishes its counts when it ends.  The parked tiles'
// rows are compared with the thresholds later, in time the epilogue would otherwise spend waiting.  The list's consumer
// checks the counts (at least k2 rows in all, no segment overrun) and falls back to the group maxima otherwise.  Every
// wait (for the arrivals, for the calibrations) is bounded; when one runs out nothing is listed and the fallback serves.
//
// Tiling: facts on M (128 rows per tile = the 128 TMEM lanes), queries on N (64), K = E in chunks of 64 fp16
// (one 128-byte swizzle row).  All queries stay in shared memory for the kernel's lifetime (E/64 chunks of 8 KiB);
// embedding tiles stream through a ring of 16 KiB TMA boxes that takes the rest of the shared memory (6 stages at
// E = 1024).  Four working accumulators of 64 columns live in tensor memory (plus the parked ones), so that the MMAs -
// and with them the loads, which a stalled MMA lane stalls - can run several tiles ahead of the epilogue.
//   warp 0     TMA producer (one elected lane)
//   warp 1     TMEM allocation, tcgen05.mma issue (one elected lane), tcgen05.commit -> mbarriers
//   warps 2-5  epilogue: tcgen05.ld of the warp's 32 TMEM lanes, row mask, 8-row max by shuffles, 16-byte stores
//   warp 6     thresholds of the candidate emission (idle without it)
// Every mbarrier wait is bounded; a time-out sets *error_flag, the roles stop, TMEM is released and the CTA leaves.
#pragma once
#include <cuda.h>

#include "inject_tma.cuh"  // mbarrier helpers

namespace ms {

constexpr int kGemmTileRows = 128;
constexpr int kGemmKChunk = 64;       // fp16 elements per swizzle row (128 bytes)
constexpr int kGemmMaxStages = 8;   // the ring holds as many 16 KiB tiles as fit beside the queries, at most this many
constexpr size_t kGemmSmemBytes = 232448;  // all the dynamic shared memory a CTA can have: always requested
constexpr int kGemmMaxQ = 64;
constexpr int kGemmGroupRows = 8;
constexpr int kGemmGroupsPerTile = kGemmTileRows / kGemmGroupRows;  // 16
constexpr int kGemmThreads = 224;
constexpr int kGemmTmemCols = 512;    // all of an SM's tensor memory (one CTA per SM, and an allocation is a power of two)
constexpr int kGemmAccBufs = 4;       // working accumulators of 64 columns: the MMAs may run this many tiles ahead of the epilogue
constexpr int kGemmParked = 2;        // first tiles of a CTA whose accumulators stay in tensor memory (candidate emission only)
constexpr int kHistFine = 256;        // linear buckets over the query's calibrated span
constexpr int kHistCoarse = 16;       // 16 fine buckets each
constexpr int kHistWords = kHistCoarse + kHistFine;  // one query's counters: [coarse][fine]
constexpr int kCalibWords = 4;        // one query's calibration: {lowest score, buckets per unit, ready, -}, 16 bytes that a reader loads at once
constexpr int kRawPerLane = 40;       // parked-tile maxima per query <= 32 * this (2 tiles x 4 warps x CTAs)
constexpr uint32_t kRawEmpty = 0xffffffffu;  // (a NaN pattern: never a score)
constexpr int kGemmABytes = kGemmTileRows * kGemmKChunk * 2;  // 16 KiB
constexpr int kGemmQBytes = kGemmMaxQ * kGemmKChunk * 2;      // 8 KiB per chunk
constexpr int kGemmMaxE = 1024;

struct GemmParams {
  int n_rows;   // rows of the segment
  int emb_dim;  // multiple of 64, at most kGemmMaxE
  int nq;       // queries of this batch, at most kGemmMaxQ
  float* gmax;  // [nq][gmax_stride]: entry [q][g] = max over rows 8g..8g+7 of the score of query q
  int64_t gmax_stride;  // multiple of 16, >= 16 * ceil(n_rows / 128)
  int* error_flag;
  uint32_t smem_bytes;  // dynamic shared memory of the launch
  uint32_t spin_limit;  // 0: the default bound of every wait; else a test's shorter bound
  int mute_producer;    // test aid: the producer role issues nothing, so the other roles' waits run out
  const uint32_t* removed_bits;  // one bit per row of the segment, or nullptr: removed rows take no part in a group's maximum
  // candidate emission (hist == nullptr: off).  All counters are zero when the kernel starts.
  uint32_t* hist;         // [kGemmMaxQ][kHistWords]
  uint32_t* calib;        // [kGemmMaxQ][kCalibWords], zero when the kernel starts (kept apart from the counters: every CTA polls it)
  float* raw;             // [kGemmMaxQ][32 * kRawPerLane]: the best score of every epilogue warp's rows in its parked tiles;
                          // every word is kRawEmpty when the kernel starts
  uint32_t* cand_cnt;     // [kGemmMaxQ][gridDim.x * 4]: rows the warp found for the query (beyond cand_seg: the surplus was dropped)
  uint32_t* thr_used;     // [kGemmMaxQ]: order key of the highest threshold any CTA applied (0: none)
  unsigned long long* cand;  // [kGemmMaxQ][gridDim.x * 4][cand_seg]: (order key of the filter score << 32) | row
  int cand_seg;
  int k2;                 // group maxima the threshold keeps at or above it
};

__device__ __forceinline__ uint32_t gemm_order_key(float s) {
  const uint32_t u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float gemm_key_value(uint32_t kx) {
  return __uint_as_float((kx & 0x80000000u) ? (kx & 0x7fffffffu) : ~kx);
}

// The bucket of a score in a query's calibrated histogram.
__device__ __forceinline__ int hist_bucket(float x, float lo, float per_unit) {
  const float b = (x - lo) * per_unit;
  return b >= (float)(kHistFine - 1) ? kHistFine - 1 : b > 0.f ? (int)b : 0;
}

// The threshold of a query from its histogram: the lower edge (a quarter of a bucket further down, so that float rounding
// at an edge cannot matter) of the bucket at which the count from the top reaches `need`; `lo` while it does not.
// Two queries at once: the loads of both are issued together.
__device__ __forceinline__ void hist_thresholds2(const uint32_t* ha, const uint32_t* hb, uint32_t need, float lo_a, float pu_a, float lo_b,
                                                 float pu_b, float& ta, float& tb) {
  auto scan16 = [&](const uint4 (&c)[4], uint32_t& cum, int& at) {
    at = -1;
    auto one = [&](uint32_t x, int idx) {
      if (at < 0) {
        if (cum + x >= need) at = idx;
        else cum += x;
      }
    };
#pragma unroll
    for (int i = 3; i >= 0; --i) {
      one(c[i].w, 4 * i + 3);
      one(c[i].z, 4 * i + 2);
      one(c[i].y, 4 * i + 1);
      one(c[i].x, 4 * i);
    }
  };
  uint4 ca[4], cb[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    ca[i] = __ldcg(reinterpret_cast<const uint4*>(ha) + i);
    cb[i] = __ldcg(reinterpret_cast<const uint4*>(hb) + i);
  }
  uint32_t cum_a = 0, cum_b = 0;
  int at_a, at_b, fa, fb;
  scan16(ca, cum_a, at_a);
  scan16(cb, cum_b, at_b);
  const int a0 = at_a < 0 ? 0 : at_a, b0 = at_b < 0 ? 0 : at_b;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    ca[i] = __ldcg(reinterpret_cast<const uint4*>(ha + kHistCoarse + a0 * 16) + i);
    cb[i] = __ldcg(reinterpret_cast<const uint4*>(hb + kHistCoarse + b0 * 16) + i);
  }
  scan16(ca, cum_a, fa);  // (a coarse counter may run ahead of its fine ones for a moment: then the coarse bucket's edge)
  scan16(cb, cum_b, fb);
  const float ea = (float)(a0 * 16 + (fa < 0 ? 0 : fa)) - 0.25f, eb = (float)(b0 * 16 + (fb < 0 ? 0 : fb)) - 0.25f;
  ta = (at_a < 0 || !(pu_a > 0.f)) ? lo_a : fmaxf(lo_a, lo_a + ea / pu_a);
  tb = (at_b < 0 || !(pu_b > 0.f)) ? lo_b : fmaxf(lo_b, lo_b + eb / pu_b);
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t* p, uint32_t v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Shared memory after the 1 KiB alignment of the base: queries, ring, epilogue staging (4 warps x [4 groups][32
// queries] floats), barriers.
constexpr uint32_t kGemmStagingBytes = 4 * 4 * 32 * sizeof(float);
constexpr uint32_t kGemmBarrierBytes = 512;  // barriers and flags (< 256 bytes), 64 thresholds
__host__ __device__ constexpr int gemm_stages(uint32_t usable_bytes, int emb_dim) {
  const int64_t left = (int64_t)usable_bytes - (int64_t)(emb_dim / kGemmKChunk) * kGemmQBytes - kGemmStagingBytes - kGemmBarrierBytes;
  const int64_t n = left / kGemmABytes;
  return n > kGemmMaxStages ? kGemmMaxStages : (int)n;
}

__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(smem_dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, 128-byte swizzled, 8-row atoms 1 KiB apart.
__device__ __forceinline__ uint64_t umma_desc_k_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);  // start address, bits [0,14)
  d |= (uint64_t)1 << 16;                        // leading byte offset (unused for swizzled K-major), bits [16,30)
  d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset between 8-row atoms, bits [32,46)
  d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                        // 128-byte swizzle
  return d;
}

// Instruction descriptor: D = fp32, A = B = fp16, both K-major, M = 128, N = 64.
constexpr uint32_t kGemmIdesc = (1u << 4) | ((uint32_t)(kGemmMaxQ >> 3) << 17) | ((uint32_t)(kGemmTileRows >> 4) << 24);

__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t"
      ".reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t"
      "}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* r) {
  uint32_t* u = reinterpret_cast<uint32_t*>(r);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, "
      "%18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]), "=r"(u[9]),
        "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), "=r"(u[16]), "=r"(u[17]), "=r"(u[18]),
        "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]), "=r"(u[25]), "=r"(u[26]), "=r"(u[27]),
        "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// One column of the warp's 32 tensor-memory lanes; the value is there after tmem_ld_wait().
__device__ __forceinline__ uint32_t tmem_ld1_issue(uint32_t taddr) {
  uint32_t u;
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(u) : "r"(taddr) : "memory");
  return u;
}
__device__ __forceinline__ float4 lds_volatile_f4(const volatile float* p) {
  float4 r;
  asm volatile("ld.volatile.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "r"(smem_u32(const_cast<const float*>(p))));
  return r;
}

__global__ void __launch_bounds__(kGemmThreads, 1)
    score_gemm_groupmax_kernel(const __grid_constant__ CUtensorMap tmap_emb, const __grid_constant__ CUtensorMap tmap_q,
                               const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int nkc = p.emb_dim / kGemmKChunk;
  uint8_t* q_smem = smem;                                   // nkc chunks of [64 queries][128 B]
  // the ring takes what the alignment of the base and the queries leave: 6 tiles for 1024-d embeddings, 8 below
  const int n_stages = gemm_stages(p.smem_bytes - (uint32_t)(smem - smem_raw), p.emb_dim);
  uint8_t* a_smem = q_smem + (size_t)nkc * kGemmQBytes;     // n_stages tiles of [128 rows][128 B]
  float* stage_f = reinterpret_cast<float*>(a_smem + (size_t)n_stages * kGemmABytes);  // [4 warps][4 groups][32 q]
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(stage_f) + kGemmStagingBytes);
  uint64_t* q_full = bars;
  uint64_t* full = bars + 1;
  uint64_t* empty = full + kGemmMaxStages;
  uint64_t* acc_full = empty + kGemmMaxStages;
  uint64_t* acc_empty = acc_full + kGemmAccBufs + kGemmParked;  // acc_full[kGemmAccBufs + j]: parked tile j
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + kGemmAccBufs);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* thr_ready = abort_flag + 1;  // every query of the batch has a threshold
  volatile int* epi_done = abort_flag + 2;   // epilogue warps that have finished
  volatile float* s_thr = reinterpret_cast<volatile float*>(reinterpret_cast<uint8_t*>(bars) + 256);  // [64]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (n_stages < 2) {  // cannot happen with the launch this library makes; nothing has been set up yet
    if (threadIdx.x == 0) atomicExch(p.error_flag, 1);
    return;
  }
  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int b = 0; b < kGemmAccBufs; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], 4);
    }
    for (int j = 0; j < kGemmParked; ++j) mbar_init(&acc_full[kGemmAccBufs + j], 1);
    *abort_flag = 0;
    *thr_ready = 0;
    *epi_done = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (threadIdx.x < kGemmMaxQ) s_thr[threadIdx.x] = -INFINITY;
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kGemmTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int n_tiles = (p.n_rows + kGemmTileRows - 1) / kGemmTileRows;
  const uint32_t limit = p.spin_limit ? p.spin_limit : kSpinLimit;
  const bool emitting = p.hist != nullptr;
  const int n_parked = emitting ? kGemmParked : 0;
  grid_dependency_wait();    // launched as a programmatic dependent itself: the set-up above overlaps the end of the preceding kernel
  grid_launch_dependents();  // the kernels that follow are programmatic dependents: they are placed as SMs free up and wait for this grid

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && !p.mute_producer) {
      mbar_arrive_expect_tx(q_full, (uint32_t)nkc * kGemmQBytes);
      for (int kc = 0; kc < nkc; ++kc) tma_load_2d(q_smem + (size_t)kc * kGemmQBytes, &tmap_q, kc * kGemmKChunk, 0, q_full);
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x) {
        for (int kc = 0; kc < nkc; ++kc) {
          ok = mbar_wait(&empty[s], ph ^ 1u, abort_flag, limit);
          if (!ok) break;
          mbar_arrive_expect_tx(&full[s], kGemmABytes);
          tma_load_2d(a_smem + (size_t)s * kGemmABytes, &tmap_emb, kc * kGemmKChunk, tile * kGemmTileRows, &full[s]);
          if (++s == n_stages) {
            s = 0;
            ph ^= 1u;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = mbar_wait(q_full, 0, abort_flag, limit);
      int s = 0;
      uint32_t ph = 0;
      int it = 0;
      for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x, ++it) {
        // with emission on, the CTA's first tiles go to the parked columns (nobody reuses them); the others take the
        // working buffers in turn
        const bool parked = it < n_parked;
        const int wi = it - n_parked;
        const int b = parked ? kGemmAccBufs + it : wi % kGemmAccBufs;
        if (!parked) {
          ok = mbar_wait(&acc_empty[b], (uint32_t)((wi / kGemmAccBufs) & 1) ^ 1u, abort_flag, limit);
          if (!ok) break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(b * kGemmMaxQ);
        for (int kc = 0; kc < nkc; ++kc) {
          ok = mbar_wait(&full[s], ph, abort_flag, limit);
          if (!ok) break;
          tc_fence_after();
          const uint64_t a_desc = umma_desc_k_sw128(smem_u32(a_smem + (size_t)s * kGemmABytes));
          const uint64_t b_desc = umma_desc_k_sw128(smem_u32(q_smem + (size_t)kc * kGemmQBytes));
#pragma unroll
          for (int k4 = 0; k4 < kGemmKChunk / 16; ++k4)  // 16 fp16 = 32 bytes per MMA along K: +2 in the address field
            umma_f16(d_tmem, a_desc + (uint64_t)(2 * k4), b_desc + (uint64_t)(2 * k4), kGemmIdesc, (kc | k4) != 0 ? 1u : 0u);
          umma_commit(&empty[s]);  // the stage is free once these MMAs have read it
          if (++s == n_stages) {
            s = 0;
            ph ^= 1u;
          }
        }
        if (ok) umma_commit(&acc_full[b]);  // accumulator complete
      }
    }
    __syncwarp();
  } else if (warp == 6) {
    // ------------------------------------------------------------------ thresholds (candidate emission only)
    if (emitting) {
      constexpr unsigned kFull = 0xffffffffu;
      const int n_raw = (int)(gridDim.x * 4u * (uint32_t)kGemmParked);  // values per query in the table: epilogue warps x parked tiles
      // (a) the warp of CTA q calibrates query q once the parked tiles of all CTAs are in the table
      if ((int)blockIdx.x < p.nq) {
        const int q = blockIdx.x;
        float lo = INFINITY, per_unit = 0.f;  // (nothing reaches +infinity: no row is listed and the group maxima serve the query)
        bool ok = false;
        uint32_t key[kRawPerLane];
        if (n_raw <= 32 * kRawPerLane && n_raw >= p.k2) {
          const uint32_t* rq = reinterpret_cast<const uint32_t*>(p.raw) + (size_t)q * (32 * kRawPerLane);
          for (uint32_t w = 0; w < limit && !*abort_flag && !ok; ++w) {  // until every entry has been written
            bool full = true;
#pragma unroll
            for (int j = 0; j < kRawPerLane; ++j) {
              const int i = j * 32 + lane;
              const uint32_t bits = i < n_raw ? __ldcg(rq + i) : 0u;
              full = full && bits != kRawEmpty;
              key[j] = i < n_raw ? gemm_order_key(__uint_as_float(bits)) : 0u;
            }
            ok = __all_sync(kFull, full);
            if (!ok) __nanosleep(256);
          }
        }
        if (ok) {
          // the k2-th largest key, two bits at a time: the largest value that at least k2 keys reach
          uint32_t kth = 0u, top = 0u;
          for (int bit = 30; bit >= 0; bit -= 2) {
            const uint32_t c1 = kth | (1u << bit), c2 = kth | (2u << bit), c3 = kth | (3u << bit);
            int n1 = 0, n2 = 0, n3 = 0;
#pragma unroll
            for (int j = 0; j < kRawPerLane; ++j) {
              n1 += key[j] >= c1;
              n2 += key[j] >= c2;
              n3 += key[j] >= c3;
            }
            n1 = __reduce_add_sync(kFull, n1);
            n2 = __reduce_add_sync(kFull, n2);
            n3 = __reduce_add_sync(kFull, n3);
            kth = n3 >= p.k2 ? c3 : n2 >= p.k2 ? c2 : n1 >= p.k2 ? c1 : kth;
          }
#pragma unroll
          for (int j = 0; j < kRawPerLane; ++j) top = max(top, key[j]);
          top = __reduce_max_sync(kFull, top);
          const float t0 = gemm_key_value(kth), hi = gemm_key_value(top);
          if (t0 > -INFINITY && hi < INFINITY) {
            lo = t0;
            const float span = 2.f * (hi - t0);  // room above the best score seen so far; scores beyond it share the last bucket
            per_unit = span > 1e-30f ? (float)kHistFine / span : 0.f;
            // (The table's own values are not counted in the histogram: until k2 later maxima have reached the threshold
            // it stays where it is, and afterwards it is read from those alone - lower than with the table's values
            // counted too, never invalid.  Counting them costs atomics on a few addresses right when every warp of the
            // GPU waits for this calibration: same-address atomics take 50 - 100 ns each while the embeddings stream.)
          }
        }
        __syncwarp();
        if (lane == 0) {
          uint32_t* cq = p.calib + (size_t)q * kCalibWords;
          cq[0] = __float_as_uint(lo);
          cq[1] = __float_as_uint(per_unit);
          __threadfence();  // the two words above before the flag
          st_release_u32(cq + 2, 1u);
        }
      }
      // (b) the calibration of every query: lane l looks after queries l and l + 32
      const int qa = lane < p.nq ? lane : 0, qb = lane + 32 < p.nq ? lane + 32 : 0;
      const uint32_t* ha = p.hist + (size_t)qa * kHistWords;
      const uint32_t* hb = p.hist + (size_t)qb * kHistWords;
      // (one 16-byte load per query and poll, every half microsecond: 148 CTAs poll the same 64 entries)
      bool have = false;
      uint4 ca = make_uint4(0u, 0u, 0u, 0u), cb = ca;
      for (uint32_t w = 0; w < limit && !*abort_flag && *epi_done < 4; ++w) {
        ca = __ldcg(reinterpret_cast<const uint4*>(p.calib + (size_t)qa * kCalibWords));
        cb = __ldcg(reinterpret_cast<const uint4*>(p.calib + (size_t)qb * kCalibWords));
        have = ca.z != 0u && cb.z != 0u;
        if (__all_sync(kFull, have)) break;
        __nanosleep(512);
      }
      have = __all_sync(kFull, have);
      __threadfence();
      float lo_a = INFINITY, pu_a = 0.f, lo_b = INFINITY, pu_b = 0.f;
      if (have) {
        lo_a = __uint_as_float(ca.x);
        pu_a = __uint_as_float(ca.y);
        lo_b = __uint_as_float(cb.x);
        pu_b = __uint_as_float(cb.y);
      }
      float mine_a = lo_a, mine_b = lo_b;
      if (lane < p.nq) {
        s_thr[lane] = mine_a;
        if (mine_a < INFINITY) atomicMax(p.thr_used + lane, gemm_order_key(mine_a));
      }
      if (lane + 32 < p.nq) {
        s_thr[lane + 32] = mine_b;
        if (mine_b < INFINITY) atomicMax(p.thr_used + lane + 32, gemm_order_key(mine_b));
      }
      __syncwarp();
      __threadfence_block();
      if (lane == 0) *thr_ready = 1;
      // (c) the histograms, over and over: two loads of a line per query and round.  The thresholds settle within the first
      // few tiles: read quickly at first, then every 16 us or so; asleep in short naps so that the end of the CTA is
      // noticed at once.  Ends when the four epilogue warps have, or after a bounded number of rounds.
      for (uint32_t round = 0; have && round < limit && *epi_done < 4 && !*abort_flag; ++round) {
        float ta, tb;
        hist_thresholds2(ha, hb, (uint32_t)p.k2, lo_a, pu_a, lo_b, pu_b, ta, tb);
        if (lane < p.nq && ta > mine_a && ta < INFINITY) {
          mine_a = ta;
          s_thr[lane] = ta;
          atomicMax(p.thr_used + lane, gemm_order_key(ta));
        }
        if (lane + 32 < p.nq && tb > mine_b && tb < INFINITY) {
          mine_b = tb;
          s_thr[lane + 32] = tb;
          atomicMax(p.thr_used + lane + 32, gemm_order_key(tb));
        }
        const int naps = round < 6 ? 1 << round : 64;
        for (int w = 0; w < naps && *epi_done < 4 && !*abort_flag; ++w) __nanosleep(256);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    constexpr unsigned kFull = 0xffffffffu;
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, 32*quarter + 32) belong to this warp
    float* my_stage = stage_f + (size_t)(warp - 2) * 4 * 32;
    const uint32_t lane_taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    // Which of the thread's 64 scores (its row against every query) reach the query's threshold: one bit per query.
    // Kept short (the rest of the work is done only for the few queries with a bit set in some lane of the warp).
    auto passes = [&](const float (&v)[kGemmMaxQ], bool out, uint32_t& m_lo, uint32_t& m_hi) {
      m_lo = m_hi = 0u;
#pragma unroll
      for (int q4 = 0; q4 < kGemmMaxQ / 4; ++q4) {
        const float4 t = lds_volatile_f4(s_thr + 4 * q4);
        const uint32_t bits = (v[4 * q4] >= t.x ? 1u : 0u) | (v[4 * q4 + 1] >= t.y ? 2u : 0u) | (v[4 * q4 + 2] >= t.z ? 4u : 0u) |
                              (v[4 * q4 + 3] >= t.w ? 8u : 0u);
        if (q4 < 8) m_lo |= bits << (4 * (q4 & 7));
        else m_hi |= bits << (4 * (q4 & 7));
      }
      if (out) m_lo = m_hi = 0u;
      if (p.nq < 32) {
        m_lo &= (1u << p.nq) - 1u;
        m_hi = 0u;
      } else if (p.nq < 64) {
        m_hi &= (1u << (p.nq - 32)) - 1u;
      }
    };
    // For every query with a bit set somewhere in the warp (two of them at a time, so that their chains of dependent
    // instructions overlap): the score is read again from tensor memory (a dynamic column; the 64 values in registers can
    // only be indexed at compile time).  Rows whose bit is set join the query's candidate list, in this warp's own
    // segment of it (lane l counts the rows found for queries l and l + 32).  publish: the best of the warp's rows for
    // the query is counted in the histogram (it reaches the threshold; lower values could not raise it): one lane per
    // level, both queries in one instruction.
    uint32_t cnt_lo = 0u, cnt_hi = 0u;
    float cal_lo_lo = INFINITY, cal_pu_lo = 0.f, cal_lo_hi = INFINITY, cal_pu_hi = 0.f;  // lane l: the calibrations of queries l and l + 32
    const size_t my_seg = (size_t)blockIdx.x * 4 + (size_t)(warp - 2);
    const size_t n_seg = (size_t)gridDim.x * 4;
    auto serve = [&](uint32_t taddr, int row, uint32_t m_lo, uint32_t m_hi, bool publish) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint32_t m = h ? m_hi : m_lo;
        uint32_t& cnt = h ? cnt_hi : cnt_lo;
        uint32_t any = __reduce_or_sync(kFull, m);
        while (any) {
          const int qa = __ffs(any) - 1;
          any &= any - 1u;
          const bool two = any != 0u;
          const int qb = two ? __ffs(any) - 1 : qa;
          if (two) any &= any - 1u;
          const uint32_t ua = tmem_ld1_issue(taddr + (uint32_t)(qa + 32 * h)), ub = tmem_ld1_issue(taddr + (uint32_t)(qb + 32 * h));
          tmem_ld_wait();
          const uint32_t ka = gemm_order_key(__uint_as_float(ua)), kb = gemm_order_key(__uint_as_float(ub));
          const bool pa = (m >> qa) & 1u, pb = two && ((m >> qb) & 1u);  // (no bit is set for a row that is masked out)
          const unsigned va = __ballot_sync(kFull, pa), vb = __ballot_sync(kFull, pb);
          const uint32_t base_a = __shfl_sync(kFull, cnt, qa), base_b = __shfl_sync(kFull, cnt, qb);
          if (lane == qa) cnt += (uint32_t)__popc(va);
          if (two && lane == qb) cnt += (uint32_t)__popc(vb);
          const unsigned below = (1u << lane) - 1u;
          const uint32_t slot_a = base_a + (uint32_t)__popc(va & below), slot_b = base_b + (uint32_t)__popc(vb & below);
          if (pa && slot_a < (uint32_t)p.cand_seg)
            p.cand[((size_t)(qa + 32 * h) * n_seg + my_seg) * p.cand_seg + slot_a] = ((unsigned long long)ka << 32) | (uint32_t)row;
          if (pb && slot_b < (uint32_t)p.cand_seg)
            p.cand[((size_t)(qb + 32 * h) * n_seg + my_seg) * p.cand_seg + slot_b] = ((unsigned long long)kb << 32) | (uint32_t)row;
          if (publish) {
            const uint32_t best_a = __reduce_max_sync(kFull, pa ? ka : 0u), best_b = __reduce_max_sync(kFull, pb ? kb : 0u);
            const float lo_a = __shfl_sync(kFull, h ? cal_lo_hi : cal_lo_lo, qa), pu_a = __shfl_sync(kFull, h ? cal_pu_hi : cal_pu_lo, qa);
            const float lo_b = __shfl_sync(kFull, h ? cal_lo_hi : cal_lo_lo, qb), pu_b = __shfl_sync(kFull, h ? cal_pu_hi : cal_pu_lo, qb);
            if (lane < (two ? 4 : 2)) {  // lanes 0, 1: the two levels of query a; lanes 2, 3: of query b
              const bool second = lane >= 2;
              const float lo = second ? lo_b : lo_a;
              if (lo < INFINITY) {
                const int b = hist_bucket(gemm_key_value(second ? best_b : best_a), lo, second ? pu_b : pu_a);
                uint32_t* hq = p.hist + (size_t)((second ? qb : qa) + 32 * h) * kHistWords;
                atomicAdd((lane & 1) ? hq + (b >> 4) : hq + kHistCoarse + b, 1u);
              }
            }
          }
        }
      }
      __syncwarp();
    };
    auto row_of = [&](int tile, bool& out) {
      const int row = tile * kGemmTileRows + quarter * 32 + lane;
      out = row >= p.n_rows;
      if (!out && p.removed_bits != nullptr) out = (__ldg(p.removed_bits + (row >> 5)) >> (row & 31)) & 1u;
      return row;
    };
    // The rows of parked tile j (the CTA's j-th tile) against the thresholds as they stand now.
    auto emit_parked = [&](int j) {
      tc_fence_after();
      float v[kGemmMaxQ];
      const uint32_t taddr = lane_taddr + (uint32_t)((kGemmAccBufs + j) * kGemmMaxQ);
      tmem_ld32(taddr, v);
      tmem_ld32(taddr + 32, v + 32);
      tmem_ld_wait();
      bool out;
      const int row = row_of((int)blockIdx.x + j * (int)gridDim.x, out);
      uint32_t m_lo, m_hi;
      passes(v, out, m_lo, m_hi);
      serve(taddr, row, m_lo, m_hi, false);
      tc_fence_before();
    };
    // Before the first rows are compared with thresholds: give the threshold warp a moment to see the first tiles of
    // the other CTAs (bounded; without thresholds every row would be listed).  The MMAs go on meanwhile.
    auto await_thresholds = [&]() {
      for (int w = 0; w < 1024 && !*thr_ready && !*abort_flag; ++w) __nanosleep(128);
      if (*thr_ready) {  // the calibrations are published: this lane's two, for the histogram updates
        const uint32_t* ha = p.calib + (size_t)(lane < p.nq ? lane : 0) * kCalibWords;
        const uint32_t* hb = p.calib + (size_t)(lane + 32 < p.nq ? lane + 32 : 0) * kCalibWords;
        // (the threshold warp saw every calibration's flag before it raised thr_ready, and these loads go to the L2)
        __threadfence();
        const uint4 ca = __ldcg(reinterpret_cast<const uint4*>(ha)), cb = __ldcg(reinterpret_cast<const uint4*>(hb));
        if (ca.z != 0u) {
          cal_lo_lo = __uint_as_float(ca.x);
          cal_pu_lo = __uint_as_float(ca.y);
        }
        if (cb.z != 0u) {
          cal_lo_hi = __uint_as_float(cb.x);
          cal_pu_hi = __uint_as_float(cb.y);
        }
      }
    };
    int it = 0, parked_emitted = 0;
    bool complete = true;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
      const bool parked = it < n_parked;
      const int wi = it - n_parked;
      const int b = parked ? kGemmAccBufs + it : wi % kGemmAccBufs;
      if (emitting && it == n_parked) await_thresholds();  // the first tile whose rows are compared with thresholds
      if (!mbar_wait(&acc_full[b], parked ? 0u : (uint32_t)((wi / kGemmAccBufs) & 1), abort_flag, limit)) {
        complete = false;
        break;
      }
      tc_fence_after();
      float v[kGemmMaxQ];
      const uint32_t taddr = lane_taddr + (uint32_t)(b * kGemmMaxQ);
      tmem_ld32(taddr, v);
      tmem_ld32(taddr + 32, v + 32);
      tmem_ld_wait();
      bool out;
      const int row = row_of(tile, out);
      if (emitting && !parked) {
        uint32_t m_lo, m_hi;
        passes(v, out, m_lo, m_hi);
        serve(taddr, row, m_lo, m_hi, true);
      }
      tc_fence_before();
      __syncwarp();
      if (!parked && lane == 0) mbar_arrive(&acc_empty[b]);  // the MMAs of a later tile may overwrite this buffer
      if (out) {
#pragma unroll
        for (int q = 0; q < kGemmMaxQ; ++q) v[q] = -INFINITY;
      }
#pragma unroll
      for (int q = 0; q < kGemmMaxQ; ++q) {
        float x = v[q];
        x = fmaxf(x, __shfl_xor_sync(kFull, x, 1));
        x = fmaxf(x, __shfl_xor_sync(kFull, x, 2));
        x = fmaxf(x, __shfl_xor_sync(kFull, x, 4));
        v[q] = x;
      }
      // transpose through shared memory, 32 queries at a time: lane q then owns the four group maxima of query q
      const int64_t col = (int64_t)tile * kGemmGroupsPerTile + quarter * 4;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if ((lane & 7) == 0) {
          float4* dst = reinterpret_cast<float4*>(my_stage + (lane >> 3) * 32);
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4)
            dst[q4] = make_float4(v[32 * h + 4 * q4], v[32 * h + 4 * q4 + 1], v[32 * h + 4 * q4 + 2], v[32 * h + 4 * q4 + 3]);
        }
        __syncwarp();
        const int q = lane + 32 * h;
        if (q < p.nq) {
          const float4 g = make_float4(my_stage[lane], my_stage[32 + lane], my_stage[64 + lane], my_stage[96 + lane]);
          *reinterpret_cast<float4*>(p.gmax + (int64_t)q * p.gmax_stride + col) = g;
          // a parked tile is computed before any threshold exists: the best of the warp's 32 rows goes to the table the
          // thresholds are calibrated from, and the rows are looked at again later
          if (parked) p.raw[(size_t)q * (32 * kRawPerLane) + (my_seg * kGemmParked + (size_t)it)] = fmaxf(fmaxf(g.x, g.y), fmaxf(g.z, g.w));
        }
        __syncwarp();
      }
      // the parked tiles' rows, once the thresholds have seen a few tiles of every CTA, in time the epilogue would
      // otherwise spend waiting for the next accumulator
      if (parked_emitted < n_parked && it >= n_parked + 3 + 2 * parked_emitted) emit_parked(parked_emitted++);
    }
    if (complete && parked_emitted < n_parked && parked_emitted < it) {  // a CTA with few tiles
      if (it <= n_parked) await_thresholds();
      while (parked_emitted < n_parked && parked_emitted < it) emit_parked(parked_emitted++);
    }
    if (emitting) {
      if (lane < p.nq) p.cand_cnt[(size_t)lane * n_seg + my_seg] = cnt_lo;
      if (lane + 32 < p.nq) p.cand_cnt[(size_t)(lane + 32) * n_seg + my_seg] = cnt_hi;
    }
    __syncwarp();
    if (lane == 0) atomicAdd(const_cast<int*>(epi_done), 1);
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int w = 0; w < 4096; ++w) __nanosleep(256);  // let copies that may still be in flight land
    if (threadIdx.x == 0) atomicExch(p.error_flag, 1);
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kGemmTmemCols) : "memory");
  }
}

// ---- host side: TMA tensor map of a row-major fp16 matrix [n_rows][row_elems], box = 64 elements x box_rows rows,
// 128-byte swizzle, zero fill outside the matrix.  The encoder is a driver entry point looked up through the runtime.
inline bool make_tmap_rows_f16(CUtensorMap* out, const void* base, uint64_t n_rows, uint64_t row_elems, uint32_t box_rows) {
  typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static encode_fn encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
      return false;
    encode = reinterpret_cast<encode_fn>(fn);
  }
  const cuuint64_t dims[2] = {row_elems, n_rows};
  const cuuint64_t strides[1] = {row_elems * 2};  // bytes between rows
  const cuuint32_t box[2] = {(cuuint32_t)kGemmKChunk, box_rows};
  const cuuint32_t elem_strides[2] = {1, 1};
  return encode(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem_strides,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace ms
