// Batched scoring on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), sm_100a only.  Step R2 for many
// queries that search ONE segment (Sec. 3.2: inner-product search; here 64 queries x 1M facts is a dense
// [facts x E] x [E x queries] contraction, the one place on the path that is GEMM-shaped).
//
// The kernel does not write the score matrix.  It is a FILTER: for every group of 8 consecutive embedding rows
// and every query it writes the largest score of the group (fp32), 1/8 of a score matrix.  A later step picks the
// best groups per query and rescores their rows with the exact CUDA-core routine, so tensor-core rounding never
// decides a rank; it only has to keep every top-k row inside a selected group.
//
// Tiling: facts on M (128 rows per tile = the 128 TMEM lanes), queries on N (64), K = E in chunks of 64 fp16
// (one 128-byte swizzle row).  All queries stay in shared memory for the kernel's lifetime (E/64 chunks of 8 KiB);
// embedding tiles stream through a 4-stage ring of 16 KiB TMA boxes.  Accumulators are double-buffered in TMEM
// (2 x 64 columns) so that the epilogue of a tile overlaps the MMAs of the next.
//   warp 0     TMA producer (one elected lane)
//   warp 1     TMEM allocation, tcgen05.mma issue (one elected lane), tcgen05.commit -> mbarriers
//   warps 2-5  epilogue: tcgen05.ld of the warp's 32 TMEM lanes, row mask, 8-row max by shuffles, 16-byte stores
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
constexpr int kGemmThreads = 192;
constexpr int kGemmTmemCols = 128;
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
};

// Shared memory after the 1 KiB alignment of the base: queries, ring, epilogue staging (4 warps x [4 groups][32
// queries] floats), barriers.
constexpr uint32_t kGemmStagingBytes = 4 * 4 * 32 * sizeof(float);
constexpr uint32_t kGemmBarrierBytes = 256;
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
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

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
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], 4);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
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
        const int b = it & 1;
        ok = mbar_wait(&acc_empty[b], (uint32_t)((it >> 1) & 1) ^ 1u, abort_flag, limit);
        if (!ok) break;
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
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, 32*quarter + 32) belong to this warp
    float* my_stage = stage_f + (size_t)(warp - 2) * 4 * 32;
    int it = 0;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
      const int b = it & 1;
      if (!mbar_wait(&acc_full[b], (uint32_t)((it >> 1) & 1), abort_flag, limit)) break;
      tc_fence_after();
      float v[kGemmMaxQ];
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(b * kGemmMaxQ);
      tmem_ld32(taddr, v);
      tmem_ld32(taddr + 32, v + 32);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[b]);  // the MMAs of the tile after next may overwrite this buffer
      const int row = tile * kGemmTileRows + quarter * 32 + lane;
      bool out = row >= p.n_rows;
      if (!out && p.removed_bits != nullptr) out = (__ldg(p.removed_bits + (row >> 5)) >> (row & 31)) & 1u;
      if (out) {
#pragma unroll
        for (int q = 0; q < kGemmMaxQ; ++q) v[q] = -INFINITY;
      }
#pragma unroll
      for (int q = 0; q < kGemmMaxQ; ++q) {
        float x = v[q];
        x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 1));
        x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 2));
        x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 4));
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
        }
        __syncwarp();
      }
    }
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
