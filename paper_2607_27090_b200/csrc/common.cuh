// Shared device-side definitions of libmemstore (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ms {

// One row of the device fact table (the paper keeps this id -> location map on the CPU, Sec. 6.7;
// here it lives in HBM so that ids never leave the device).
struct FactRec {
  int32_t tok_off;   // first token of the fact in the K/V arena
  int32_t n_tokens;  // length of the fact in tokens
  int32_t user;      // owner segment
  int32_t resident;  // 0: embedding only, 1: K/V in the HBM arena, 2: K/V in the pinned host arena
};

// Tokens per injection tile: 8 consecutive positions aligned to a multiple of 8, so a tile never
// straddles a cache block whose size is a multiple of 8 (and covers whole smaller power-of-two blocks).
constexpr int kTileTokens = 8;

// A source token index with this bit set lives in the pinned host arena (the paper's CPU-offloaded store, Sec. 6.8)
// and is read over PCIe by the copy kernel; both arenas hold fewer than 2^30 tokens.
constexpr int32_t kHostTierBit = 0x40000000;

// A source token index with this bit set lives in the composition cache (see CcSlot): keys stored there are already
// rotated for the positions of the cached segment, so the copy kernel copies them as they are.
constexpr int32_t kCacheTierBit = 0x20000000;
constexpr int32_t kNoFill = (int32_t)0x80000000;  // TileDesc::fill_tok0 of a tile that is not recorded in the composition cache

// Work description of one tile, written by the plan kernel and read by the copy kernel.
struct __align__(16) TileDesc {
  int32_t pos0;                 // position of lane 0 (multiple of kTileTokens)
  int32_t fill_tok0;            // composition-cache token that lane 0's composed token is recorded at, or kNoFill
  int32_t pad[2];
  int32_t src_tok[kTileTokens]; // arena token of each lane, -1: nothing to do
  int64_t dst_off[kTileTokens]; // element offset block*block_stride + token*token_stride in the cache
};

// Counters shared by the plan and copy kernels of one inject call.  A store keeps two of them and alternates:
// the plan kernel of a call clears the pair the next call will use (calls on a store are ordered on the device).
// Control block of the injection calls of one store.  The planning CTAs of a call (one per request) leave it ready
// for the copy kernel and clean for the next call by themselves - the last one to finish publishes the tile count
// and zeroes the rest - so a call depends on no earlier call, memset or host-side bookkeeping, and a call recorded
// in a CUDA graph can be replayed at any time.
struct InjectCtrl {
  uint32_t n_tiles;    // tiles of this call: written by the last planning CTA, read by the copy kernel
  uint32_t work_next;  // work ticket of the staged copy kernel (zeroed by the last planning CTA)
  uint32_t acc;        // tiles claimed so far by the planning CTAs of the running call (zero between calls)
  uint32_t planned;    // planning CTAs that have finished (zero between calls)
};

// Composition cache (the paper's closing remark of the appendix "Position independence and rotation fidelity": the
// composed segment is cached across queries that reuse the same memory; it pays where composing is expensive, i.e. for
// facts of the host tier, Sec. 6.8).  A slot holds the composed K (rotated, bf16) and V of one request, keyed by the
// request's id list as given, its start position, its placement flags and the instruction prefix it used.
constexpr int kCcMaxK = 256;     // longest id list a segment can be keyed by
constexpr int kCcMaxSlots = 64;
struct CcSlot {
  uint32_t hash_lo, hash_hi;
  int32_t k, start, flags, prefix_src, prefix_len, m;
  uint32_t epoch;     // the store's cache epoch when the slot was filled (a different epoch: the slot is empty)
  uint32_t last_use;  // injection call that filled or hit the slot last
  int32_t pad[2];
  int32_t ids[kCcMaxK];
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}

__device__ __forceinline__ void st_stream8(uint2* p, const uint2& v) {
  asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(v.x), "r"(v.y) : "memory");
}

// Programmatic dependent launch: wait until the preceding kernel in the stream has completed and its
// writes are visible / allow the next kernel in the stream to start its prologue.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::); }


}  // namespace ms
