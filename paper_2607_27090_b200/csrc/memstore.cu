// Host side of libmemstore.so: the fact store in HBM and the C ABI declared in include/memstore.h.
// All compute is in the kernels of inject.cuh / retrieve.cuh; this file validates arguments, owns
// device memory and enqueues launches.  There is no CPU implementation of any step.
#include "../../include/memstore.h"

#include <atomic>
#include <chrono>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include <nvtx3/nvToolsExt.h>  // header-only: ranges cost nothing unless a profiler is attached

#include "common.cuh"
#include "inject.cuh"
#include "inject_tma.cuh"
#include "retrieve.cuh"
#include "score_gemm.cuh"
#include "ann.cuh"

using namespace ms;

struct memstore {
  memstore_config cfg{};
  int sm_count = 0;
  // device memory
  __nv_bfloat16* k_arena = nullptr;  // [L][max_kv_tokens][h][d]
  __nv_bfloat16* v_arena = nullptr;
  void* arena_alloc = nullptr;       // non-null when the store owns the arena
  __nv_bfloat16* k_host = nullptr;   // pinned host arena [L][max_host_kv_tokens][h][d] (K then V), host address
  __nv_bfloat16* v_host = nullptr;
  __nv_bfloat16* k_host_dev = nullptr;  // the same memory as the device sees it
  __nv_bfloat16* v_host_dev = nullptr;
  void* host_arena_alloc = nullptr;
  int64_t host_tokens_used = 0;
  void* emb = nullptr;               // [n_users][max_facts_per_user][emb_dim]
  int32_t* emb_fact_id = nullptr;    // [n_users][max_facts_per_user]
  int32_t* user_count_d = nullptr;   // [n_users]
  FactRec* facts_d = nullptr;        // [n_users * max_facts_per_user]
  float* inv_freq_d = nullptr;       // [d/2]
  // scratch shared by all calls (ordered on the device through `last_done`)
  float* scores = nullptr;
  uint32_t* tickets = nullptr;  // one wait-free counter per query of the fused retrieve kernel
  // tensor-core retrieve path (allocated on first use): group maxima, selected groups, candidate scores / rows
  float* tc_gmax = nullptr;
  int64_t tc_gmax_stride = 0;
  int32_t* tc_sel = nullptr;
  float* tc_cand_scores = nullptr;
  int32_t* tc_cand_rows = nullptr;
  uint32_t* tc_tickets = nullptr;
  float* tc_next_best = nullptr;  // per query: the filter's best score among the rows that are not rescored
  float* tc_kth = nullptr;        // per query: the k-th exact score after rescoring
  int* tc_redo = nullptr;         // per query: the margin check failed, the fix-up kernel rescans the segment
  float* tc_scores_out = nullptr; // [64][kTcMaxK] exact scores by rank when the caller asks for none
  uint32_t* tc_fix_counts = nullptr;
  unsigned long long* tc_fix_keys = nullptr;  // [64][kFixupCap]
  uint32_t* tc_fix_tickets = nullptr;
  uint32_t* tc_n_fixups = nullptr;  // queries the fix-up kernel has redone since creation
  int* tc_error = nullptr;
  uint32_t* serve_flag_dev = nullptr;  // memstore_serve_host, early return: device address of the pinned flag word, while its call runs
  uint32_t serve_seq = 0;              // value the flag takes for the current request
  // candidate rows emitted by the filter kernel (see score_gemm.cuh)
  uint32_t* tc_hist = nullptr;      // [64][kHistWords] + thr_used[64] (zero between calls) + cand_cnt[64][kCandMaxSegs]
  float* tc_raw = nullptr;                // [64][32 * kRawPerLane]: the table the thresholds of the lists are calibrated from
  unsigned long long* tc_emit = nullptr;  // [64][kTcCandPlaces]: candidate rows listed by the filter kernel
  float* tc_exact = nullptr;        // [64][kListMaxK2]: exact scores of the listed rows that were rescored, by filter rank
  unsigned long long* tc_list_stats = nullptr;  // queries served from their candidate list, rows listed for them, fallbacks
  bool tc_ready = false;
  int64_t scores_nq = 0;
  TileDesc* tiles = nullptr;
  int prof_repeats = 1;        // measurement aid: launches of the copy kernel per inject call while profile events are set
  bool store_changed = false;  // facts, prefix or removals enqueued since the last serving call: that call must order itself after them
  uint32_t tiles_capacity = 0;
  InjectCtrl* ctrl = nullptr;  // one control block, kept clean by the planning kernels themselves
  cudaEvent_t last_done = nullptr;
  cudaEvent_t prof_before = nullptr, prof_after = nullptr;  // caller-owned, optional
  // memstore_serve_host staging: one pinned host buffer and one device buffer, inputs first, outputs after
  unsigned char* host_stage = nullptr;
  cudaStream_t serve_stream = nullptr;  // memstore_serve_host, early return: the inputs go up on this stream
  unsigned char* dev_stage = nullptr;
  size_t stage_bytes = 0;
  cudaStream_t last_stream = nullptr;
  bool have_last = false;
  // host mirrors
  std::vector<int64_t> user_count;
  int64_t n_facts = 0, n_resident = 0, kv_tokens_used = 0;
  int32_t max_fact_len = 0;
  // proximity graphs, one per user segment (memstore_build_graph / memstore_set_graph): [n_users][graph_cap_rows][graph_deg],
  // rows of a user's graph are rows of that user's segment
  int32_t* graph = nullptr;
  std::vector<int64_t> graph_rows;  // rows each user's graph covers
  int32_t* graph_rows_d = nullptr;  // the same on the device, [n_users]
  int32_t* graph_users_d = nullptr; // scratch: a batch of equal user numbers (queries of one user while building)
  int64_t graph_cap_rows = 0;  // rows per user the graph array has room for (a single-segment store grows it geometrically)
  int32_t graph_deg = 0;
  // removed facts (memstore_remove_fact): one bit per embedding row, host mirror and device copy (allocated on first removal)
  std::vector<uint32_t> removed_bits;
  uint32_t* removed_bits_d = nullptr;
  int64_t n_removed = 0;
  struct IdRun { int32_t first_id, n, user; int64_t slot0; };
  std::vector<IdRun> id_runs;  // which rows the ids of each add call went to (ids are dense in insertion order)
  int32_t* graph_topk = nullptr;  // build scratch: [64][deg + 1] ids
  size_t graph_topk_cap = 0;      // its size in entries
  unsigned long long* append_pairs = nullptr;  // graph_append scratch: sorted (old row, new row) offers, then their count
  int64_t prefix_off = 0;   // instruction prefix (memstore_set_prefix): first arena token and length (0 = none)
  int32_t prefix_len = 0;
  int64_t prefix_tokens_total = 0;  // arena tokens taken by this and earlier prefixes (not facts)
  int64_t max_user_count = 0;
  int64_t retrieve_calls = 0, inject_calls = 0, kernels_launched = 0;
  // composition cache (memstore_compose_cache): composed segments of earlier requests, least recently used evicted
  CcSlot* cc_slots = nullptr;
  __nv_bfloat16* cc_arena = nullptr;  // K half then V half, each [L][cc_n_slots * cc_slot_tokens][h][d]
  uint32_t* cc_counters = nullptr;    // [0] hits, [1] fills
  int32_t cc_n_slots = 0, cc_slot_tokens = 0, cc_fill_all = 0;
  uint32_t cc_epoch = 1, cc_call = 0;
  uint32_t test_spin_limit = 0;  // memstore_test_hooks
  int test_mute_producers = 0;
  int copy_ctas_per_sm = 1;
  bool tma_path = false;  // MS_STORE_TMA_COPY_PATH
  std::recursive_mutex mu;  // recursive: memstore_serve_host holds it across retrieve and inject
  std::string err;
};

namespace {

// MEMSTORE_LOG=1 in the environment makes every refused call print its reason to stderr (read once).
bool log_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("MEMSTORE_LOG");
    return e && e[0] && e[0] != '0';
  }();
  return on;
}

ms_status fail(memstore* s, ms_status code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (s) s->err = buf;
  if (log_enabled()) fprintf(stderr, "[memstore] status %d: %s\n", (int)code, buf);
  return code;
}

// A named range around a public call, visible in profilers' timelines.
struct Range {
  explicit Range(const char* name) { nvtxRangePushA(name); }
  ~Range() { nvtxRangePop(); }
};

#define MS_CUDA(s, call)                                                                         \
  do {                                                                                           \
    cudaError_t e_ = (call);                                                                     \
    if (e_ != cudaSuccess)                                                                       \
      return fail(s, e_ == cudaErrorMemoryAllocation ? MS_ERR_OOM : MS_ERR_CUDA, "%s: %s", #call, \
                  cudaGetErrorString(e_));                                                       \
  } while (0)

size_t emb_elem_size(int dtype) { return dtype == MS_DTYPE_F32 ? 4 : 2; }

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    if (prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

ms_status check_config(const memstore_config* c) {
  if (!c) return MS_ERR_INVALID_ARG;
  if (c->n_layers <= 0 || c->n_kv_heads <= 0 || c->emb_dim <= 0 || c->n_users <= 0) return MS_ERR_INVALID_ARG;
  if (c->max_facts_per_user <= 0 || c->max_kv_tokens < 0) return MS_ERR_INVALID_ARG;
  if (c->max_position <= 0 || c->max_position > (1 << 24)) return MS_ERR_INVALID_ARG;
  if (c->rope_style != MS_ROPE_HALF_SPLIT && c->rope_style != MS_ROPE_INTERLEAVED) return MS_ERR_INVALID_ARG;
  if (!(c->rope_theta > 0.0) && !c->inv_freq_override) return MS_ERR_INVALID_ARG;
  if (c->flags & ~(uint32_t)MS_STORE_TMA_COPY_PATH) return MS_ERR_INVALID_ARG;
  if (c->kv_dtype != MS_DTYPE_BF16) return MS_ERR_UNSUPPORTED;
  if (c->emb_dtype != MS_DTYPE_F32 && c->emb_dtype != MS_DTYPE_F16) return MS_ERR_UNSUPPORTED;
  if (c->emb_dim % 8) return MS_ERR_UNSUPPORTED;
  // the copy kernels give 32 or more threads to a token and one frequency octet to a thread: d/16 must divide 32
  const int d = c->head_dim;
  if (!(d == 16 || d == 32 || d == 64 || d == 128 || d == 256)) return MS_ERR_UNSUPPORTED;
  if (c->rotary_dim < 0 || c->rotary_dim > d || (c->rotary_dim % 16) || c->reserved1 != 0) return MS_ERR_INVALID_ARG;
  if (c->max_host_kv_tokens < 0 || c->max_host_kv_tokens >= (1ll << 30) || c->max_kv_tokens >= (1ll << 30) || (int64_t)c->n_users * c->max_facts_per_user >= (1ll << 31))
    return MS_ERR_UNSUPPORTED;
  return MS_OK;
}

// ---- arena append: src [L][T][row] -> arena [L][cap][row] at token offset, K and V in one launch ----
__global__ void __launch_bounds__(256) arena_append_kernel(const uint4* __restrict__ k_src, const uint4* __restrict__ v_src,
                                                           uint4* __restrict__ k_dst, uint4* __restrict__ v_dst,
                                                           int64_t vec_per_layer_src, int64_t vec_per_layer_dst,
                                                           int64_t dst_vec_off) {
  const int layer = blockIdx.y;
  const uint4* s = (blockIdx.z ? v_src : k_src) + (int64_t)layer * vec_per_layer_src;
  uint4* d = (blockIdx.z ? v_dst : k_dst) + (int64_t)layer * vec_per_layer_dst + dst_vec_off;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < vec_per_layer_src; i += (int64_t)gridDim.x * blockDim.x)
    d[i] = s[i];
}

// The dynamic shared memory limit of a kernel is a per-device property of the function, shared by all stores:
// it is only ever raised.
cudaError_t ensure_fused_smem(int device, size_t bytes) {
  static std::mutex mu;
  static size_t set_bytes[64] = {0};
  std::lock_guard<std::mutex> lock(mu);
  const int d = device & 63;
  if (bytes <= set_bytes[d]) return cudaSuccess;
  cudaError_t e = cudaSuccess;
  const void* fns[] = {(const void*)score_topk_fused_kernel<__half, kFusedThreadsFew>, (const void*)score_topk_fused_kernel<float, kFusedThreadsFew>,
                       (const void*)score_topk_fused_kernel<__half, kFusedThreadsBig>, (const void*)score_topk_fused_kernel<float, kFusedThreadsBig>,
                       (const void*)score_topk_plan_kernel<__half, kFusedThreadsBig>, (const void*)score_topk_plan_kernel<float, kFusedThreadsBig>,
                       (const void*)score_topk_fused_kernel<__half, kFusedThreadsMany>, (const void*)score_topk_fused_kernel<float, kFusedThreadsMany>,
                       (const void*)score_topk_plan_kernel<__half, kFusedThreadsFew>, (const void*)score_topk_plan_kernel<float, kFusedThreadsFew>,
                       (const void*)score_topk_plan_kernel<__half, kFusedThreadsMany>, (const void*)score_topk_plan_kernel<float, kFusedThreadsMany>};
  for (const void* fn : fns)
    if (e == cudaSuccess) e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) set_bytes[d] = bytes;
  return e;
}

// ---- tensor-core retrieve path -------------------------------------------------------------------------------
constexpr int kTcMinQueries = 8;     // below this the CUDA-core kernels re-reading the segment per query are cheaper ...
constexpr int64_t kTcFewQueriesRows = 131072;  // ... unless the segment is long: the filter reads it once whatever the number
                                               // of queries and leaves 1/8 of the scores to select from, while the CUDA-core
                                               // path ends in one CTA selecting among ALL scores at one SM's bandwidth
constexpr int kTcMaxK = 256;
constexpr int kTcGroupMargin = 28;   // groups selected beyond k: slack for tensor-core vs CUDA-core rounding at the k-th score
constexpr int kTcMaxK2 = kTcMaxK + kTcGroupMargin;
constexpr int kTcCandPlaces = 16384;  // candidate places per query over all epilogue warps of the filter kernel
constexpr int kTcCandSeg = 24;                          // places per epilogue warp of the filter kernel and query
constexpr int kTcMaxCtas = kCandMaxSegs / 4;
constexpr int kTcRowMargin = 28;     // candidate rows rescored beyond k
static_assert(kTcMaxK + kTcRowMargin <= kListMaxK2, "the list kernel's per-query arrays hold k + margin rows");
constexpr size_t kTcHistWords = (size_t)kGemmMaxQ * (kHistWords + kCalibWords + 1 + kCandMaxSegs);

// Launch as a programmatic dependent of the kernel before it in the stream (the kernel calls griddepcontrol.wait before
// it touches anything the earlier kernels write).
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t lc{};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.gridDim = grid;
  lc.blockDim = block;
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, kernel, KArgs(std::forward<Args>(args))...);
}

bool tc_path_applies(const memstore* s, const int32_t* query_users, int nq, int k, int64_t n_max) {
  const memstore_config& c = s->cfg;
  return c.emb_dtype == MS_DTYPE_F16 && c.emb_dim % kGemmKChunk == 0 && c.emb_dim <= kGemmMaxE && !query_users &&
         (nq >= kTcMinQueries || n_max >= kTcFewQueriesRows) && k <= kTcMaxK && n_max > kFusedMaxRows;
}

ms_status tc_prepare(memstore* s) {
  if (s->tc_ready) return MS_OK;
  const memstore_config& c = s->cfg;
  const int64_t tiles = (c.max_facts_per_user + kGemmTileRows - 1) / kGemmTileRows;
  s->tc_gmax_stride = tiles * kGemmGroupsPerTile;
  MS_CUDA(s, cudaDeviceSynchronize());
  MS_CUDA(s, cudaMalloc(&s->tc_gmax, (size_t)kGemmMaxQ * s->tc_gmax_stride * sizeof(float)));
  MS_CUDA(s, cudaMalloc(&s->tc_sel, (size_t)kGemmMaxQ * kTcMaxK2 * sizeof(int32_t)));
  MS_CUDA(s, cudaMalloc(&s->tc_cand_scores, (size_t)kGemmMaxQ * kTcMaxK2 * 8 * sizeof(float)));
  MS_CUDA(s, cudaMalloc(&s->tc_cand_rows, (size_t)kGemmMaxQ * kTcMaxK2 * 8 * sizeof(int32_t)));
  MS_CUDA(s, cudaMalloc(&s->tc_tickets, (size_t)kGemmMaxQ * sizeof(uint32_t)));
  MS_CUDA(s, cudaMalloc(&s->tc_next_best, (size_t)kGemmMaxQ * sizeof(float)));
  MS_CUDA(s, cudaMalloc(&s->tc_kth, (size_t)kGemmMaxQ * sizeof(float)));
  MS_CUDA(s, cudaMalloc(&s->tc_redo, (size_t)kGemmMaxQ * sizeof(int)));
  MS_CUDA(s, cudaMalloc(&s->tc_scores_out, (size_t)kGemmMaxQ * kTcMaxK * sizeof(float)));
  MS_CUDA(s, cudaMalloc(&s->tc_fix_counts, (size_t)kGemmMaxQ * sizeof(uint32_t)));
  MS_CUDA(s, cudaMalloc(&s->tc_fix_keys, (size_t)kGemmMaxQ * kFixupCap * sizeof(unsigned long long)));
  MS_CUDA(s, cudaMalloc(&s->tc_fix_tickets, (size_t)kGemmMaxQ * sizeof(uint32_t)));
  MS_CUDA(s, cudaMalloc(&s->tc_n_fixups, 2 * sizeof(uint32_t)));
  MS_CUDA(s, cudaMalloc(&s->tc_error, 2 * sizeof(int)));
  MS_CUDA(s, cudaMalloc(&s->tc_hist, kTcHistWords * sizeof(uint32_t)));
  MS_CUDA(s, cudaMalloc(&s->tc_emit, (size_t)kGemmMaxQ * kTcCandPlaces * sizeof(unsigned long long)));
  MS_CUDA(s, cudaMalloc(&s->tc_raw, (size_t)kGemmMaxQ * 32 * kRawPerLane * sizeof(float)));
  MS_CUDA(s, cudaMemset(s->tc_raw, 0xff, (size_t)kGemmMaxQ * 32 * kRawPerLane * sizeof(float)));  // every word kRawEmpty
  MS_CUDA(s, cudaMalloc(&s->tc_exact, (size_t)kGemmMaxQ * kListMaxK2 * sizeof(float)));
  MS_CUDA(s, cudaMemset(s->tc_hist, 0, kTcHistWords * sizeof(uint32_t)));
  MS_CUDA(s, cudaMalloc(&s->tc_list_stats, 3 * sizeof(unsigned long long)));
  MS_CUDA(s, cudaMemset(s->tc_list_stats, 0, 3 * sizeof(unsigned long long)));
  MS_CUDA(s, cudaMemset(s->tc_tickets, 0, (size_t)kGemmMaxQ * sizeof(uint32_t)));
  MS_CUDA(s, cudaMemset(s->tc_redo, 0, (size_t)kGemmMaxQ * sizeof(int)));
  MS_CUDA(s, cudaMemset(s->tc_fix_counts, 0, (size_t)kGemmMaxQ * sizeof(uint32_t)));
  MS_CUDA(s, cudaMemset(s->tc_fix_tickets, 0, (size_t)kGemmMaxQ * sizeof(uint32_t)));
  MS_CUDA(s, cudaMemset(s->tc_n_fixups, 0, 2 * sizeof(uint32_t)));
  MS_CUDA(s, cudaMemset(s->tc_error, 0, 2 * sizeof(int)));
  MS_CUDA(s, cudaFuncSetAttribute(tc_fixup_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kFixupCap * sizeof(unsigned long long))));
  MS_CUDA(s, cudaFuncSetAttribute(score_gemm_groupmax_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGemmSmemBytes));
  const size_t rs = (size_t)kTcMaxK2 * 8 * sizeof(uint32_t);
  MS_CUDA(s, cudaFuncSetAttribute(rescore_topk_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rs));
  s->tc_ready = true;
  return MS_OK;
}

// Many queries on the one segment of user 0: (1) tcgen05 GEMM that keeps only the maximum score of every group of 8
// rows, (2) per query the k + margin best groups, (3) exact CUDA-core rescoring of their rows and top-k.
ms_status retrieve_tensor_core(memstore* s, const RetrieveParams& base, int64_t n_rows, cudaStream_t st) {
  const memstore_config& c = s->cfg;
  ms_status rc = tc_prepare(s);
  if (rc != MS_OK) return rc;
  const int n_groups = (int)((n_rows + kGemmGroupRows - 1) / kGemmGroupRows);
  const int k2 = std::min(kTcMaxK2, base.k + kTcGroupMargin);
  const int n_tiles = (int)((n_rows + kGemmTileRows - 1) / kGemmTileRows);
  CUtensorMap tmap_emb;
  if (!make_tmap_rows_f16(&tmap_emb, s->emb, (uint64_t)n_rows, (uint64_t)c.emb_dim, kGemmTileRows))
    return fail(s, MS_ERR_CUDA, "cuTensorMapEncodeTiled failed for the embedding matrix");
  const size_t esz = 2;
  for (int q0 = 0; q0 < base.nq; q0 += kGemmMaxQ) {
    const int nqb = std::min(kGemmMaxQ, base.nq - q0);
    const char* qptr = (const char*)base.queries + (size_t)q0 * c.emb_dim * esz;
    CUtensorMap tmap_q;
    if (!make_tmap_rows_f16(&tmap_q, qptr, (uint64_t)nqb, (uint64_t)c.emb_dim, kGemmMaxQ))
      return fail(s, MS_ERR_CUDA, "cuTensorMapEncodeTiled failed for the query batch");
    // Candidate rows from the filter kernel itself when k leaves room in the selection that ranks them and the CTAs
    // have several tiles each (the thresholds need the other CTAs' first tiles); the group maxima serve the rest and
    // any query whose list turns out unusable.
    const int k2r = base.k + kTcRowMargin;
    const int n_ctas = std::min(n_tiles, s->sm_count);
    const int n_seg = n_ctas * 4;
    const int seg = std::min(kTcCandSeg, kTcCandPlaces / n_seg);
    const bool emit = k2r <= kListMaxK2 && n_tiles >= kGemmParked * s->sm_count && n_rows >= k2r && n_ctas <= kTcMaxCtas && seg >= 8 &&
                      n_ctas >= nqb && n_ctas * 4 * kGemmParked <= 32 * kRawPerLane && n_ctas * 4 * kGemmParked >= k2r;
    uint32_t* hist = s->tc_hist;
    uint32_t* calib = hist + (size_t)kGemmMaxQ * kHistWords;  // (the list kernel zeroes a query's counters and calibration as one run of words)
    uint32_t* thr_used = calib + (size_t)kGemmMaxQ * kCalibWords;
    uint32_t* cand_cnt = thr_used + kGemmMaxQ;
    GemmParams gp{(int)n_rows, c.emb_dim, nqb, s->tc_gmax, s->tc_gmax_stride, s->tc_error, (uint32_t)kGemmSmemBytes,
                  s->test_spin_limit, s->test_mute_producers, s->removed_bits_d,
                  emit ? hist : nullptr, calib, s->tc_raw, cand_cnt, thr_used, s->tc_emit, seg, k2r};
    MS_CUDA(s, launch_dependent(score_gemm_groupmax_kernel, dim3((unsigned)n_ctas), dim3(kGemmThreads), kGemmSmemBytes, st, tmap_emb, tmap_q, gp));
    RetrieveParams p = base;
    p.queries = qptr;
    p.nq = nqb;
    p.out_ids = base.out_ids + (int64_t)q0 * base.k;
    p.out_scores = base.out_scores ? base.out_scores + (int64_t)q0 * base.k : nullptr;
    float* scores_out = p.out_scores ? p.out_scores : s->tc_scores_out;
    if (emit) {
      // one launch selects among the listed rows, rescores them and writes the top-k (a query whose list is unusable is
      // served from the group maxima by one CTA of the same launch)
      MS_CUDA(s, launch_dependent(list_topk_kernel<__half>, dim3(kListCtas, (unsigned)nqb), dim3(kListThreads), (size_t)k2 * 8 * sizeof(uint32_t),
                                  st, p, (const unsigned long long*)s->tc_emit, n_seg, seg, (const uint32_t*)cand_cnt, thr_used, hist, kHistWords, calib,
                                  k2r, s->tc_exact, s->tc_tickets, scores_out, s->tc_redo, s->tc_kth, s->tc_list_stats, (const float*)s->tc_gmax,
                                  s->tc_gmax_stride, n_groups, k2, (int)n_rows, s->tc_cand_scores, s->tc_cand_rows, reinterpret_cast<uint32_t*>(s->tc_raw),
                                  32 * kRawPerLane, n_ctas * 4 * kGemmParked));
      s->kernels_launched += 1;
    } else {
      MS_CUDA(s, launch_dependent(select_groups_kernel, dim3((unsigned)nqb), dim3(kTopkThreads), 0, st, (const float*)s->tc_gmax,
                                  s->tc_gmax_stride, n_groups, k2, s->tc_sel, s->tc_next_best));
      dim3 grid((unsigned)((k2 + kScoreWarps - 1) / kScoreWarps), (unsigned)nqb);
      MS_CUDA(s, launch_dependent(rescore_topk_kernel<__half>, grid, dim3(kScoreThreads), (size_t)k2 * 8 * sizeof(uint32_t), st, p,
                                  (const int32_t*)s->tc_sel, k2, (int)n_rows, s->tc_cand_scores, s->tc_cand_rows, s->tc_tickets, scores_out,
                                  (const float*)s->tc_next_best, s->tc_redo, s->tc_kth));
      s->kernels_launched += 2;
    }
    // the fix-up of the queries whose margin check failed (its CTAs leave at once for all the others, so the grid is
    // kept small: a few CTAs per query, each taking a slice of the segment)
    const int fix_ctas = std::max(1, std::min(8 * s->sm_count / nqb, (int)((n_rows + 2047) / 2048)));
    const int fix_rows = (int)(((n_rows + fix_ctas - 1) / fix_ctas + 1) & ~(int64_t)1);
    dim3 fgrid((unsigned)((n_rows + fix_rows - 1) / fix_rows), (unsigned)nqb);
    MS_CUDA(s, launch_dependent(tc_fixup_kernel<__half>, fgrid, dim3(kScoreThreads), kFixupCap * sizeof(unsigned long long), st, p,
                                (int)n_rows, fix_rows, s->tc_redo, (const float*)s->tc_kth, s->tc_fix_counts, s->tc_fix_keys,
                                s->tc_fix_tickets, scores_out, s->tc_error + 1, s->tc_n_fixups));
    s->kernels_launched += 2;
  }
  return MS_OK;
}

// Launch of the one-launch scoring + top-k (+ plan) kernels: 1024-thread CTAs when few queries are served (the last
// CTA of a query selects and plans alone, which wants many threads), 256-thread CTAs otherwise.
template <typename T, int THREADS, bool PLAN>
void launch_score_topk_threads(int sm_count, int nq, int64_t n_max, const RetrieveParams& p, uint32_t* tickets, int keys_cap, int n_host,
                               const InjectParams* ip, size_t smem, cudaStream_t st, int early) {
  // enough CTAs to fill the GPU, at least one row per warp
  constexpr int64_t kWarps = THREADS / 32;
  // (a 1024-thread CTA fills an SM: more CTAs than SMs would only queue behind the first wave)
  // (256-thread CTAs are held to 64 registers so that four of them share an SM: as many CTAs as fit at once, so that the
  // whole grid is one wave and nothing waits for an SM to be refilled)
  const int64_t target_ctas = std::max<int64_t>(1, (int64_t)sm_count * (THREADS >= 1024 ? 1 : THREADS >= 512 ? 2 : 4) / nq);
  int64_t rows = std::max<int64_t>(kWarps, (std::max<int64_t>(n_max, 1) + target_ctas - 1) / target_ctas);
  rows = (rows + kWarps - 1) / kWarps * kWarps;
  const int rows_per_cta = (int)rows;
  const dim3 grid((unsigned)((std::max<int64_t>(n_max, 1) + rows_per_cta - 1) / rows_per_cta), (unsigned)nq);
  if constexpr (PLAN) {
    // A programmatic dependent of whatever precedes it in the stream: when that is this library's copy kernel (which
    // lets its dependents go as soon as all its CTAs have started) the CTAs of this kernel are placed on the SMs while
    // the copy kernel drains, and the launch latency between two requests disappears.  The kernel waits for the
    // preceding grid before it touches anything, so ordering is that of an ordinary launch.
    cudaLaunchConfig_t lc{};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.gridDim = grid;
    lc.blockDim = dim3(THREADS);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    lc.attrs = attr;
    lc.numAttrs = 1;
    cudaLaunchKernelEx(&lc, score_topk_plan_kernel<T, THREADS>, p, rows_per_cta, tickets, keys_cap, n_host, *ip, early);
  } else {
    // (a programmatic dependent as well: when retrieve calls follow one another, a call's CTAs are placed while the
    // call before it drains; the kernel waits for the preceding grid before it touches anything)
    launch_dependent(score_topk_fused_kernel<T, THREADS>, grid, dim3(THREADS), smem, st, p, rows_per_cta, tickets, keys_cap, n_host);
  }
}
template <typename T, bool PLAN>
void launch_score_topk(int sm_count, int nq, int64_t n_max, const RetrieveParams& p, uint32_t* tickets, int keys_cap, int n_host,
                       const InjectParams* ip, size_t smem, cudaStream_t st, int early = 0) {
  if (nq <= kFusedFewQueries && (n_max > (int64_t)kFusedThreadsFew * kExtractMaxKpl || (PLAN && p.k > kFusedPlanBigK)))
    launch_score_topk_threads<T, kFusedThreadsBig, PLAN>(sm_count, nq, n_max, p, tickets, keys_cap, n_host, ip, smem, st, early);
  else if (nq <= kFusedFewQueries)
    launch_score_topk_threads<T, kFusedThreadsFew, PLAN>(sm_count, nq, n_max, p, tickets, keys_cap, n_host, ip, smem, st, early);
  else
    launch_score_topk_threads<T, kFusedThreadsMany, PLAN>(sm_count, nq, n_max, p, tickets, keys_cap, n_host, ip, smem, st, early);
}

RetrieveParams retrieve_params(const memstore* s, const void* queries, const int32_t* query_users, int nq, int k, float* scores,
                               int32_t* out_ids, float* out_scores) {
  const memstore_config& c = s->cfg;
  RetrieveParams p{};
  p.emb = s->emb;
  p.emb_fact_id = s->emb_fact_id;
  p.user_count = s->user_count_d;
  p.seg_capacity = c.max_facts_per_user;
  p.n_users = c.n_users;
  p.emb_dim = c.emb_dim;
  p.queries = queries;
  p.query_users = query_users;
  p.nq = nq;
  p.k = k;
  p.scores = scores;
  p.score_stride = c.max_facts_per_user;
  p.out_ids = out_ids;
  p.out_scores = out_scores;
  p.removed_bits = s->removed_bits_d;
  p.return_rows = 0;
  return p;
}

// Scratch that grows on first use.  Each helper synchronises the device only when it really has to allocate;
// memstore_reserve calls them ahead of serving so that no later call does.
ms_status ensure_scores(memstore* s, int64_t nq) {
  if (nq <= s->scores_nq) return MS_OK;
  MS_CUDA(s, cudaDeviceSynchronize());
  cudaFree(s->scores);
  cudaFree(s->tickets);
  s->scores = nullptr;
  s->tickets = nullptr;
  s->scores_nq = 0;
  MS_CUDA(s, cudaMalloc(&s->scores, (size_t)nq * s->cfg.max_facts_per_user * sizeof(float)));
  MS_CUDA(s, cudaMalloc(&s->tickets, (size_t)nq * sizeof(uint32_t)));
  MS_CUDA(s, cudaMemset(s->tickets, 0, (size_t)nq * sizeof(uint32_t)));
  s->scores_nq = nq;
  return MS_OK;
}

ms_status ensure_tiles(memstore* s, int64_t tiles_needed) {
  if (tiles_needed <= s->tiles_capacity) return MS_OK;
  if (tiles_needed > 0x7fffffff) return fail(s, MS_ERR_UNSUPPORTED, "request batch too large");
  MS_CUDA(s, cudaDeviceSynchronize());
  cudaFree(s->tiles);
  s->tiles = nullptr;
  s->tiles_capacity = 0;
  MS_CUDA(s, cudaMalloc(&s->tiles, (size_t)tiles_needed * sizeof(TileDesc)));
  s->tiles_capacity = (uint32_t)tiles_needed;
  return MS_OK;
}

ms_status ensure_stage(memstore* s, size_t bytes) {
  if (bytes <= s->stage_bytes) return MS_OK;
  MS_CUDA(s, cudaDeviceSynchronize());
  cudaFree(s->dev_stage);
  if (s->host_stage) cudaFreeHost(s->host_stage);
  s->dev_stage = nullptr;
  s->host_stage = nullptr;
  s->stage_bytes = 0;
  const size_t want = bytes * 2;
  MS_CUDA(s, cudaMalloc(&s->dev_stage, want));
  MS_CUDA(s, cudaHostAlloc(&s->host_stage, want, cudaHostAllocMapped));
  if (!s->serve_stream) MS_CUDA(s, cudaStreamCreateWithFlags(&s->serve_stream, cudaStreamNonBlocking));
  s->stage_bytes = want;
  return MS_OK;
}

// staging bytes of one memstore_serve_host request: [query | header | block table] and [ids | n_tokens, status]
void serve_host_layout(const memstore_config& c, int32_t max_blocks, int32_t k, size_t* q_bytes, size_t* in_bytes, size_t* out_bytes) {
  *q_bytes = ((size_t)c.emb_dim * emb_elem_size(c.emb_dtype) + 15) & ~(size_t)15;
  *in_bytes = *q_bytes + 16 + (((size_t)max_blocks * 4 + 15) & ~(size_t)15);
  *out_bytes = ((((size_t)k + 2) * 4 + 15) & ~(size_t)15) + 16;  // (the last 16 bytes: the flag word of an early return)
}

// Serialise use of the shared scratch across streams without a host sync: when a call arrives on another
// stream than the previous one, an event recorded at the tail of the previous stream is waited for.
// A stream that is being captured into a CUDA graph: the calls recorded on it run later, at every replay, and cannot
// wait on other streams' work.
bool stream_is_capturing(cudaStream_t st) {
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return cs != cudaStreamCaptureStatusNone;
}

ms_status order_after_last(memstore* s, cudaStream_t st) {
  if (stream_is_capturing(st)) return MS_OK;  // ordering a replay against other uses of the store is the caller's job
  if (s->have_last && s->last_stream != st) {
    MS_CUDA(s, cudaEventRecord(s->last_done, s->last_stream));
    MS_CUDA(s, cudaStreamWaitEvent(st, s->last_done, 0));
  }
  return MS_OK;
}
ms_status mark_last(memstore* s, cudaStream_t st) {
  if (stream_is_capturing(st)) return MS_OK;
  s->last_stream = st;
  s->have_last = true;
  return MS_OK;
}

}  // namespace

extern "C" {

const char* memstore_version(void) { return "memstore 0.1 sm_100a"; }

size_t memstore_arena_bytes(const memstore_config* c) {
  if (!c) return 0;
  return (size_t)2 * c->n_layers * (size_t)c->max_kv_tokens * c->n_kv_heads * c->head_dim * sizeof(__nv_bfloat16);
}

ms_status memstore_rope_table_llama3(int32_t rotary_dim, double rope_theta, double factor, double low_freq_factor,
                                     double high_freq_factor, double original_max_position, float* out) {
  if (rotary_dim <= 0 || (rotary_dim & 1) || !out || !(rope_theta > 0.0) || !(factor > 0.0) ||
      !(high_freq_factor > low_freq_factor) || !(low_freq_factor > 0.0) || !(original_max_position > 0.0))
    return MS_ERR_INVALID_ARG;
  const double kTwoPi = 6.283185307179586476925286766559;
  const double long_wave = original_max_position / low_freq_factor, short_wave = original_max_position / high_freq_factor;
  for (int i = 0; i < rotary_dim / 2; ++i) {
    const double f = std::pow(rope_theta, -(double)(2 * i) / (double)rotary_dim);
    const double wave = kTwoPi / f;
    double g = f;
    if (wave > long_wave) {
      g = f / factor;
    } else if (!(wave < short_wave)) {
      const double t = (original_max_position / wave - low_freq_factor) / (high_freq_factor - low_freq_factor);
      g = (1.0 - t) * f / factor + t * f;
    }
    out[i] = (float)g;
  }
  return MS_OK;
}

ms_status memstore_create(const memstore_config* config, memstore_t** out) {
  if (out) *out = nullptr;
  if (!out) return MS_ERR_INVALID_ARG;
  ms_status st = check_config(config);
  if (st != MS_OK) return st;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || config->device < 0 || config->device >= ndev) return MS_ERR_CUDA;
  memstore* s = new (std::nothrow) memstore();
  if (!s) return MS_ERR_OOM;
  s->cfg = *config;
  s->cfg.inv_freq_override = nullptr;
  DeviceGuard g(config->device);
  auto bail = [&](ms_status code) {
    memstore_destroy(s);
    return code;
  };
  if (!g.ok) return bail(MS_ERR_CUDA);
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, config->device) != cudaSuccess) return bail(MS_ERR_CUDA);
  s->sm_count = prop.multiProcessorCount;

  const size_t arena_bytes = memstore_arena_bytes(config);
  if (config->kv_arena) {
    if (config->kv_arena_bytes < arena_bytes || ((uintptr_t)config->kv_arena & 15)) return bail(MS_ERR_INVALID_ARG);
    s->k_arena = (__nv_bfloat16*)config->kv_arena;
  } else if (arena_bytes) {
    if (cudaMalloc(&s->arena_alloc, arena_bytes) != cudaSuccess) {
      cudaGetLastError();
      return bail(MS_ERR_OOM);
    }
    s->k_arena = (__nv_bfloat16*)s->arena_alloc;
  }
  s->v_arena = s->k_arena ? (__nv_bfloat16*)((char*)s->k_arena + arena_bytes / 2) : nullptr;
  if (config->max_host_kv_tokens > 0) {
    const size_t half = (size_t)config->n_layers * (size_t)config->max_host_kv_tokens * config->n_kv_heads * config->head_dim * sizeof(__nv_bfloat16);
    void* dptr = nullptr;
    if (cudaHostAlloc(&s->host_arena_alloc, 2 * half, cudaHostAllocMapped | cudaHostAllocPortable) != cudaSuccess ||
        cudaHostGetDevicePointer(&dptr, s->host_arena_alloc, 0) != cudaSuccess) {
      cudaGetLastError();
      return bail(MS_ERR_OOM);
    }
    s->k_host = (__nv_bfloat16*)s->host_arena_alloc;
    s->v_host = (__nv_bfloat16*)((char*)s->host_arena_alloc + half);
    s->k_host_dev = (__nv_bfloat16*)dptr;
    s->v_host_dev = (__nv_bfloat16*)((char*)dptr + half);
  }

  const int64_t rows = (int64_t)config->n_users * config->max_facts_per_user;
  const size_t esz = emb_elem_size(config->emb_dtype);
  bool ok = cudaMalloc(&s->emb, (size_t)rows * config->emb_dim * esz) == cudaSuccess &&
            cudaMalloc(&s->emb_fact_id, (size_t)rows * sizeof(int32_t)) == cudaSuccess &&
            cudaMalloc(&s->facts_d, (size_t)rows * sizeof(FactRec)) == cudaSuccess &&
            cudaMalloc(&s->user_count_d, (size_t)config->n_users * sizeof(int32_t)) == cudaSuccess &&
            cudaMalloc(&s->inv_freq_d, (size_t)(config->head_dim / 2) * sizeof(float)) == cudaSuccess &&
            cudaMalloc(&s->ctrl, sizeof(InjectCtrl)) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return bail(MS_ERR_OOM);
  }
  // RoPE frequencies: theta^(-2i/R) in double, rounded once to fp32 (Sec. 2.4; models keep this vector in fp32);
  // R = the rotary dimension, the whole head unless the configuration says otherwise.  Entries beyond R/2 are unused.
  if (s->cfg.rotary_dim == 0) s->cfg.rotary_dim = config->head_dim;
  const int R = s->cfg.rotary_dim;
  std::vector<float> f(config->head_dim / 2, 0.f);
  for (int i = 0; i < R / 2; ++i)
    f[i] = config->inv_freq_override ? config->inv_freq_override[i] : (float)std::pow(config->rope_theta, -(double)(2 * i) / (double)R);
  ok = cudaMemcpy(s->inv_freq_d, f.data(), f.size() * sizeof(float), cudaMemcpyHostToDevice) == cudaSuccess &&
       cudaMemset(s->user_count_d, 0, (size_t)config->n_users * sizeof(int32_t)) == cudaSuccess &&
       cudaMemset(s->ctrl, 0, sizeof(InjectCtrl)) == cudaSuccess &&
       cudaEventCreateWithFlags(&s->last_done, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return bail(MS_ERR_CUDA);
  }
  s->user_count.assign(config->n_users, 0);
  s->tma_path = (config->flags & MS_STORE_TMA_COPY_PATH) != 0 && config->max_host_kv_tokens == 0;  // HBM arena only
  int occ = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, inject_copy_kernel<0, 0>, kCopyThreads, 0) == cudaSuccess && occ > 0)
    s->copy_ctas_per_sm = occ;
  if (cudaFuncSetAttribute(inject_copy_tma_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTmaSmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(inject_copy_tma_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTmaSmemBytes) != cudaSuccess) {
    cudaGetLastError();
    return bail(MS_ERR_CUDA);
  }
  *out = s;
  return MS_OK;
}

ms_status memstore_destroy(memstore_t* s) {
  if (!s) return MS_OK;
  {
    DeviceGuard g(s->cfg.device);
    cudaDeviceSynchronize();
    cudaFree(s->arena_alloc);
    if (s->host_arena_alloc) cudaFreeHost(s->host_arena_alloc);
    cudaFree(s->emb);
    cudaFree(s->emb_fact_id);
    cudaFree(s->facts_d);
    cudaFree(s->user_count_d);
    cudaFree(s->inv_freq_d);
    cudaFree(s->ctrl);
    cudaFree(s->scores);
    cudaFree(s->tickets);
    cudaFree(s->tc_gmax);
    cudaFree(s->tc_sel);
    cudaFree(s->tc_cand_scores);
    cudaFree(s->tc_cand_rows);
    cudaFree(s->tc_tickets);
    cudaFree(s->tc_next_best);
    cudaFree(s->tc_kth);
    cudaFree(s->tc_redo);
    cudaFree(s->tc_scores_out);
    cudaFree(s->tc_fix_counts);
    cudaFree(s->tc_fix_keys);
    cudaFree(s->tc_fix_tickets);
    cudaFree(s->tc_n_fixups);
    cudaFree(s->tc_error);
    cudaFree(s->tc_hist);
    cudaFree(s->tc_emit);
    cudaFree(s->tc_raw);
    cudaFree(s->tc_exact);
    cudaFree(s->tc_list_stats);
    cudaFree(s->tiles);
    cudaFree(s->cc_slots);
    cudaFree(s->cc_arena);
    cudaFree(s->cc_counters);
    cudaFree(s->graph);
    cudaFree(s->graph_rows_d);
    cudaFree(s->graph_users_d);
    cudaFree(s->removed_bits_d);
    cudaFree(s->graph_topk);
    cudaFree(s->append_pairs);
    cudaFree(s->dev_stage);
    if (s->host_stage) cudaFreeHost(s->host_stage);
    if (s->serve_stream) cudaStreamDestroy(s->serve_stream);
    if (s->last_done) cudaEventDestroy(s->last_done);
    cudaGetLastError();
  }
  delete s;
  return MS_OK;
}

// tier 1: k_pre / v are device buffers appended to the HBM arena; tier 2: host buffers copied into the pinned host arena
static ms_status add_facts_tier(memstore_t* s, int32_t user, int64_t n, const void* embs, const void* k_pre, const void* v,
                                const int32_t* n_tokens, int32_t* out_first_id, ms_stream stream, int tier) {
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  const memstore_config& c = s->cfg;
  if (user < 0 || user >= c.n_users) return fail(s, MS_ERR_INVALID_ARG, "user %d out of range", user);
  if (n < 0 || (n > 0 && (!embs || !n_tokens))) return fail(s, MS_ERR_INVALID_ARG, "null embeddings or lengths");
  s->store_changed = true;
  if (n == 0) {
    if (out_first_id) *out_first_id = (int32_t)s->n_facts;
    return MS_OK;
  }
  int64_t T = 0;
  for (int64_t i = 0; i < n; ++i) {
    if (n_tokens[i] < 0) return fail(s, MS_ERR_INVALID_ARG, "negative token count");
    T += n_tokens[i];
  }
  if (T > 0 && (!k_pre || !v)) return fail(s, MS_ERR_INVALID_ARG, "null K/V for %lld tokens", (long long)T);
  if (((uintptr_t)embs & 15) || (tier == 1 && (((uintptr_t)k_pre & 15) || ((uintptr_t)v & 15))))
    return fail(s, MS_ERR_INVALID_ARG, "device buffers must be 16-byte aligned");
  if (s->user_count[user] + n > c.max_facts_per_user)
    return fail(s, MS_ERR_CAPACITY, "user %d segment full (%lld + %lld > %lld)", user, (long long)s->user_count[user],
                (long long)n, (long long)c.max_facts_per_user);
  if (tier == 1 && s->kv_tokens_used + T > c.max_kv_tokens)
    return fail(s, MS_ERR_CAPACITY, "K/V arena full (%lld + %lld > %lld tokens)", (long long)s->kv_tokens_used,
                (long long)T, (long long)c.max_kv_tokens);
  if (tier == 2 && s->host_tokens_used + T > c.max_host_kv_tokens)
    return fail(s, MS_ERR_CAPACITY, "host K/V arena full (%lld + %lld > %lld tokens)", (long long)s->host_tokens_used,
                (long long)T, (long long)c.max_host_kv_tokens);
  DeviceGuard g(c.device);
  cudaStream_t st = (cudaStream_t)stream;
  const int64_t slot0 = s->user_count[user];
  const int64_t row0 = (int64_t)user * c.max_facts_per_user + slot0;
  const size_t esz = emb_elem_size(c.emb_dtype);

  std::vector<FactRec> recs(n);
  std::vector<int32_t> ids(n);
  int64_t off = tier == 1 ? s->kv_tokens_used : s->host_tokens_used;
  int64_t resident = 0;
  int32_t max_len = s->max_fact_len;
  for (int64_t i = 0; i < n; ++i) {
    recs[i] = FactRec{(int32_t)off, n_tokens[i], user, n_tokens[i] > 0 ? tier : 0};
    ids[i] = (int32_t)(s->n_facts + i);
    off += n_tokens[i];
    resident += n_tokens[i] > 0;
    if (n_tokens[i] > max_len) max_len = n_tokens[i];
  }
  const int32_t new_count = (int32_t)(slot0 + n);
  MS_CUDA(s, cudaMemcpyAsync((char*)s->emb + (size_t)row0 * c.emb_dim * esz, embs, (size_t)n * c.emb_dim * esz,
                             cudaMemcpyDeviceToDevice, st));
  // the three small host arrays are pageable: cudaMemcpyAsync stages them before returning
  MS_CUDA(s, cudaMemcpyAsync(s->facts_d + s->n_facts, recs.data(), (size_t)n * sizeof(FactRec), cudaMemcpyHostToDevice, st));
  MS_CUDA(s, cudaMemcpyAsync(s->emb_fact_id + row0, ids.data(), (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  MS_CUDA(s, cudaMemcpyAsync(s->user_count_d + user, &new_count, sizeof(int32_t), cudaMemcpyHostToDevice, st));
  if (T > 0 && tier == 2) {
    // host tier: plain host copies, layer by layer, into the pinned arena (visible to later kernels as is)
    const size_t row = (size_t)c.n_kv_heads * c.head_dim * sizeof(__nv_bfloat16);
    for (int l = 0; l < c.n_layers; ++l) {
      const size_t dst = ((size_t)l * c.max_host_kv_tokens + s->host_tokens_used) * row;
      memcpy((char*)s->k_host + dst, (const char*)k_pre + (size_t)l * T * row, (size_t)T * row);
      memcpy((char*)s->v_host + dst, (const char*)v + (size_t)l * T * row, (size_t)T * row);
    }
  } else if (T > 0) {
    const int64_t row_vec = (int64_t)c.n_kv_heads * c.head_dim * 2 / 16;
    const int64_t src_vec = T * row_vec;
    int gx = (int)std::min<int64_t>((src_vec + 255) / 256, 4 * s->sm_count);
    dim3 grid(gx > 0 ? gx : 1, c.n_layers, 2);
    arena_append_kernel<<<grid, 256, 0, st>>>((const uint4*)k_pre, (const uint4*)v, (uint4*)s->k_arena, (uint4*)s->v_arena,
                                              src_vec, c.max_kv_tokens * row_vec, s->kv_tokens_used * row_vec);
    MS_CUDA(s, cudaGetLastError());
    s->kernels_launched++;
  }
  if (out_first_id) *out_first_id = (int32_t)s->n_facts;
  s->id_runs.push_back(memstore::IdRun{(int32_t)s->n_facts, (int32_t)n, user, slot0});
  s->user_count[user] += n;
  if (s->user_count[user] > s->max_user_count) s->max_user_count = s->user_count[user];
  s->n_facts += n;
  s->n_resident += resident;
  if (tier == 1) s->kv_tokens_used += T; else s->host_tokens_used += T;
  s->max_fact_len = max_len;
  return MS_OK;
}

ms_status memstore_add_facts(memstore_t* s, int32_t user, int64_t n, const void* embs, const void* k_pre, const void* v,
                             const int32_t* n_tokens, int32_t* out_first_id, ms_stream stream) {
  Range range("memstore_add_facts");
  return add_facts_tier(s, user, n, embs, k_pre, v, n_tokens, out_first_id, stream, 1);
}

ms_status memstore_add_facts_host(memstore_t* s, int32_t user, int64_t n, const void* embs, const void* k_pre_host,
                                  const void* v_host, const int32_t* n_tokens, int32_t* out_first_id, ms_stream stream) {
  Range range("memstore_add_facts_host");
  if (s && s->cfg.max_host_kv_tokens == 0) return fail(s, MS_ERR_INVALID_ARG, "store was created without a host K/V arena");
  return add_facts_tier(s, user, n, embs, k_pre_host, v_host, n_tokens, out_first_id, stream, 2);
}

ms_status memstore_add_fact(memstore_t* s, int32_t user, const void* emb, const void* k_pre, const void* v,
                            int32_t n_tokens, int32_t* out_fact_id, ms_stream stream) {
  return memstore_add_facts(s, user, 1, emb, k_pre, v, &n_tokens, out_fact_id, stream);
}

ms_status memstore_set_prefix(memstore_t* s, const void* k_pre, const void* v, int32_t n_tokens, ms_stream stream) {
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  const memstore_config& c = s->cfg;
  if (n_tokens < 0) return fail(s, MS_ERR_INVALID_ARG, "negative token count");
  s->store_changed = true;
  if (n_tokens == 0) {
    s->prefix_len = 0;
    return MS_OK;
  }
  if (!k_pre || !v) return fail(s, MS_ERR_INVALID_ARG, "null K/V for the prefix");
  if (((uintptr_t)k_pre & 15) || ((uintptr_t)v & 15)) return fail(s, MS_ERR_INVALID_ARG, "device buffers must be 16-byte aligned");
  if (!s->k_arena || s->kv_tokens_used + n_tokens > c.max_kv_tokens)
    return fail(s, MS_ERR_CAPACITY, "K/V arena full (%lld + %d > %lld tokens)", (long long)s->kv_tokens_used, n_tokens,
                (long long)c.max_kv_tokens);
  DeviceGuard g(c.device);
  cudaStream_t st = (cudaStream_t)stream;
  const int64_t row_vec = (int64_t)c.n_kv_heads * c.head_dim * 2 / 16;
  const int64_t src_vec = (int64_t)n_tokens * row_vec;
  const int gx = (int)std::min<int64_t>((src_vec + 255) / 256, 4 * s->sm_count);
  dim3 grid(gx > 0 ? gx : 1, c.n_layers, 2);
  arena_append_kernel<<<grid, 256, 0, st>>>((const uint4*)k_pre, (const uint4*)v, (uint4*)s->k_arena, (uint4*)s->v_arena, src_vec,
                                            c.max_kv_tokens * row_vec, s->kv_tokens_used * row_vec);
  MS_CUDA(s, cudaGetLastError());
  s->kernels_launched++;
  s->prefix_off = s->kv_tokens_used;
  s->prefix_len = n_tokens;
  s->kv_tokens_used += n_tokens;
  s->prefix_tokens_total += n_tokens;
  return MS_OK;
}

// memstore_retrieve; return_rows != 0 (graph building) writes rows of the user's segment instead of fact ids
static ms_status retrieve_impl(memstore_t* s, const void* queries, const int32_t* query_users, int32_t nq, int32_t k, int32_t* out_ids,
                               float* out_scores, ms_stream stream, int return_rows) {
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  const memstore_config& c = s->cfg;
  if (nq < 0 || k < 1 || k > kTopkMaxK) return fail(s, MS_ERR_INVALID_ARG, "nq=%d k=%d (1 <= k <= %d)", nq, k, kTopkMaxK);
  if (nq == 0) return MS_OK;
  if (!queries || !out_ids) return fail(s, MS_ERR_INVALID_ARG, "null queries or out_ids");
  if ((uintptr_t)queries & 15) return fail(s, MS_ERR_INVALID_ARG, "queries must be 16-byte aligned");
  DeviceGuard g(c.device);
  cudaStream_t st = (cudaStream_t)stream;
  const bool tc = tc_path_applies(s, query_users, nq, k, query_users ? s->max_user_count : s->user_count[0]);
  ms_status rc = MS_OK;
  if (!tc) {  // grow the score scratch (first call, or a larger batch than ever before)
    rc = ensure_scores(s, nq);
    if (rc != MS_OK) return rc;
  }
  rc = order_after_last(s, st);
  if (rc != MS_OK) return rc;

  RetrieveParams p = retrieve_params(s, queries, query_users, nq, k, s->scores, out_ids, out_scores);
  p.return_rows = return_rows;

  const int64_t n_max = query_users ? s->max_user_count : s->user_count[0];
  if (tc) {
    rc = retrieve_tensor_core(s, p, n_max, st);
    if (rc != MS_OK) return rc;
    s->retrieve_calls++;
    return mark_last(s, st);
  }
  // enough CTAs to fill the GPU, at least one row per warp
  const int64_t target_ctas = std::max<int64_t>(1, (int64_t)s->sm_count * 8 / nq);
  int64_t rows_per_cta = std::max<int64_t>(kScoreWarps, (std::max<int64_t>(n_max, 1) + target_ctas - 1) / target_ctas);
  rows_per_cta = (rows_per_cta + kScoreWarps - 1) / kScoreWarps * kScoreWarps;
  dim3 grid((unsigned)((std::max<int64_t>(n_max, 1) + rows_per_cta - 1) / rows_per_cta), (unsigned)nq);
  if (n_max <= kFusedMaxRows) {
    // small segments: scoring and top-k in one launch
    const int keys_cap = (int)std::max<int64_t>(n_max, 1);
    const size_t smem = (size_t)keys_cap * sizeof(uint32_t);
    const int n_host = query_users ? -1 : (int)n_max;
    MS_CUDA(s, ensure_fused_smem(c.device, smem));
    if (c.emb_dtype == MS_DTYPE_F16)
      launch_score_topk<__half, false>(s->sm_count, nq, n_max, p, s->tickets, keys_cap, n_host, nullptr, smem, st);
    else
      launch_score_topk<float, false>(s->sm_count, nq, n_max, p, s->tickets, keys_cap, n_host, nullptr, smem, st);
    MS_CUDA(s, cudaGetLastError());
    s->kernels_launched++;
  } else {
    const size_t smem = (size_t)c.emb_dim * sizeof(float);
    if (c.emb_dtype == MS_DTYPE_F16)
      score_rows_kernel<__half><<<grid, kScoreThreads, smem, st>>>(p, (int)rows_per_cta);
    else
      score_rows_kernel<float><<<grid, kScoreThreads, smem, st>>>(p, (int)rows_per_cta);
    MS_CUDA(s, cudaGetLastError());
    topk_kernel<<<nq, kTopkThreads, 0, st>>>(p);
    MS_CUDA(s, cudaGetLastError());
    s->kernels_launched += 2;
  }
  s->retrieve_calls++;
  return mark_last(s, st);
}

ms_status memstore_retrieve(memstore_t* s, const void* queries, const int32_t* query_users, int32_t nq, int32_t k,
                            int32_t* out_ids, float* out_scores, ms_stream stream) {
  Range range("memstore_retrieve");
  return retrieve_impl(s, queries, query_users, nq, k, out_ids, out_scores, stream, 0);
}

// ---- graph index -------------------------------------------------------------------------------------------------
// (Re)allocates the graph array for `cap_rows` rows per user; every user's graph is empty afterwards.
static ms_status graph_alloc(memstore* s, int64_t cap_rows, int32_t degree) {
  const memstore_config& c = s->cfg;
  MS_CUDA(s, cudaDeviceSynchronize());
  cudaFree(s->graph);
  s->graph = nullptr;
  s->graph_cap_rows = 0;
  s->graph_deg = 0;
  s->graph_rows.assign(c.n_users, 0);
  if (!s->graph_rows_d) MS_CUDA(s, cudaMalloc(&s->graph_rows_d, (size_t)c.n_users * sizeof(int32_t)));
  if (!s->graph_users_d) MS_CUDA(s, cudaMalloc(&s->graph_users_d, 256 * sizeof(int32_t)));
  MS_CUDA(s, cudaMemset(s->graph_rows_d, 0, (size_t)c.n_users * sizeof(int32_t)));
  if (cap_rows > 0) MS_CUDA(s, cudaMalloc(&s->graph, (size_t)c.n_users * cap_rows * degree * sizeof(int32_t)));
  s->graph_cap_rows = cap_rows;
  s->graph_deg = degree;
  return MS_OK;
}

static ms_status graph_publish_rows(memstore* s, cudaStream_t st) {
  std::vector<int32_t> rows(s->graph_rows.begin(), s->graph_rows.end());
  MS_CUDA(s, cudaMemcpyAsync(s->graph_rows_d, rows.data(), rows.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  return MS_OK;
}

static ms_status graph_check_degree(memstore* s, int32_t degree) {
  if (degree < 1 || degree > kAnnMaxCand || degree + 1 > kTcMaxK)
    return fail(s, MS_ERR_INVALID_ARG, "degree %d out of range (1..%d)", degree, kTcMaxK - 1);
  return MS_OK;
}

// The batch of equal user numbers that accompanies a batch of one user's rows used as queries (multi-user stores only).
static const int32_t* graph_batch_users(memstore* s, int32_t user, int n, cudaStream_t st) {
  if (s->cfg.n_users == 1) return nullptr;
  std::vector<int32_t> u(n, user);
  if (cudaMemcpyAsync(s->graph_users_d, u.data(), (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice, st) != cudaSuccess) return nullptr;
  return s->graph_users_d;
}

// Rows [row0, row1) of `user` get their exact lists (rows of the segment as queries through the exact retrieval kernels)
// and, when n_old > 0, the rows below n_old are offered the new rows that list them.
static ms_status graph_link_rows(memstore* s, int32_t user, int64_t row0, int64_t row1, int64_t n_old, ms_stream stream) {
  const memstore_config& c = s->cfg;
  cudaStream_t st = (cudaStream_t)stream;
  const int deg = s->graph_deg, k1 = deg + 1;
  const int batch = std::max(1, std::min(kAppendMaxOffers, kAppendMaxPairs / deg));
  const size_t row_bytes = (size_t)c.emb_dim * emb_elem_size(c.emb_dtype);
  const char* seg = (const char*)s->emb + (size_t)user * c.max_facts_per_user * row_bytes;
  int32_t* graph_u = s->graph + (size_t)user * s->graph_cap_rows * deg;
  RetrieveParams p{};
  p.emb = seg;
  p.queries = seg;  // the rows are scored against one another
  p.emb_dim = c.emb_dim;
  int* n_pairs = s->append_pairs ? reinterpret_cast<int*>(s->append_pairs + kAppendMaxPairs) : nullptr;
  for (int64_t r0 = row0; r0 < row1; r0 += batch) {
    const int nb = (int)std::min<int64_t>(batch, row1 - r0);
    const int32_t* users = graph_batch_users(s, user, nb, st);
    if (c.n_users > 1 && !users) return fail(s, MS_ERR_CUDA, "staging the user numbers of a graph batch");
    ms_status rc = retrieve_impl(s, seg + (size_t)r0 * row_bytes, users, nb, k1, s->graph_topk, nullptr, stream, 1);
    if (rc != MS_OK) return rc;
    graph_rows_kernel<<<(nb + 7) / 8, dim3(32, 8), 0, st>>>(s->graph_topk, k1, graph_u, deg, r0, nb);
    s->kernels_launched++;
    if (n_old > 0) {
      append_pairs_kernel<<<1, 1024, 0, st>>>(graph_u, deg, r0, nb, n_old, s->append_pairs, n_pairs);
      const int grid = kAppendMaxPairs / kAppendWarps;
      if (c.emb_dtype == MS_DTYPE_F16)
        append_update_kernel<__half><<<grid, kAppendWarps * 32, 0, st>>>(p, graph_u, deg, row1, s->append_pairs, n_pairs);
      else
        append_update_kernel<float><<<grid, kAppendWarps * 32, 0, st>>>(p, graph_u, deg, row1, s->append_pairs, n_pairs);
      s->kernels_launched += 2;
    }
    if (cudaGetLastError() != cudaSuccess) return fail(s, MS_ERR_CUDA, "graph kernels failed to launch");
  }
  return MS_OK;
}

static ms_status graph_scratch(memstore* s) {
  const size_t need = (size_t)kAppendMaxOffers * (s->graph_deg + 1);
  if (s->graph_topk_cap < need) {
    MS_CUDA(s, cudaDeviceSynchronize());
    cudaFree(s->graph_topk);
    s->graph_topk = nullptr;
    s->graph_topk_cap = 0;
    MS_CUDA(s, cudaMalloc(&s->graph_topk, need * sizeof(int32_t)));
    s->graph_topk_cap = need;
  }
  if (!s->append_pairs) MS_CUDA(s, cudaMalloc(&s->append_pairs, (size_t)kAppendMaxPairs * sizeof(unsigned long long) + 16));
  return MS_OK;
}

static void graph_drop(memstore* s) {  // a half-made graph must not be searched
  s->graph_rows.assign(s->cfg.n_users, 0);
  if (s->graph_rows_d) cudaMemset(s->graph_rows_d, 0, (size_t)s->cfg.n_users * sizeof(int32_t));
  s->graph_deg = 0;
}

ms_status memstore_build_graph(memstore_t* s, int32_t degree, ms_stream stream) {
  Range range("memstore_build_graph");
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  ms_status rc = graph_check_degree(s, degree);
  if (rc != MS_OK) return rc;
  const memstore_config& c = s->cfg;
  DeviceGuard g(c.device);
  // a single segment gets exactly the rows it has (memstore_graph_append grows the array); several segments share one
  // array with room for every segment's capacity
  const int64_t cap = c.n_users == 1 ? s->user_count[0] : c.max_facts_per_user;
  rc = graph_alloc(s, cap, degree);
  if (rc != MS_OK) return rc;
  rc = graph_scratch(s);
  for (int32_t u = 0; rc == MS_OK && u < c.n_users; ++u) {
    rc = graph_link_rows(s, u, 0, s->user_count[u], 0, stream);
    if (rc == MS_OK) s->graph_rows[u] = s->user_count[u];
  }
  if (rc == MS_OK) rc = graph_publish_rows(s, (cudaStream_t)stream);
  if (rc != MS_OK) graph_drop(s);
  return rc;
}

ms_status memstore_graph_append(memstore_t* s, ms_stream stream) {
  Range range("memstore_graph_append");
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  if (!s->graph_deg) return fail(s, MS_ERR_INVALID_ARG, "no graph to grow: call memstore_build_graph or memstore_set_graph first");
  const memstore_config& c = s->cfg;
  const int deg = s->graph_deg;
  bool any = false;
  for (int32_t u = 0; u < c.n_users; ++u) any = any || s->user_count[u] > s->graph_rows[u];
  if (!any) return MS_OK;
  DeviceGuard g(c.device);
  if (c.n_users == 1 && s->user_count[0] > s->graph_cap_rows) {
    // room for the new rows: the array grows geometrically (to at least 1.5 times its size, at most the segment's
    // capacity), so that a stream of small appends does not reallocate and copy the whole graph each time
    const int64_t n = s->user_count[0], n_old = s->graph_rows[0];
    const int64_t cap = std::min<int64_t>(c.max_facts_per_user, std::max<int64_t>(n, s->graph_cap_rows + s->graph_cap_rows / 2 + 1024));
    MS_CUDA(s, cudaDeviceSynchronize());
    int32_t* grown = nullptr;
    MS_CUDA(s, cudaMalloc(&grown, (size_t)cap * deg * sizeof(int32_t)));
    if (n_old) {
      const cudaError_t e = cudaMemcpy(grown, s->graph, (size_t)n_old * deg * sizeof(int32_t), cudaMemcpyDeviceToDevice);
      if (e != cudaSuccess) {  // the old graph stays in place and usable
        cudaFree(grown);
        return fail(s, MS_ERR_CUDA, "copying the graph into its larger array: %s", cudaGetErrorString(e));
      }
    }
    cudaFree(s->graph);
    s->graph = grown;
    s->graph_cap_rows = cap;
  }
  ms_status rc = graph_scratch(s);
  for (int32_t u = 0; rc == MS_OK && u < c.n_users; ++u) {
    const int64_t n_old = s->graph_rows[u], n = s->user_count[u];
    if (n == n_old) continue;
    rc = graph_link_rows(s, u, n_old, n, n_old, stream);
    if (rc == MS_OK) s->graph_rows[u] = n;
  }
  if (rc == MS_OK) rc = graph_publish_rows(s, (cudaStream_t)stream);
  if (rc != MS_OK) graph_drop(s);
  return rc;
}

ms_status memstore_set_graph_user(memstore_t* s, int32_t user, const int32_t* graph, int64_t n_rows, int32_t degree, ms_stream stream) {
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  const memstore_config& c = s->cfg;
  if (user < 0 || user >= c.n_users) return fail(s, MS_ERR_INVALID_ARG, "user %d out of range", user);
  ms_status rc = graph_check_degree(s, degree);
  if (rc != MS_OK) return rc;
  if (n_rows < 0 || n_rows > s->user_count[user] || (n_rows > 0 && !graph))
    return fail(s, MS_ERR_INVALID_ARG, "graph of %lld rows for a segment of %lld", (long long)n_rows, (long long)s->user_count[user]);
  DeviceGuard g(c.device);
  const int64_t want_cap = c.n_users == 1 ? n_rows : c.max_facts_per_user;
  if (!s->graph_deg || s->graph_deg != degree || want_cap > s->graph_cap_rows || c.n_users == 1) {
    // another degree (or the first graph of this store): every segment's graph starts over
    rc = graph_alloc(s, want_cap, degree);
    if (rc != MS_OK) return rc;
  }
  if (n_rows > 0)
    MS_CUDA(s, cudaMemcpyAsync(s->graph + (size_t)user * s->graph_cap_rows * degree, graph, (size_t)n_rows * degree * sizeof(int32_t),
                               cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  s->graph_rows[user] = n_rows;
  return graph_publish_rows(s, (cudaStream_t)stream);
}

ms_status memstore_set_graph(memstore_t* s, const int32_t* graph, int64_t n_rows, int32_t degree, ms_stream stream) {
  return memstore_set_graph_user(s, 0, graph, n_rows, degree, stream);
}

ms_status memstore_get_graph_user(memstore_t* s, int32_t user, int32_t* out, int64_t out_capacity, int64_t* out_rows, int32_t* out_degree,
                                  ms_stream stream) {
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  if (user < 0 || user >= s->cfg.n_users) return fail(s, MS_ERR_INVALID_ARG, "user %d out of range", user);
  const int64_t rows = s->graph_deg && !s->graph_rows.empty() ? s->graph_rows[user] : 0;
  if (out_rows) *out_rows = rows;
  if (out_degree) *out_degree = s->graph_deg;
  if (!out) return MS_OK;
  const int64_t need = rows * s->graph_deg;
  if (out_capacity < need) return fail(s, MS_ERR_CAPACITY, "graph holds %lld entries, the buffer %lld", (long long)need, (long long)out_capacity);
  DeviceGuard g(s->cfg.device);
  if (need)
    MS_CUDA(s, cudaMemcpyAsync(out, s->graph + (size_t)user * s->graph_cap_rows * s->graph_deg, (size_t)need * sizeof(int32_t),
                               cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return MS_OK;
}

ms_status memstore_get_graph(memstore_t* s, int32_t* out, int64_t out_capacity, int64_t* out_rows, int32_t* out_degree, ms_stream stream) {
  return memstore_get_graph_user(s, 0, out, out_capacity, out_rows, out_degree, stream);
}

ms_status memstore_retrieve_ann_users(memstore_t* s, const void* queries, const int32_t* query_users, int32_t nq, int32_t k,
                                      const ms_ann_params* params, int32_t* out_ids, float* out_scores, int32_t* out_counters,
                                      ms_stream stream) {
  Range range("memstore_retrieve_ann");
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  const memstore_config& c = s->cfg;
  if (!s->graph_deg) return fail(s, MS_ERR_INVALID_ARG, "no graph: call memstore_build_graph or memstore_set_graph first");
  const int beam = params && params->beam > 0 ? params->beam : 64;
  const int parents = params && params->parents > 0 ? params->parents : std::max(1, std::min(8, kAnnMaxCand / s->graph_deg));
  const int n_entry = params && params->n_entry > 0 ? params->n_entry : 64;
  const int max_iters = params && params->max_iters > 0 ? params->max_iters : 32;
  if (nq < 0 || k < 1 || k > kAnnMaxList || beam > kAnnMaxList)
    return fail(s, MS_ERR_INVALID_ARG, "nq=%d k=%d beam=%d (k, beam <= %d)", nq, k, beam, kAnnMaxList);
  if (parents > 32 || (int64_t)parents * s->graph_deg > kAnnMaxCand || n_entry > kAnnMaxCand)
    return fail(s, MS_ERR_INVALID_ARG, "parents=%d (<= 32, parents * degree <= %d), n_entry=%d (<= %d)", parents, kAnnMaxCand, n_entry, kAnnMaxCand);
  if (nq == 0) return MS_OK;
  if (!queries || !out_ids) return fail(s, MS_ERR_INVALID_ARG, "null queries or out_ids");
  // visited table: a power of two that the rows that can ever be scored fill to 80 % at most (a search that
  // converges, as searches do, scores a fraction of that bound)
  const int64_t max_scored = (int64_t)n_entry + (int64_t)max_iters * parents * s->graph_deg;
  const int64_t want_slots = max_scored + max_scored / 4;
  uint32_t slots = 1024;
  while ((int64_t)slots < want_slots && slots < (1u << 20)) slots <<= 1;
  const size_t smem = (size_t)c.emb_dim * sizeof(float) + (size_t)slots * sizeof(uint32_t);
  if ((int64_t)slots < want_slots || smem > 200 * 1024)
    return fail(s, MS_ERR_UNSUPPORTED, "max_iters * parents * degree = %lld rows do not fit the visited table in shared memory",
                (long long)max_scored);
  DeviceGuard g(c.device);
  cudaStream_t st = (cudaStream_t)stream;
  AnnParams p{};
  p.emb = s->emb;
  p.graph = s->graph;
  p.queries = queries;
  p.query_users = query_users;
  p.graph_rows = s->graph_rows_d;
  p.emb_fact_id = c.n_users == 1 ? nullptr : s->emb_fact_id;
  p.seg_capacity = c.max_facts_per_user;
  p.graph_cap_rows = s->graph_cap_rows;
  p.n_users = c.n_users;
  p.emb_dim = c.emb_dim;
  p.deg = s->graph_deg;
  p.k = k;
  p.list_len = std::max(beam, k);
  p.parents = parents;
  p.n_entry = n_entry;
  p.max_iters = max_iters;
  p.table_mask = slots - 1;
  p.out_ids = out_ids;
  p.out_scores = out_scores;
  p.out_counters = out_counters;
  p.removed_bits = s->removed_bits_d;
  ms_status rc = order_after_last(s, st);
  if (rc != MS_OK) return rc;
  // one cluster per query; its size spreads a small batch over the GPU (a single SM cannot pull the candidate rows
  // fast enough), shrinking as the batch grows so that all clusters still run at once
  int cluster = 8;
  while (cluster > 1 && (int64_t)nq * cluster > s->sm_count) cluster >>= 1;
  const void* fn = c.emb_dtype == MS_DTYPE_F16 ? (const void*)ann_search_kernel<__half> : (const void*)ann_search_kernel<float>;
  MS_CUDA(s, cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
  cudaLaunchConfig_t lc{};
  cudaLaunchAttribute attr[1];
  lc.blockDim = dim3(kAnnThreads);
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = 1;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  for (;; cluster >>= 1) {  // a cluster that the device cannot co-schedule with this much shared memory: halve it
    attr[0].val.clusterDim.x = (unsigned)cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.gridDim = dim3((unsigned)nq * (unsigned)cluster);
    int n_clusters = 0;
    if (cluster == 1 || (cudaOccupancyMaxActiveClusters(&n_clusters, fn, &lc) == cudaSuccess && n_clusters > 0)) break;
    cudaGetLastError();
  }
  void* args[] = {(void*)&p};
  MS_CUDA(s, cudaLaunchKernelExC(&lc, fn, args));
  s->kernels_launched++;
  s->retrieve_calls++;
  return mark_last(s, st);
}

ms_status memstore_retrieve_ann(memstore_t* s, const void* queries, int32_t nq, int32_t k, const ms_ann_params* params,
                                int32_t* out_ids, float* out_scores, int32_t* out_counters, ms_stream stream) {
  return memstore_retrieve_ann_users(s, queries, nullptr, nq, k, params, out_ids, out_scores, out_counters, stream);
}

// ---- removing a fact ---------------------------------------------------------------------------------------------
ms_status memstore_remove_fact(memstore_t* s, int32_t fact_id, ms_stream stream) {
  Range range("memstore_remove_fact");
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  const memstore_config& c = s->cfg;
  if (fact_id < 0 || fact_id >= s->n_facts) return fail(s, MS_ERR_INVALID_ARG, "fact id %d out of range (0..%lld)", fact_id, (long long)s->n_facts - 1);
  s->store_changed = true;
  // the embedding row of the id: ids are dense in insertion order, each add call put a run of them into one segment
  size_t lo = 0, hi = s->id_runs.size();
  while (lo + 1 < hi) {
    const size_t mid = (lo + hi) / 2;
    if (s->id_runs[mid].first_id <= fact_id) lo = mid; else hi = mid;
  }
  const memstore::IdRun& run = s->id_runs[lo];
  const int64_t grow = (int64_t)run.user * c.max_facts_per_user + run.slot0 + (fact_id - run.first_id);
  const int64_t n_rows = (int64_t)c.n_users * c.max_facts_per_user;
  DeviceGuard g(c.device);
  cudaStream_t st = (cudaStream_t)stream;
  if (!s->removed_bits_d) {
    const size_t words = (size_t)((n_rows + 31) / 32);
    MS_CUDA(s, cudaDeviceSynchronize());
    MS_CUDA(s, cudaMalloc(&s->removed_bits_d, words * sizeof(uint32_t)));
    MS_CUDA(s, cudaMemset(s->removed_bits_d, 0, words * sizeof(uint32_t)));
    s->removed_bits.assign(words, 0u);
  }
  uint32_t& word = s->removed_bits[(size_t)(grow >> 5)];
  if ((word >> (grow & 31)) & 1u) return fail(s, MS_ERR_INVALID_ARG, "fact %d has been removed already", fact_id);
  ms_status rc = order_after_last(s, st);
  if (rc != MS_OK) return rc;
  word |= 1u << (grow & 31);
  // retrieval stops returning the row; injection refuses the id like a fact without K/V (its arena tokens are not reclaimed)
  MS_CUDA(s, cudaMemcpyAsync(s->removed_bits_d + (grow >> 5), &word, sizeof(uint32_t), cudaMemcpyHostToDevice, st));
  const int32_t zero = 0;
  MS_CUDA(s, cudaMemcpyAsync(reinterpret_cast<char*>(s->facts_d + fact_id) + offsetof(FactRec, resident), &zero, sizeof(int32_t),
                             cudaMemcpyHostToDevice, st));
  s->n_removed++;
  s->cc_epoch++;  // composed segments that contain the fact must not be served any more
  return mark_last(s, st);
}

// ---- memstore_retrieve_static: the allocation-free variant of retrieve ---------------------------------------
// Scratch of the variant: fp32 scores first, then one ticket per query.  A file-scope device array: every GPU
// that loads this library carries it until the process ends.  In HOST code the name below is only a stand-in for
// the symbol, not a device address; the address each device gives it comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_retrieve_static_scratch[MEMSTORE_STATIC_SCRATCH_BYTES];

namespace {
// Device address of g_retrieve_static_scratch on `device` (which must be current), looked up once per device.
cudaError_t static_scratch_address(int device, unsigned char** out) {
  static std::mutex mu;
  static unsigned char* addr[64] = {nullptr};
  if (device < 0 || device >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  if (!addr[device]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_retrieve_static_scratch);
    if (e != cudaSuccess) return e;
    addr[device] = static_cast<unsigned char*>(p);
  }
  *out = addr[device];
  return cudaSuccess;
}
}  // namespace

ms_status memstore_retrieve_static(memstore_t* s, const void* queries, const int32_t* query_users, int32_t nq, int32_t k,
                                   int32_t* out_ids, float* out_scores, ms_stream stream) {
  Range range("memstore_retrieve_static");
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  const memstore_config& c = s->cfg;
  if (nq < 0 || k < 1 || k > kTopkMaxK) return fail(s, MS_ERR_INVALID_ARG, "nq=%d k=%d (1 <= k <= %d)", nq, k, kTopkMaxK);
  if (nq == 0) return MS_OK;
  if (!queries || !out_ids) return fail(s, MS_ERR_INVALID_ARG, "null queries or out_ids");
  if ((uintptr_t)queries & 15) return fail(s, MS_ERR_INVALID_ARG, "queries must be 16-byte aligned");
  if (nq > MEMSTORE_STATIC_MAX_QUERIES || (int64_t)nq * c.max_facts_per_user > MEMSTORE_STATIC_MAX_SCORES)
    return fail(s, MS_ERR_CAPACITY,
                "static scratch holds %d queries and %d scores: nq=%d x max_facts_per_user=%lld does not fit "
                "(use memstore_retrieve)",
                MEMSTORE_STATIC_MAX_QUERIES, MEMSTORE_STATIC_MAX_SCORES, nq, (long long)c.max_facts_per_user);
  DeviceGuard g(c.device);
  cudaStream_t st = (cudaStream_t)stream;
  unsigned char* scratch = nullptr;
  MS_CUDA(s, static_scratch_address(c.device, &scratch));
  float* scores = reinterpret_cast<float*>(scratch);
  uint32_t* tickets = reinterpret_cast<uint32_t*>(scratch + (size_t)MEMSTORE_STATIC_MAX_SCORES * sizeof(float));
  ms_status rc = order_after_last(s, st);
  if (rc != MS_OK) return rc;
  // the tickets must start at zero whatever an earlier call (of any store) left behind
  MS_CUDA(s, cudaMemsetAsync(tickets, 0, (size_t)nq * sizeof(uint32_t), st));

  RetrieveParams p = retrieve_params(s, queries, query_users, nq, k, scores, out_ids, out_scores);

  const int64_t n_max = query_users ? s->max_user_count : s->user_count[0];
  const int64_t target_ctas = std::max<int64_t>(1, (int64_t)s->sm_count * 8 / nq);
  int64_t rows_per_cta = std::max<int64_t>(kScoreWarps, (std::max<int64_t>(n_max, 1) + target_ctas - 1) / target_ctas);
  rows_per_cta = (rows_per_cta + kScoreWarps - 1) / kScoreWarps * kScoreWarps;
  dim3 grid((unsigned)((std::max<int64_t>(n_max, 1) + rows_per_cta - 1) / rows_per_cta), (unsigned)nq);
  if (n_max <= kFusedMaxRows) {
    const int keys_cap = (int)std::max<int64_t>(n_max, 1);
    const size_t smem = (size_t)keys_cap * sizeof(uint32_t);
    const int n_host = query_users ? -1 : (int)n_max;
    MS_CUDA(s, ensure_fused_smem(c.device, smem));  // a function attribute, not an allocation
    if (c.emb_dtype == MS_DTYPE_F16)
      launch_score_topk<__half, false>(s->sm_count, nq, n_max, p, tickets, keys_cap, n_host, nullptr, smem, st);
    else
      launch_score_topk<float, false>(s->sm_count, nq, n_max, p, tickets, keys_cap, n_host, nullptr, smem, st);
    MS_CUDA(s, cudaGetLastError());
    s->kernels_launched++;
  } else {
    const size_t smem = (size_t)c.emb_dim * sizeof(float);
    if (c.emb_dtype == MS_DTYPE_F16)
      score_rows_kernel<__half><<<grid, kScoreThreads, smem, st>>>(p, (int)rows_per_cta);
    else
      score_rows_kernel<float><<<grid, kScoreThreads, smem, st>>>(p, (int)rows_per_cta);
    MS_CUDA(s, cudaGetLastError());
    topk_kernel<<<nq, kTopkThreads, 0, st>>>(p);
    MS_CUDA(s, cudaGetLastError());
    s->kernels_launched += 2;
  }
  s->retrieve_calls++;
  return mark_last(s, st);
}

namespace {

// Validation, scratch sizing and parameter block shared by memstore_inject and memstore_retrieve_inject.
// the staged (bulk-async) copy kernel serves the plain parameterisation only (whole-head rotation, bf16 cache)
bool copy_uses_tma(const memstore* s, const ms_paged_cache* cache) {
  const memstore_config& c = s->cfg;
  const int row_bytes = c.n_kv_heads * c.head_dim * 2;
  return s->tma_path && !s->cc_slots && row_bytes <= kTmaAreaBytes && c.rotary_dim == c.head_dim && cache->dtype == MS_CACHE_BF16;
}

ms_status prepare_inject(memstore* s, const int32_t* fact_ids, int32_t nreq, int32_t k, const int32_t* start_pos,
                         const int32_t* block_tables, int32_t max_blocks, const ms_paged_cache* cache, int32_t* out_n_tokens,
                         int32_t* out_status, int64_t* out_slot_mapping, int64_t slot_stride, uint32_t flags, cudaStream_t st,
                         InjectParams* out, int64_t* out_tiles_needed) {
  const memstore_config& c = s->cfg;
  if (flags & ~(uint32_t)(MS_INJECT_REVERSE | MS_INJECT_PREFIX)) return fail(s, MS_ERR_INVALID_ARG, "unknown flags 0x%x", flags);
  const bool with_prefix = (flags & MS_INJECT_PREFIX) != 0;
  if (with_prefix && s->prefix_len == 0) return fail(s, MS_ERR_INVALID_ARG, "MS_INJECT_PREFIX without a stored prefix (memstore_set_prefix)");
  // the planning code keeps one entry per fact, plus one for the prefix, in shared memory
  if (nreq < 0 || k < 0 || k + (with_prefix ? 1 : 0) > kPlanMaxK)
    return fail(s, MS_ERR_INVALID_ARG, "nreq=%d k=%d (k <= %d, one less with a prefix)", nreq, k, kPlanMaxK);
  if (!start_pos || !block_tables || !cache || (k > 0 && !fact_ids) || max_blocks < 0)
    return fail(s, MS_ERR_INVALID_ARG, "null request arrays");
  if (!cache->k_base || !cache->v_base || cache->block_size <= 0 || cache->num_blocks <= 0)
    return fail(s, MS_ERR_INVALID_ARG, "bad cache description");
  if (((uintptr_t)cache->k_base & 15) || ((uintptr_t)cache->v_base & 15) || (cache->layer_stride % 8) ||
      (cache->block_stride % 8) || (cache->token_stride % 8) || (cache->head_stride % 8) || cache->layer_stride < 0 ||
      cache->block_stride < 0 || cache->token_stride < 0 || cache->head_stride < 0)
    return fail(s, MS_ERR_INVALID_ARG, "cache bases must be 16-byte aligned and strides non-negative multiples of 8");
  if (cache->dtype != MS_CACHE_BF16 && cache->dtype != MS_CACHE_FP8_E4M3) return fail(s, MS_ERR_INVALID_ARG, "unknown cache dtype %d", cache->dtype);
  if (cache->dtype == MS_CACHE_FP8_E4M3 && !(cache->k_scale > 0.f && cache->v_scale > 0.f && std::isfinite(cache->k_scale) && std::isfinite(cache->v_scale)))
    return fail(s, MS_ERR_INVALID_ARG, "an 8-bit cache needs finite positive k_scale and v_scale");
  if (out_slot_mapping && slot_stride < 0) return fail(s, MS_ERR_INVALID_ARG, "negative slot_stride");
  if ((c.max_kv_tokens == 0 || !s->k_arena) && !s->k_host) return fail(s, MS_ERR_INVALID_ARG, "store has no K/V arena");

  // upper bound on tiles: each request composes at most k * (longest fact) tokens, plus a ragged first tile
  const int64_t max_m = (int64_t)k * s->max_fact_len + (with_prefix ? s->prefix_len : 0);
  if (max_m > 0x3fffffff) return fail(s, MS_ERR_UNSUPPORTED, "a request could compose %lld tokens (k x longest fact): more than 2^30", (long long)max_m);
  const int64_t tiles_per_req = (max_m + kTileTokens - 1) / kTileTokens + 1;
  const int64_t tiles_needed = std::max<int64_t>(1, tiles_per_req * nreq);
  {
    const ms_status rc = ensure_tiles(s, tiles_needed);
    if (rc != MS_OK) return rc;
  }
  *out_tiles_needed = tiles_needed;

  InjectParams p{};
  p.facts = s->facts_d;
  p.n_facts = (int32_t)s->n_facts;
  p.k_arena = s->k_arena;
  p.v_arena = s->v_arena;
  p.arena_tokens = c.max_kv_tokens;
  p.k_host = s->k_host_dev;
  p.v_host = s->v_host_dev;
  p.host_tokens = c.max_host_kv_tokens;
  p.inv_freq = s->inv_freq_d;
  p.n_layers = c.n_layers;
  p.n_heads = c.n_kv_heads;
  p.head_dim = c.head_dim;
  p.rope_style = c.rope_style;
  p.rotary_dim = c.rotary_dim;
  p.max_position = (int32_t)c.max_position;
  p.fact_ids = fact_ids;
  p.nreq = nreq;
  p.k = k;
  p.prefix_src = with_prefix ? (int32_t)s->prefix_off : 0;
  p.prefix_len = with_prefix ? s->prefix_len : 0;
  p.start_pos = start_pos;
  p.block_tables = block_tables;
  p.max_blocks = max_blocks;
  p.flags = flags;
  p.k_cache = (__nv_bfloat16*)cache->k_base;
  p.v_cache = (__nv_bfloat16*)cache->v_base;
  p.layer_stride = cache->layer_stride;
  p.block_stride = cache->block_stride;
  p.token_stride = cache->token_stride;
  p.head_stride = cache->head_stride;
  p.num_blocks = cache->num_blocks;
  p.block_size = cache->block_size;
  p.k_scale = cache->dtype == MS_CACHE_FP8_E4M3 ? cache->k_scale : 1.0f;
  p.v_scale = cache->dtype == MS_CACHE_FP8_E4M3 ? cache->v_scale : 1.0f;
  // reciprocals rounded once to fp32 (a double quotient rounds to the same float as the exact one)
  p.k_recip = (float)(1.0 / (double)p.k_scale);
  p.v_recip = (float)(1.0 / (double)p.v_scale);
  p.out_n_tokens = out_n_tokens;
  p.out_status = out_status;
  p.out_slot_mapping = out_slot_mapping;
  p.slot_stride = slot_stride;
  p.tiles = s->tiles;
  p.tiles_capacity = s->tiles_capacity;
  p.ctrl = s->ctrl;
  p.spin_limit = s->test_spin_limit;
  p.mute_producer = s->test_mute_producers;
  p.host_flag = nreq == 1 ? s->serve_flag_dev : nullptr;  // (set by memstore_serve_host for the one call it makes)
  p.host_seq = s->serve_seq;
  p.host_flag_in_copy = copy_uses_tma(s, cache) ? 0 : 1;
  if (s->cc_slots) {
    const int64_t cc_tokens = (int64_t)s->cc_n_slots * s->cc_slot_tokens;
    p.cc_slots = s->cc_slots;
    p.cc_k = s->cc_arena;
    p.cc_v = s->cc_arena + (size_t)c.n_layers * cc_tokens * c.n_kv_heads * c.head_dim;
    p.cc_tokens = cc_tokens;
    p.cc_n_slots = s->cc_n_slots;
    p.cc_slot_tokens = s->cc_slot_tokens;
    p.cc_epoch = s->cc_epoch;
    p.cc_call = ++s->cc_call;
    p.cc_fill_all = s->cc_fill_all;
    p.cc_counters = s->cc_counters;
  }

  // layers per work item (bulk-async kernel): the largest power of two that still leaves every CTA about 16 items
  const int row_bytes = c.n_kv_heads * c.head_dim * 2;
  const bool use_tma = copy_uses_tma(s, cache);
  const int resident_ctas = use_tma ? s->sm_count : s->sm_count * s->copy_ctas_per_sm;
  const int64_t est_tiles = std::max<int64_t>(1, ((int64_t)k * (s->max_fact_len + 1) / 2 + p.prefix_len + kTileTokens - 1) / kTileTokens * nreq);
  int lpi = 1;
  while (lpi * 2 <= c.n_layers && c.n_layers % (lpi * 2) == 0 && est_tiles * (c.n_layers / (lpi * 2)) >= 16ll * resident_ctas) lpi *= 2;
  p.layers_per_item = lpi;
  *out = p;
  return MS_OK;
}

// Launches the copy kernel as a programmatic dependent of the kernel that planned the request(s).
// programmatic: launch the copy kernel as a programmatic dependent of the planning kernel before it.  That hides the
// launch latency of a single request (a few microseconds of ≈ 90).  It is not used after planning kernels made of many
// small CTAs (a call with many requests): copy CTAs that were placed on the SMs beside those ran the whole copy kernel
// 1 - 6 % slower (3.36 ms against 3.16 ms for 100 requests of 800 tokens), and such a copy is milliseconds long anyway.
ms_status launch_copy(memstore* s, const InjectParams& p, const ms_paged_cache* cache, int64_t tiles_needed, cudaStream_t st,
                      bool programmatic) {
  const memstore_config& c = s->cfg;
  const int row_bytes = c.n_kv_heads * c.head_dim * 2;
  // the staged kernel serves the plain parameterisation only (whole-head rotation, bf16 cache)
  const bool use_tma = copy_uses_tma(s, cache);
  cudaLaunchConfig_t lc{};
  lc.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = 1;
  if (!programmatic) lc.numAttrs = 0;
  const bool prof = s->prof_before && s->prof_after;
  if (prof) {
    lc.numAttrs = 0;  // an event between the two kernels: no programmatic overlap
    MS_CUDA(s, cudaEventRecord(s->prof_before, st));
  }
  cudaError_t e = cudaSuccess;
  // (measurement aid: the direct kernel may be launched several times in a row on the same plan - its writes are the same
  // every time - as ordinary launches, each after the one before it has ended)
  const int repeats = (prof && !use_tma) ? std::max(1, s->prof_repeats) : 1;
  for (int rep = 0; rep < repeats && e == cudaSuccess; ++rep) {
    if (use_tma) {
      // bulk-async staged kernel: one persistent CTA per SM
      int ts = kTileTokens;
      while (ts > 1 && ts * row_bytes > kTmaAreaBytes) ts >>= 1;
      const int v_rows = cache->head_stride == c.head_dim ? 1 : 0;
      lc.gridDim = dim3((unsigned)s->sm_count);
      lc.blockDim = dim3(kTmaThreads);
      lc.dynamicSmemBytes = kTmaSmemBytes;
      if (c.rope_style == MS_ROPE_HALF_SPLIT)
        e = cudaLaunchKernelEx(&lc, inject_copy_tma_kernel<0>, p, ts, v_rows);
      else
        e = cudaLaunchKernelEx(&lc, inject_copy_tma_kernel<1>, p, ts, v_rows);
    } else {
      // direct kernel: one CTA per (tile, layer, row part).  The ids are on the device, so the host sizes the grid
      // from the mean length of the resident facts (plus a ragged tile per request and 3 %); the kernel's
      // grid-stride loop makes any grid correct, and the worst case (every fact of maximal length) bounds it.
      const int units = c.n_kv_heads * (c.head_dim / 16);
      const double mean_len = s->n_resident > 0 ? (double)(s->kv_tokens_used - s->prefix_tokens_total + s->host_tokens_used) / (double)s->n_resident : 0.0;
      int64_t est_tiles_grid = (int64_t)((((double)p.k * mean_len + p.prefix_len) / kTileTokens + 2.0) * p.nreq * 1.03) + 1;
      est_tiles_grid = std::min(est_tiles_grid, tiles_needed);
      const int64_t items = std::max<int64_t>(1, est_tiles_grid) * c.n_layers;
      if (items > 0x7fffffff) return fail(s, MS_ERR_UNSUPPORTED, "request batch too large");
      lc.gridDim = dim3((unsigned)items, (unsigned)((units + kUnitsPerPart - 1) / kUnitsPerPart));
      lc.blockDim = dim3(kCopyThreads);
      lc.dynamicSmemBytes = 0;
      // 8-bit caches: a scale whose significand is all ones, or one so extreme that it or its reciprocal is not a normal
      // number, takes the kernel variant that divides with the hardware routine (see div_by_scale)
      auto awkward = [](float sc, float rc) {
        uint32_t u;
        memcpy(&u, &sc, 4);
        return (u & 0x7fffffu) == 0x7fffffu || !std::isnormal(rc) || !std::isnormal(sc);
      };
      const int fp8 = cache->dtype != MS_CACHE_FP8_E4M3 ? 0 : (awkward(p.k_scale, p.k_recip) || awkward(p.v_scale, p.v_recip)) ? 2 : 1;
      if (c.rope_style == MS_ROPE_HALF_SPLIT)
        e = fp8 == 0 ? cudaLaunchKernelEx(&lc, inject_copy_kernel<0, 0>, p)
            : fp8 == 1 ? cudaLaunchKernelEx(&lc, inject_copy_kernel<0, 1>, p) : cudaLaunchKernelEx(&lc, inject_copy_kernel<0, 2>, p);
      else
        e = fp8 == 0 ? cudaLaunchKernelEx(&lc, inject_copy_kernel<1, 0>, p)
            : fp8 == 1 ? cudaLaunchKernelEx(&lc, inject_copy_kernel<1, 1>, p) : cudaLaunchKernelEx(&lc, inject_copy_kernel<1, 2>, p);
    }
  }
  if (e != cudaSuccess) {
    // (the planning kernel has left the control block clean: nothing to undo)
    return fail(s, MS_ERR_CUDA, "copy kernel launch: %s", cudaGetErrorString(e));
  }
  if (prof) MS_CUDA(s, cudaEventRecord(s->prof_after, st));
  s->kernels_launched += repeats;
  s->inject_calls++;
  return MS_OK;
}

}  // namespace

ms_status memstore_inject(memstore_t* s, const int32_t* fact_ids, int32_t nreq, int32_t k, const int32_t* start_pos,
                          const int32_t* block_tables, int32_t max_blocks, const ms_paged_cache* cache,
                          int32_t* out_n_tokens, int32_t* out_status, int64_t* out_slot_mapping, int64_t slot_stride,
                          uint32_t flags, ms_stream stream) {
  Range range("memstore_inject");
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  if (nreq == 0) return MS_OK;
  DeviceGuard g(s->cfg.device);
  cudaStream_t st = (cudaStream_t)stream;
  InjectParams p;
  int64_t tiles_needed = 0;
  ms_status rc = prepare_inject(s, fact_ids, nreq, k, start_pos, block_tables, max_blocks, cache, out_n_tokens, out_status,
                                out_slot_mapping, slot_stride, flags, st, &p, &tiles_needed);
  if (rc != MS_OK) return rc;
  rc = order_after_last(s, st);
  if (rc != MS_OK) return rc;
  {
    // a programmatic dependent of what precedes it (see launch_score_topk_threads): placed on the SMs while the
    // previous call's copy kernel drains; the kernel waits for that grid before it does anything
    cudaLaunchConfig_t lc{};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.gridDim = dim3((unsigned)nreq);
    const bool wide = nreq <= s->sm_count;  // every planning CTA has an SM to itself
    // one long request (and no composition cache, whose bookkeeping one CTA does): several CTAs share its per-token work,
    // one per 1024 tokens (one pass of a CTA) the request is expected to hold
    const double mean_len = s->n_resident > 0 ? (double)(s->kv_tokens_used - s->prefix_tokens_total + s->host_tokens_used) / (double)s->n_resident : 0.0;
    const int64_t est_tokens = (int64_t)((double)k * mean_len) + p.prefix_len;
    const int parts = (nreq == 1 && !s->cc_slots) ? (int)std::max<int64_t>(1, std::min<int64_t>(kPlanMaxParts, est_tokens / 1024)) : 1;
    lc.gridDim = dim3((unsigned)nreq, (unsigned)parts);
    lc.blockDim = dim3(wide ? kPlanThreadsWide : kPlanThreads);
    lc.stream = st;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (wide)
      MS_CUDA(s, cudaLaunchKernelEx(&lc, inject_plan_kernel<kPlanThreadsWide>, p));
    else
      MS_CUDA(s, cudaLaunchKernelEx(&lc, inject_plan_kernel<kPlanThreads>, p));
  }
  s->kernels_launched++;
  rc = launch_copy(s, p, cache, tiles_needed, st, /*programmatic=*/nreq <= s->sm_count);
  if (rc != MS_OK) return rc;
  return mark_last(s, st);
}

ms_status memstore_retrieve_inject(memstore_t* s, const void* queries, const int32_t* query_users, int32_t nq, int32_t k,
                                   const int32_t* start_pos, const int32_t* block_tables, int32_t max_blocks,
                                   const ms_paged_cache* cache, int32_t* out_ids, float* out_scores, int32_t* out_n_tokens,
                                   int32_t* out_status, int64_t* out_slot_mapping, int64_t slot_stride, uint32_t flags,
                                   ms_stream stream) {
  Range range("memstore_retrieve_inject");
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  const memstore_config& c = s->cfg;
  if (nq < 0 || k < 1 || k > kTopkMaxK) return fail(s, MS_ERR_INVALID_ARG, "nq=%d k=%d (1 <= k <= %d)", nq, k, kTopkMaxK);
  if (nq == 0) return MS_OK;
  if (!queries || !out_ids) return fail(s, MS_ERR_INVALID_ARG, "null queries or out_ids");
  if ((uintptr_t)queries & 15) return fail(s, MS_ERR_INVALID_ARG, "queries must be 16-byte aligned");
  // MS_INPUTS_STABLE only matters to the one-launch retrieval + planning kernel below; every other route orders itself
  // after the preceding work of the stream as an ordinary launch does
  // (not right after the store itself was changed on the stream: the kernels read its tables)
  const int early = ((flags & MS_INPUTS_STABLE) && !s->store_changed) ? 1 : 0;
  flags &= ~(uint32_t)MS_INPUTS_STABLE;
  if (flags & MS_RETRIEVE_ANN) {
    ms_status rc = memstore_retrieve_ann_users(s, queries, query_users, nq, k, nullptr, out_ids, out_scores, nullptr, stream);
    if (rc != MS_OK) return rc;
    return memstore_inject(s, out_ids, nq, k, start_pos, block_tables, max_blocks, cache, out_n_tokens, out_status,
                           out_slot_mapping, slot_stride, flags & ~(uint32_t)MS_RETRIEVE_ANN, stream);
  }
  const int64_t n_max = query_users ? s->max_user_count : s->user_count[0];
  if (n_max > kFusedMaxRows || nq > s->scores_nq || ((flags & MS_INJECT_PREFIX) && k + 1 > kTopkMaxK)) {
    // large segments (or a first call that still has to size its scratch): the two calls one after the other
    ms_status rc = memstore_retrieve(s, queries, query_users, nq, k, out_ids, out_scores, stream);
    if (rc != MS_OK) return rc;
    return memstore_inject(s, out_ids, nq, k, start_pos, block_tables, max_blocks, cache, out_n_tokens, out_status,
                           out_slot_mapping, slot_stride, flags, stream);
  }
  DeviceGuard g(c.device);
  cudaStream_t st = (cudaStream_t)stream;
  InjectParams ip;
  int64_t tiles_needed = 0;
  ms_status rc = prepare_inject(s, out_ids, nq, k, start_pos, block_tables, max_blocks, cache, out_n_tokens, out_status,
                                out_slot_mapping, slot_stride, flags, st, &ip, &tiles_needed);
  if (rc != MS_OK) return rc;
  rc = order_after_last(s, st);
  if (rc != MS_OK) return rc;

  RetrieveParams p = retrieve_params(s, queries, query_users, nq, k, s->scores, out_ids, out_scores);
  const int keys_cap = (int)std::max<int64_t>(n_max, 1);
  const size_t smem = (size_t)keys_cap * sizeof(uint32_t);
  const int n_host = query_users ? -1 : (int)n_max;
  MS_CUDA(s, ensure_fused_smem(c.device, smem));
  if (c.emb_dtype == MS_DTYPE_F16)
    launch_score_topk<__half, true>(s->sm_count, nq, n_max, p, s->tickets, keys_cap, n_host, &ip, smem, st, early);
  else
    launch_score_topk<float, true>(s->sm_count, nq, n_max, p, s->tickets, keys_cap, n_host, &ip, smem, st, early);
  MS_CUDA(s, cudaGetLastError());
  s->kernels_launched++;
  s->retrieve_calls++;
  rc = launch_copy(s, ip, cache, tiles_needed, st, /*programmatic=*/nq <= kFusedFewQueries);
  if (rc != MS_OK) return rc;
  s->store_changed = false;  // this call's kernels waited for everything before them (the plan kernel always does before it ends)
  return mark_last(s, st);
}

ms_status memstore_serve_host(memstore_t* s, const void* query, int32_t user, int32_t k, int32_t start_pos,
                              const int32_t* block_table, int32_t max_blocks, const ms_paged_cache* cache, uint32_t flags,
                              int32_t* out_ids, int32_t* out_n_tokens, int32_t* out_status, ms_stream stream) {
  Range range("memstore_serve_host");
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  const memstore_config& c = s->cfg;
  if (!query || !block_table || !out_ids || max_blocks <= 0 || k < 1 || k > kTopkMaxK)
    return fail(s, MS_ERR_INVALID_ARG, "memstore_serve_host: null buffer, max_blocks=%d or k=%d out of range", max_blocks, k);
  if (user < 0 || user >= c.n_users) return fail(s, MS_ERR_INVALID_ARG, "user %d out of range", user);
  if (start_pos < 0) return fail(s, MS_ERR_INVALID_ARG, "negative start position %d", start_pos);
  DeviceGuard g(c.device);
  cudaStream_t st = (cudaStream_t)stream;
  // layout of both staging buffers: [query | start_pos, user, pad, pad | block table] then [ids | n_tokens, status]
  size_t q_bytes, in_bytes, out_bytes;
  serve_host_layout(c, max_blocks, k, &q_bytes, &in_bytes, &out_bytes);
  {
    const ms_status rc = ensure_stage(s, in_bytes + out_bytes);
    if (rc != MS_OK) return rc;
  }
  unsigned char* h = s->host_stage;
  unsigned char* d = s->dev_stage;
  memcpy(h, query, (size_t)c.emb_dim * emb_elem_size(c.emb_dtype));
  int32_t* hdr = reinterpret_cast<int32_t*>(h + q_bytes);
  hdr[0] = start_pos;
  hdr[1] = user;
  memcpy(h + q_bytes + 16, block_table, (size_t)max_blocks * 4);
  const bool early_return = (flags & MS_SERVE_EARLY_RETURN) != 0;
  flags &= ~(uint32_t)MS_SERVE_EARLY_RETURN;
  if (early_return) {
    // The previous request's planning is over (its call saw the results), so the staging buffer on the device is free
    // although that request's copy kernel may still run: the inputs go up beside it on a stream of their own and the
    // host waits for them here.  They are then complete before this request is launched, which is all the early
    // scoring of MS_INPUTS_STABLE needs: the retrieval runs while the previous copy kernel drains.
    MS_CUDA(s, cudaMemcpyAsync(d, h, in_bytes, cudaMemcpyHostToDevice, s->serve_stream));
    MS_CUDA(s, cudaStreamSynchronize(s->serve_stream));
    flags |= MS_INPUTS_STABLE;
  } else {
    MS_CUDA(s, cudaMemcpyAsync(d, h, in_bytes, cudaMemcpyHostToDevice, st));
  }
  int32_t* d_hdr = reinterpret_cast<int32_t*>(d + q_bytes);
  // The results (k ids, token count, status: a few hundred bytes) are written by the kernels straight into the pinned
  // host buffer through its device address, so that no copy back has to be queued behind the copy kernel.
  void* res_dev = nullptr;
  MS_CUDA(s, cudaHostGetDevicePointer(&res_dev, h + in_bytes, 0));
  int32_t* d_ids = static_cast<int32_t*>(res_dev);
  volatile uint32_t* flag_host = reinterpret_cast<volatile uint32_t*>(h + in_bytes + out_bytes - 16);
  if (early_return) {
    s->serve_seq += 1;
    if (s->serve_seq == 0) s->serve_seq = 1;
    *flag_host = 0;
    s->serve_flag_dev = reinterpret_cast<uint32_t*>(static_cast<unsigned char*>(res_dev) + out_bytes - 16);
  }
  ms_status rc = memstore_retrieve_inject(s, d, c.n_users > 1 ? d_hdr + 1 : nullptr, 1, k, d_hdr,
                                          reinterpret_cast<const int32_t*>(d + q_bytes + 16), max_blocks, cache, d_ids, nullptr,
                                          d_ids + k, d_ids + k + 1, nullptr, 0, flags, stream);
  s->serve_flag_dev = nullptr;
  if (rc != MS_OK) return rc;
  bool seen = false;
  if (early_return) {
    // the planning CTA writes the flag after the results; a launch that failed, or a device that is busy with other
    // work for long, ends the wait and the stream is synchronised as usual
    const auto t0 = std::chrono::steady_clock::now();
    for (uint32_t spins = 1; !seen; ++spins) {
      seen = *flag_host == s->serve_seq;
      if (!seen && (spins & 1023u) == 0 && std::chrono::steady_clock::now() - t0 > std::chrono::milliseconds(200)) break;
    }
    std::atomic_thread_fence(std::memory_order_acquire);
  }
  if (!seen) MS_CUDA(s, cudaStreamSynchronize(st));
  const int32_t* res = reinterpret_cast<const int32_t*>(h + in_bytes);
  memcpy(out_ids, res, (size_t)k * 4);
  if (out_n_tokens) *out_n_tokens = res[k];
  if (out_status) *out_status = res[k + 1];
  return MS_OK;
}

ms_status memstore_stats(memstore_t* s, memstore_stats_t* out) {
  if (!s || !out) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  out->n_facts = s->n_facts;
  out->n_resident_facts = s->n_resident;
  out->n_removed_facts = s->n_removed;
  out->kv_tokens_used = s->kv_tokens_used;
  out->host_kv_tokens_used = s->host_tokens_used;
  out->retrieve_calls = s->retrieve_calls;
  out->inject_calls = s->inject_calls;
  out->kernels_launched = s->kernels_launched;
  out->arena_bytes = (int64_t)memstore_arena_bytes(&s->cfg);
  out->embedding_bytes = (int64_t)s->cfg.n_users * s->cfg.max_facts_per_user * s->cfg.emb_dim * (int64_t)emb_elem_size(s->cfg.emb_dtype);
  out->compose_cache_hits = out->compose_cache_fills = 0;
  out->compose_cache_segments = s->cc_n_slots;
  if (s->cc_counters) {
    DeviceGuard g(s->cfg.device);
    uint32_t cnt[2] = {0, 0};
    MS_CUDA(s, cudaMemcpy(cnt, s->cc_counters, sizeof cnt, cudaMemcpyDeviceToHost));
    out->compose_cache_hits = cnt[0];
    out->compose_cache_fills = cnt[1];
  }
  out->kernel_timeouts = 0;
  out->filter_fixups = 0;
  out->filter_fixup_overflows = 0;
  out->filter_list_queries = out->filter_list_rows = out->filter_list_fallbacks = 0;
  if (s->tc_error) {
    DeviceGuard g(s->cfg.device);
    int flags[2] = {0, 0};
    uint32_t fix = 0;
    MS_CUDA(s, cudaMemcpy(flags, s->tc_error, sizeof flags, cudaMemcpyDeviceToHost));
    MS_CUDA(s, cudaMemcpy(&fix, s->tc_n_fixups, sizeof fix, cudaMemcpyDeviceToHost));
    out->kernel_timeouts = flags[0];
    out->filter_fixup_overflows = flags[1];
    out->filter_fixups = fix;
    unsigned long long ls[3] = {0, 0, 0};
    MS_CUDA(s, cudaMemcpy(ls, s->tc_list_stats, sizeof ls, cudaMemcpyDeviceToHost));
    out->filter_list_queries = (int64_t)ls[0];
    out->filter_list_rows = (int64_t)ls[1];
    out->filter_list_fallbacks = (int64_t)ls[2];
  }
  return MS_OK;
}

ms_status memstore_compose_cache(memstore_t* s, size_t budget_bytes, int32_t max_tokens_per_segment, uint32_t flags) {
  Range range("memstore_compose_cache");
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  const memstore_config& c = s->cfg;
  if (flags & ~(uint32_t)MS_COMPOSE_CACHE_ALL) return fail(s, MS_ERR_INVALID_ARG, "unknown flags 0x%x", flags);
  DeviceGuard g(c.device);
  MS_CUDA(s, cudaDeviceSynchronize());
  cudaFree(s->cc_slots);
  cudaFree(s->cc_arena);
  cudaFree(s->cc_counters);
  s->cc_slots = nullptr;
  s->cc_arena = nullptr;
  s->cc_counters = nullptr;
  s->cc_n_slots = s->cc_slot_tokens = 0;
  if (budget_bytes == 0) return MS_OK;
  if (max_tokens_per_segment <= 0) return fail(s, MS_ERR_INVALID_ARG, "max_tokens_per_segment must be positive");
  const size_t tok_bytes = (size_t)2 * c.n_layers * c.n_kv_heads * c.head_dim * sizeof(__nv_bfloat16);
  const size_t seg_bytes = tok_bytes * (size_t)max_tokens_per_segment;
  const int64_t n_slots = std::min<int64_t>(kCcMaxSlots, (int64_t)(budget_bytes / seg_bytes));
  if (n_slots < 1) return fail(s, MS_ERR_INVALID_ARG, "a budget of %zu bytes holds no segment of %d tokens (%zu bytes)", budget_bytes, max_tokens_per_segment, seg_bytes);
  if (n_slots * max_tokens_per_segment >= (int64_t)kCacheTierBit) return fail(s, MS_ERR_UNSUPPORTED, "composition cache of 2^29 tokens or more");
  if (cudaMalloc(&s->cc_arena, (size_t)n_slots * seg_bytes) != cudaSuccess || cudaMalloc(&s->cc_slots, (size_t)n_slots * sizeof(CcSlot)) != cudaSuccess ||
      cudaMalloc(&s->cc_counters, 2 * sizeof(uint32_t)) != cudaSuccess) {
    cudaGetLastError();
    cudaFree(s->cc_slots);
    cudaFree(s->cc_arena);
    cudaFree(s->cc_counters);
    s->cc_slots = nullptr;
    s->cc_arena = nullptr;
    s->cc_counters = nullptr;
    return fail(s, MS_ERR_OOM, "composition cache of %lld segments", (long long)n_slots);
  }
  MS_CUDA(s, cudaMemset(s->cc_slots, 0, (size_t)n_slots * sizeof(CcSlot)));  // epoch 0: every slot is empty
  MS_CUDA(s, cudaMemset(s->cc_counters, 0, 2 * sizeof(uint32_t)));
  s->cc_n_slots = (int32_t)n_slots;
  s->cc_slot_tokens = max_tokens_per_segment;
  s->cc_fill_all = (flags & MS_COMPOSE_CACHE_ALL) ? 1 : 0;
  s->cc_epoch++;
  return MS_OK;
}

ms_status memstore_reserve(memstore_t* s, int32_t nq, int32_t k, int32_t nreq, int64_t max_tokens_per_request, int32_t max_blocks) {
  Range range("memstore_reserve");
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  const memstore_config& c = s->cfg;
  if (nq < 0 || nreq < 0 || k < 0 || k > kTopkMaxK || max_tokens_per_request < 0 || max_blocks < 0)
    return fail(s, MS_ERR_INVALID_ARG, "memstore_reserve: negative size or k > %d", kTopkMaxK);
  DeviceGuard g(c.device);
  ms_status rc = MS_OK;
  if (nq > 0) {
    rc = ensure_scores(s, nq);
    if (rc != MS_OK) return rc;
    const size_t smem = (size_t)std::min<int64_t>(c.max_facts_per_user, kFusedMaxRows) * sizeof(uint32_t);
    MS_CUDA(s, ensure_fused_smem(c.device, smem));
    // the tensor-core filter path serves long fp16 segments: its scratch as well, when this store can take that path
    if (c.emb_dtype == MS_DTYPE_F16 && c.emb_dim % kGemmKChunk == 0 && c.emb_dim <= kGemmMaxE && c.max_facts_per_user > kFusedMaxRows) {
      rc = tc_prepare(s);
      if (rc != MS_OK) return rc;
    }
  }
  if (nreq > 0) {
    const int64_t tiles_per_req = (max_tokens_per_request + kTileTokens - 1) / kTileTokens + 1;
    rc = ensure_tiles(s, std::max<int64_t>(1, tiles_per_req * nreq));
    if (rc != MS_OK) return rc;
  }
  if (max_blocks > 0 && k > 0) {
    size_t q_bytes, in_bytes, out_bytes;
    serve_host_layout(c, max_blocks, k, &q_bytes, &in_bytes, &out_bytes);
    rc = ensure_stage(s, in_bytes + out_bytes);
    if (rc != MS_OK) return rc;
  }
  return MS_OK;
}

ms_status memstore_test_hooks(memstore_t* s, uint32_t wait_poll_limit, int32_t mute_producers) {
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  s->test_spin_limit = wait_poll_limit;
  s->test_mute_producers = mute_producers ? 1 : 0;
  if (!wait_poll_limit && !mute_producers && s->tc_error) {  // back to normal: forget a time-out that a test provoked
    DeviceGuard g(s->cfg.device);
    MS_CUDA(s, cudaMemset(s->tc_error, 0, sizeof(int)));
  }
  return MS_OK;
}

ms_status memstore_set_profile_repeats(memstore_t* s, int32_t n) {
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  if (n < 1 || n > 1024) return fail(s, MS_ERR_INVALID_ARG, "repeats %d out of range (1..1024)", n);
  s->prof_repeats = n;
  return MS_OK;
}

ms_status memstore_set_profile_events(memstore_t* s, void* before_copy, void* after_copy) {
  if (!s) return MS_ERR_INVALID_ARG;
  std::lock_guard<std::recursive_mutex> lock(s->mu);
  if ((before_copy == nullptr) != (after_copy == nullptr)) return fail(s, MS_ERR_INVALID_ARG, "give both events or neither");
  s->prof_before = (cudaEvent_t)before_copy;
  s->prof_after = (cudaEvent_t)after_copy;
  return MS_OK;
}

const char* memstore_last_error(memstore_t* s) { return s ? s->err.c_str() : "null store"; }

}  // extern "C"
