// A client of the C ABI that knows nothing of Python or of any tensor library: plain CUDA runtime allocations,
// the calls of include/memstore.h, results read back with cudaMemcpy.  Built and run by tests/test_gpu_abi_client.py.
// One fact of 3 tokens is stored, retrieved by a query equal to its embedding and injected at position 0 (where the
// rotation is the identity): the cache must hold the stored keys and values bit for bit, every other slot untouched.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <cstring>
#include <vector>

#include "memstore.h"

#define CHECK(x)                                                  \
  do {                                                            \
    if (!(x)) {                                                   \
      std::printf("FAILED line %d: %s\n", __LINE__, #x);          \
      return 1;                                                   \
    }                                                             \
  } while (0)

int main() {
  const int L = 2, H = 2, D = 16, E = 8, T = 3, bs = 4, nb = 3;
  memstore_config cfg;
  std::memset(&cfg, 0, sizeof cfg);
  cfg.n_layers = L;
  cfg.n_kv_heads = H;
  cfg.head_dim = D;
  cfg.kv_dtype = MS_DTYPE_BF16;
  cfg.emb_dim = E;
  cfg.emb_dtype = MS_DTYPE_F32;
  cfg.rope_theta = 10000.0;
  cfg.max_position = 1 << 20;
  cfg.n_users = 1;
  cfg.max_facts_per_user = 4;
  cfg.max_kv_tokens = 8;
  memstore_t* store = nullptr;
  CHECK(memstore_create(&cfg, &store) == MS_OK && store);

  // two facts: an embedding-only one and one with K/V; bf16 bit patterns counted up so that every element differs
  std::vector<float> emb0(E, 0.f), emb1(E, 0.f);
  emb0[0] = 1.f;
  emb1[1] = 1.f;
  std::vector<uint16_t> k(L * T * H * D), v(L * T * H * D);
  for (size_t i = 0; i < k.size(); ++i) {
    k[i] = (uint16_t)(0x3c00 + i);  // small positive bf16 values
    v[i] = (uint16_t)(0xbc00 + i);  // small negative ones
  }
  float *d_emb0, *d_emb1, *d_q;
  uint16_t *d_k, *d_v, *d_kc, *d_vc;
  int32_t *d_ids, *d_start, *d_table, *d_n, *d_st;
  CHECK(cudaMalloc(&d_emb0, E * 4) == cudaSuccess && cudaMalloc(&d_emb1, E * 4) == cudaSuccess && cudaMalloc(&d_q, E * 4) == cudaSuccess);
  CHECK(cudaMalloc(&d_k, k.size() * 2) == cudaSuccess && cudaMalloc(&d_v, v.size() * 2) == cudaSuccess);
  const size_t cache_elems = (size_t)L * nb * bs * H * D;
  CHECK(cudaMalloc(&d_kc, cache_elems * 2) == cudaSuccess && cudaMalloc(&d_vc, cache_elems * 2) == cudaSuccess);
  CHECK(cudaMalloc(&d_ids, 8) == cudaSuccess && cudaMalloc(&d_start, 4) == cudaSuccess && cudaMalloc(&d_table, 8) == cudaSuccess &&
        cudaMalloc(&d_n, 4) == cudaSuccess && cudaMalloc(&d_st, 4) == cudaSuccess);
  cudaMemcpy(d_emb0, emb0.data(), E * 4, cudaMemcpyHostToDevice);
  cudaMemcpy(d_emb1, emb1.data(), E * 4, cudaMemcpyHostToDevice);
  cudaMemcpy(d_q, emb1.data(), E * 4, cudaMemcpyHostToDevice);
  cudaMemcpy(d_k, k.data(), k.size() * 2, cudaMemcpyHostToDevice);
  cudaMemcpy(d_v, v.data(), v.size() * 2, cudaMemcpyHostToDevice);
  cudaMemset(d_kc, 0x11, cache_elems * 2);
  cudaMemset(d_vc, 0x11, cache_elems * 2);
  const int32_t start = 0, table[2] = {2, 0};
  cudaMemcpy(d_start, &start, 4, cudaMemcpyHostToDevice);
  cudaMemcpy(d_table, table, 8, cudaMemcpyHostToDevice);

  int32_t id0 = -1, id1 = -1;
  CHECK(memstore_add_fact(store, 0, d_emb0, nullptr, nullptr, 0, &id0, nullptr) == MS_OK && id0 == 0);
  CHECK(memstore_add_fact(store, 0, d_emb1, d_k, d_v, T, &id1, nullptr) == MS_OK && id1 == 1);

  ms_paged_cache cache;
  std::memset(&cache, 0, sizeof cache);
  cache.k_base = d_kc;
  cache.v_base = d_vc;
  cache.layer_stride = (int64_t)nb * bs * H * D;
  cache.block_stride = (int64_t)bs * H * D;
  cache.token_stride = (int64_t)H * D;
  cache.head_stride = D;
  cache.num_blocks = nb;
  cache.block_size = bs;
  // the best fact for the query is fact 1; k = 1, so the embedding-only fact 0 is not asked for
  CHECK(memstore_retrieve_inject(store, d_q, nullptr, 1, 1, d_start, d_table, 2, &cache, d_ids, nullptr, d_n, d_st, nullptr, 0, 0,
                                 nullptr) == MS_OK);
  CHECK(cudaDeviceSynchronize() == cudaSuccess);
  int32_t got_id = -9, got_n = -9, got_st = -9;
  cudaMemcpy(&got_id, d_ids, 4, cudaMemcpyDeviceToHost);
  cudaMemcpy(&got_n, d_n, 4, cudaMemcpyDeviceToHost);
  cudaMemcpy(&got_st, d_st, 4, cudaMemcpyDeviceToHost);
  CHECK(got_id == 1 && got_n == T && got_st == 0);

  std::vector<uint16_t> kc(cache_elems), vc(cache_elems);
  cudaMemcpy(kc.data(), d_kc, cache_elems * 2, cudaMemcpyDeviceToHost);
  cudaMemcpy(vc.data(), d_vc, cache_elems * 2, cudaMemcpyDeviceToHost);
  size_t touched = 0;
  for (int l = 0; l < L; ++l)
    for (int t = 0; t < T; ++t) {
      const size_t slot = (size_t)table[t / bs] * bs + t % bs;  // positions 0..2 live in block 2
      for (int e = 0; e < H * D; ++e) {
        const size_t c = ((size_t)l * nb * bs + slot) * H * D + e, s = ((size_t)l * T + t) * H * D + e;
        CHECK(vc[c] == v[s]);              // values: a bit copy
        if (t == 0) CHECK(kc[c] == k[s]);  // position 0: the rotation is the identity
        ++touched;
      }
    }
  size_t still = 0;
  for (size_t i = 0; i < cache_elems; ++i) still += vc[i] == 0x1111;
  CHECK(still == cache_elems - touched);

  // the same request from host buffers, waited for and with an early return: the same id, token count and status, and
  // (after a synchronise) the same cache
  {
    for (uint32_t flags : {0u, (uint32_t)MS_SERVE_EARLY_RETURN}) {
      int32_t h_id = -9, h_n = -9, h_st = -9;
      CHECK(memstore_serve_host(store, emb1.data(), 0, 1, 0, table, 2, &cache, flags, &h_id, &h_n, &h_st, nullptr) == MS_OK);
      CHECK(h_id == 1 && h_n == T && h_st == 0);
      CHECK(cudaDeviceSynchronize() == cudaSuccess);
      std::vector<uint16_t> vc2(cache_elems);
      cudaMemcpy(vc2.data(), d_vc, cache_elems * 2, cudaMemcpyDeviceToHost);
      CHECK(vc2 == vc);
    }
  }

  memstore_stats_t st;
  CHECK(memstore_stats(store, &st) == MS_OK && st.n_facts == 2 && st.kv_tokens_used == T);
  CHECK(memstore_inject(store, d_ids, 1, 1, d_start, d_table, -1, &cache, nullptr, nullptr, nullptr, 0, 0, nullptr) == MS_ERR_INVALID_ARG);
  CHECK(std::strlen(memstore_last_error(store)) > 0);
  CHECK(memstore_destroy(store) == MS_OK);
  std::printf("abi client ok: %s\n", memstore_version());
  return 0;
}
