/*
 * A plain C client of the library: no Python, no torch, only the C ABI and the CUDA runtime for memory.
 * Stores two prompts that share a prefix, looks a third one up, gathers its matched K/V blocks into a paged cache
 * with the fused call, checks every byte on the host, makes room and stores the third prompt's own blocks.
 * Prints "abi client ok" and returns 0 on success.  Built and run by tests/test_gpu_parity.py (compiled only on a
 * machine without a GPU).
 */
#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "ptstore.h"

#define CHECK(x)                                                                 \
  do {                                                                           \
    int rc__ = (x);                                                              \
    if (rc__ != 0) { fprintf(stderr, "%s failed: %d (line %d)\n", #x, rc__, __LINE__); return 1; } \
  } while (0)

enum { LAYERS = 2, HEADS = 1, DIM = 8, ELEM = 2, BT = 4, POOL = 32, MAXB = 8, CACHE = 24 };

int main(void) {
  const uint64_t chunk = (uint64_t)BT * HEADS * DIM * ELEM, block = 2 * LAYERS * chunk;
  ptstore_config_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.struct_size = (uint32_t)sizeof cfg;
  cfg.num_layers = LAYERS; cfg.num_kv_heads = HEADS; cfg.head_dim = DIM; cfg.elem_bytes = ELEM; cfg.block_tokens = BT;
  cfg.max_requests = 4; cfg.max_batch_blocks = 4 * MAXB;
  cfg.salt = 7; cfg.hbm_blocks = POOL; cfg.table_slots = 64; cfg.device = 0;
  CHECK(cudaSetDevice(0));
  CHECK(cudaMalloc(&cfg.hbm_pool, POOL * block));
  cfg.workspace_bytes = ptstore_workspace_bytes(&cfg);
  if (cfg.workspace_bytes == 0) { fprintf(stderr, "bad geometry\n"); return 1; }
  CHECK(cudaMalloc(&cfg.workspace, cfg.workspace_bytes));
  ptstore_t* st = NULL;
  CHECK(ptstore_create(&cfg, &st, NULL));

  /* paged cache: per layer [2][CACHE][chunk]; host mirror filled with a pattern that names (layer, plane, block, byte) */
  const uint64_t layer_bytes = 2 * CACHE * chunk;
  unsigned char* h_cache = (unsigned char*)malloc(LAYERS * layer_bytes);
  for (uint64_t i = 0; i < LAYERS * layer_bytes; ++i) h_cache[i] = (unsigned char)(i * 131u + (i >> 7));
  void* d_layers[LAYERS];
  for (int l = 0; l < LAYERS; ++l) {
    CHECK(cudaMalloc(&d_layers[l], layer_bytes));
    CHECK(cudaMemcpy(d_layers[l], h_cache + l * layer_bytes, layer_bytes, cudaMemcpyHostToDevice));
  }
  void** d_layer_ptrs;
  CHECK(cudaMalloc((void**)&d_layer_ptrs, sizeof d_layers));
  CHECK(cudaMemcpy(d_layer_ptrs, d_layers, sizeof d_layers, cudaMemcpyHostToDevice));
  ptstore_paged_cache_t pc;
  memset(&pc, 0, sizeof pc);
  pc.layer_base = (void* const*)d_layer_ptrs; pc.kv_stride_bytes = CACHE * chunk; pc.block_stride_bytes = chunk; pc.num_blocks = CACHE;

  /* prompts: a = 5 blocks, b = first 3 blocks of a + 2 other blocks; q = first 4 blocks of a + 2 fresh blocks */
  int32_t tok[3][6 * BT];
  for (int j = 0; j < 5 * BT; ++j) tok[0][j] = 100 + j;
  for (int j = 0; j < 5 * BT; ++j) tok[1][j] = j < 3 * BT ? 100 + j : 500 + j;
  for (int j = 0; j < 6 * BT; ++j) tok[2][j] = j < 4 * BT ? 100 + j : 900 + j;
  int32_t h_tokens[10 * BT];
  memcpy(h_tokens, tok[0], 5 * BT * 4); memcpy(h_tokens + 5 * BT, tok[1], 5 * BT * 4);
  int64_t h_off[3] = {0, 5 * BT, 10 * BT};
  int32_t h_bt[2 * MAXB];
  for (int i = 0; i < 2 * MAXB; ++i) h_bt[i] = -1;
  for (int j = 0; j < 5; ++j) { h_bt[j] = j; h_bt[MAXB + j] = 5 + j; }          /* a from cache blocks 0..4, b from 5..9 */
  int32_t *d_tok, *d_bt, *d_ids, *d_new, *d_matched, *d_nev;
  int64_t* d_off;
  CHECK(cudaMalloc((void**)&d_tok, sizeof h_tokens)); CHECK(cudaMalloc((void**)&d_off, sizeof h_off)); CHECK(cudaMalloc((void**)&d_bt, sizeof h_bt));
  CHECK(cudaMalloc((void**)&d_ids, 2 * MAXB * 4)); CHECK(cudaMalloc((void**)&d_new, 2 * 4)); CHECK(cudaMalloc((void**)&d_matched, 2 * 4));
  CHECK(cudaMalloc((void**)&d_nev, 2 * 4));
  CHECK(cudaMemcpy(d_tok, h_tokens, sizeof h_tokens, cudaMemcpyHostToDevice));
  CHECK(cudaMemcpy(d_off, h_off, sizeof h_off, cudaMemcpyHostToDevice));
  CHECK(cudaMemcpy(d_bt, h_bt, sizeof h_bt, cudaMemcpyHostToDevice));
  CHECK(ptstore_insert(st, d_tok, d_off, 2, MAXB, &pc, d_bt, d_ids, d_new, NULL));
  int32_t ids[2 * MAXB], newb[2];
  CHECK(cudaMemcpy(ids, d_ids, sizeof ids, cudaMemcpyDeviceToHost));
  CHECK(cudaMemcpy(newb, d_new, sizeof newb, cudaMemcpyDeviceToHost));
  /* a creates blocks 0..4; b shares 3 of them and creates 5, 6 */
  if (newb[0] != 5 || newb[1] != 2 || ids[MAXB + 2] != 2 || ids[MAXB + 3] != 5 || ids[MAXB + 4] != 6) { fprintf(stderr, "insert ids wrong\n"); return 1; }

  /* the query matches 4 blocks of a; gather them into cache blocks 20..23 */
  int64_t q_off[2] = {0, 6 * BT};
  int32_t q_bt[MAXB] = {20, 21, 22, 23, 10, 11, -1, -1};
  CHECK(cudaMemcpy(d_tok, tok[2], 6 * BT * 4, cudaMemcpyHostToDevice));
  CHECK(cudaMemcpy(d_off, q_off, sizeof q_off, cudaMemcpyHostToDevice));
  CHECK(cudaMemcpy(d_bt, q_bt, sizeof q_bt, cudaMemcpyHostToDevice));
  CHECK(ptstore_lookup_fetch(st, d_tok, d_off, 1, MAXB, PTSTORE_PIN, &pc, d_bt, d_matched, d_ids, NULL));
  int32_t matched = -1;
  CHECK(cudaMemcpy(&matched, d_matched, 4, cudaMemcpyDeviceToHost));
  if (matched != 4) { fprintf(stderr, "matched %d, expected 4\n", matched); return 1; }
  unsigned char* got = (unsigned char*)malloc(layer_bytes);
  for (int l = 0; l < LAYERS; ++l) {
    CHECK(cudaMemcpy(got, d_layers[l], layer_bytes, cudaMemcpyDeviceToHost));
    for (int s = 0; s < 2; ++s)
      for (int j = 0; j < 4; ++j) {            /* cache block 20 + j must now equal what block j of `a` was stored from: cache block j */
        const unsigned char* want = h_cache + l * layer_bytes + (uint64_t)s * CACHE * chunk + (uint64_t)j * chunk;
        if (memcmp(got + (uint64_t)s * CACHE * chunk + (uint64_t)(20 + j) * chunk, want, chunk) != 0) { fprintf(stderr, "fetched bytes differ\n"); return 1; }
      }
    if (memcmp(got, h_cache + l * layer_bytes, 20 * chunk) != 0) { fprintf(stderr, "untouched cache blocks changed\n"); return 1; }
  }
  /* room for the query's 6 blocks minus what matched, then store them (blocks 10, 11 of the cache hold the new K/V) */
  CHECK(ptstore_reserve(st, 6, 0, d_matched, 1, 0, d_nev, NULL, 0, NULL));
  CHECK(ptstore_insert_after_lookup(st, d_tok, d_off, 1, MAXB, &pc, d_bt, d_ids, d_new, NULL));
  CHECK(ptstore_release(st, d_ids, d_matched, 1, MAXB, NULL));
  CHECK(cudaMemcpy(newb, d_new, 4, cudaMemcpyDeviceToHost));
  uint32_t status = 99;
  CHECK(ptstore_status(st, NULL, &status));
  ptstore_stats_t stats;
  CHECK(ptstore_stats(st, NULL, &stats));
  if (newb[0] != 2 || status != 0 || stats.live_nodes[0] != 9 || stats.blocks_fetched[0] != 4 || ptstore_resumed_inserts(st) != 0) {
    fprintf(stderr, "final state wrong: new %d status %u live %llu fetched %llu\n", newb[0], status, (unsigned long long)stats.live_nodes[0],
            (unsigned long long)stats.blocks_fetched[0]);
    return 1;
  }
  const unsigned long long launched = (unsigned long long)ptstore_launch_count(st);
  CHECK(ptstore_destroy(st));
  printf("abi client ok: %llu kernels launched\n", launched);
  return 0;
}
