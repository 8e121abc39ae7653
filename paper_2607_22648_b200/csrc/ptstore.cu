// Host side of the prefix tensor store library: argument checks, workspace carving, kernel launches.
// Every entry point only enqueues kernels on the caller's stream; nothing here synchronises except
// ptstore_status / ptstore_stats, and nothing allocates device memory.
#include "../../include/ptstore.h"

#include <cstdlib>
#include <cstring>
#include <new>

#include "common.cuh"
#include "lookup.cuh"
#include "copy.cuh"
#include "insert.cuh"
#include "evict.cuh"
#include "promote.cuh"

using namespace pts;

namespace {

constexpr u64 ALIGN = 256;
inline u64 align_up(u64 x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }

struct Layout {            // byte offsets into the workspace
  u64 table[2], m_key, m_parent, m_last, m_freq, m_ref, m_depth, ring[2], ctrl, blocked, sort[2], hist, room, desc, keys, eslot,
      cta_sums, prefix, promo_first, promo_cnt, links, desc_tier, desc_host, total;
  u32 n_tiles;
};

bool geometry_ok(const ptstore_config_t* c) {
  if (!c || c->struct_size != sizeof(ptstore_config_t)) return false;
  if (!c->num_layers || !c->num_kv_heads || !c->head_dim || !c->elem_bytes || !c->block_tokens) return false;
  const u64 chunk = (u64)c->block_tokens * c->num_kv_heads * c->head_dim * c->elem_bytes;
  if (chunk % 16) return false;
  if (c->hbm_blocks == 0) return false;
  if ((u64)c->hbm_blocks + c->host_blocks >= 0x7FFFFFFFull) return false;
  if (c->table_slots <= (u64)c->hbm_blocks + c->host_blocks || c->table_slots >= 0xFFFFFFFFull) return false;
  if (c->max_requests == 0 || c->max_batch_blocks == 0 || c->max_batch_blocks > 0x7FFFFFFFull) return false;
  return true;
}

Layout make_layout(const ptstore_config_t* c) {
  Layout L;
  const u64 N = (u64)c->hbm_blocks + c->host_blocks, M = c->max_batch_blocks;
  u64 o = 0;
  auto take = [&](u64 bytes) { u64 at = o; o = align_up(o + (bytes ? bytes : 1)); return at; };
  L.table[0] = take(c->table_slots * sizeof(Slot));
  L.table[1] = take(c->table_slots * sizeof(Slot));
  L.m_key = take(N * 8); L.m_parent = take(N * 8); L.m_last = take(N * 8);
  L.m_freq = take(N * 4); L.m_ref = take(N * 4); L.m_depth = take(N * 4);
  L.ring[0] = take((u64)c->hbm_blocks * 4); L.ring[1] = take((u64)c->host_blocks * 4);
  L.ctrl = take(sizeof(Ctrl));
  L.blocked = take(N);
  L.sort[0] = take(N * sizeof(Key2)); L.sort[1] = take(N * sizeof(Key2));
  const u64 sort_tile = (u64)SORT_THREADS * sort_steps_for(N);
  L.n_tiles = (u32)((N + sort_tile - 1) / sort_tile);
  L.hist = take((u64)256 * L.n_tiles * 4);
  L.room = take((u64)c->host_blocks * 4);
  L.desc = take((M > N ? M : N) * sizeof(int2));
  L.keys = take(M * 8);
  L.eslot = take(M * 4);
  L.cta_sums = take(((M + INS_THREADS - 1) / INS_THREADS + 1) * 4);
  L.prefix = take(((u64)c->max_requests + 1) * 4);
  L.promo_first = take(N * 4);
  L.promo_cnt = take(N * 4);
  L.links = take(M * sizeof(int2));
  L.desc_tier = take((u64)c->hbm_blocks * sizeof(int2));
  L.desc_host = take((c->host_blocks ? (M < c->host_blocks ? M : (u64)c->host_blocks) : 1) * sizeof(int2));
  L.total = o;
  return L;
}

}  // namespace

struct BulkVariant { int stages, stage_bytes, ctas_per_sm, group, hint; };

struct ptstore {
  ptstore_config_t cfg;
  Layout lay;
  Store st;
  Slot* stash;           // second table-sized buffer used by the in-place rebuild
  unsigned char* blocked;
  Key2* sort_buf[2];
  u32* hist;
  int* room;
  int2* desc;
  u64* keys;
  u32* eslot;
  u32* cta_sums;
  u32* prefix;
  u32* promo_first;
  u32* promo_cnt;
  int2* links;           // fetch: destination list nodes, one per (request, block) entry
  int2* desc_tier;       // demotion: {HBM id, host id} pairs
  int2* desc_host;       // fetch: descriptors of distinct host-tier source blocks
  int host_ctas;         // grid of the copies that run at host-link speed
  cudaStream_t tier_stream;   // side stream of ptstore_evict_async (created on first use)
  cudaEvent_t ev_meta, ev_copy;
  bool tier_ready, tier_pending;
  u64 epoch;
  u64 launches;
  int last_cuda;
  int sms;
  int bulk_smem_set[4];
  int bulk_multi_smem_set;  // dynamic shared memory already granted to the bulk kernel of each mode
  bool has_env_tune;
  BulkVariant env_tune;
};

namespace {

#define PTS_CHECK_LAUNCH(h)                                   \
  do {                                                        \
    cudaError_t e__ = cudaGetLastError();                     \
    (h)->launches += 1;                                       \
    if (e__ != cudaSuccess) { (h)->last_cuda = (int)e__; return PTSTORE_E_CUDA; } \
  } while (0)

inline int grid_for(long long work, int threads, int cap) {
  long long g = (work + threads - 1) / threads;
  if (g < 1) g = 1;
  if (g > cap) g = cap;
  return (int)g;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_batch(const ptstore* h, int R, int max_blocks) {
  if (!h || R < 0 || max_blocks < 1 || max_blocks > 65535) return PTSTORE_E_INVAL;
  if ((u32)R > h->cfg.max_requests || (u64)R * (u64)max_blocks > h->cfg.max_batch_blocks) return PTSTORE_E_LIMIT;
  return PTSTORE_OK;
}

int check_cache(const ptstore* h, const ptstore_paged_cache_t* pc) {
  if (!pc || !pc->layer_base) return PTSTORE_E_INVAL;
  if (pc->kv_stride_bytes % 16 || pc->block_stride_bytes % 16 || pc->block_stride_bytes < h->st.chunk_bytes) return PTSTORE_E_INVAL;
  if (pc->num_blocks == 0) return PTSTORE_E_INVAL;
  return PTSTORE_OK;
}

Paged to_paged(const ptstore_paged_cache_t* pc) {
  Paged p;
  p.layer_base = reinterpret_cast<unsigned char* const*>(pc->layer_base);
  p.kv_stride = pc->kv_stride_bytes;
  p.block_stride = pc->block_stride_bytes;
  p.num_blocks = pc->num_blocks;
  return p;
}

template <int L>
int launch_hash(ptstore* h, const int* tokens, const long long* offsets, int R, int max_blocks, u64* keys, cudaStream_t s) {
  const long long warps = ((long long)R + (32 / L) - 1) / (32 / L);
  const int grid = (int)((warps * 32 + 255) / 256);
  hash_kernel<L><<<grid, 256, 0, s>>>(h->st, tokens, offsets, R, max_blocks, keys);
  PTS_CHECK_LAUNCH(h);
  return PTSTORE_OK;
}
template <int L>
int launch_lookup(ptstore* h, const int* tokens, const long long* offsets, int R, int max_blocks, u32 flags, int* matched,
                  int* ids, cudaStream_t s) {
  const long long warps = ((long long)R + (32 / L) - 1) / (32 / L);
  const int grid = (int)((warps * 32 + 255) / 256);
  lookup_kernel<L><<<grid, 256, 0, s>>>(h->st, tokens, offsets, R, max_blocks, flags, h->epoch, matched, ids);
  PTS_CHECK_LAUNCH(h);
  return PTSTORE_OK;
}

// Lanes per request.  Many requests: narrow sub-warps (fewer blocks hashed and probed past the first miss,
// 32/L requests per warp).  Few long requests: a whole warp per request (fewer serial chunks).
// Measured on the 16,384 x 64-block lookup stress: L=8 33 us, L=16 37 us, L=32 63 us per call.
// few long requests: content hashes by one thread per block, then one warp per request chains and probes
bool split_path(const ptstore* h, int R, int max_blocks) {
  const u32 forced = (h->cfg.flags >> 8) & 0xFFu;
  return forced == 0 && R < 1024 && max_blocks > 32;
}

int launch_content(ptstore* h, const int* tokens, const long long* offsets, int R, int max_blocks, u64* out, cudaStream_t s) {
  content_kernel<<<grid_for((long long)R * max_blocks, 256, h->sms * 8), 256, 0, s>>>(h->st, tokens, offsets, R, max_blocks, out);
  PTS_CHECK_LAUNCH(h);
  return PTSTORE_OK;
}

int launch_hash_split(ptstore* h, const int* tokens, const long long* offsets, int R, int max_blocks, u64* keys, cudaStream_t s) {
  int rc = launch_content(h, tokens, offsets, R, max_blocks, keys, s);
  if (rc) return rc;
  chain_kernel<<<(R + 3) / 4, 128, 0, s>>>(h->st, keys, offsets, R, max_blocks, keys);       // in place
  PTS_CHECK_LAUNCH(h);
  return PTSTORE_OK;
}

int lanes_for(const ptstore* h, int R, int max_blocks) {
  const u32 forced = (h->cfg.flags >> 8) & 0xFFu;
  if (forced == 4 || forced == 8 || forced == 16 || forced == 32) return (int)forced;
  if (max_blocks <= 8 || R >= 4096) return 8;
  if (max_blocks <= 16 || R >= 1024) return 16;
  return 32;
}

// ---- copy engine dispatch -----------------------------------------------------------------------------------
// index = PTSTORE_COPY_VARIANT field of the flags
const BulkVariant kBulkVariants[] = {
    {0, 0, 1, 1, 0},       // 0: default, sized by auto_bulk() from the chunk size
    {8, 8192, 3, 1, 0},    // 1
    {3, 32768, 1, 1, 0},   // 2
    {4, 16384, 3, 1, 0},   // 3
    {8, 16384, 1, 1, 0},   // 4
    {12, 16384, 1, 1, 0},  // 5
    {4, 32768, 1, 1, 0},   // 6
    {6, 32768, 1, 1, 0},   // 7
    {6, 16384, 1, 2, 0},   // 8: a CTA takes whole 32 KiB chunks
    {6, 16384, 1, 1, 1},   // 9: evict-first L2 hints
    {3, 65536, 1, 1, 0},   // 10
    {24, 8192, 1, 1, 0},   // 11
};
constexpr int kNumBulkVariants = (int)(sizeof(kBulkVariants) / sizeof(kBulkVariants[0]));

// PTSTORE_BULK_TUNE="stages,stage_bytes,ctas_per_sm,group,hint" overrides the variant table (tuning aid)
bool env_bulk_tune(BulkVariant* v) {
  const char* e = std::getenv("PTSTORE_BULK_TUNE");
  if (!e) return false;
  int a[5] = {0, 0, 0, 1, 0};
  int n = 0;
  const char* p = e;
  while (*p && n < 5) {
    a[n++] = std::atoi(p);
    while (*p && *p != ',') ++p;
    if (*p == ',') ++p;
  }
  if (n < 3 || a[0] < 2 || a[0] > BULK_MAX_STAGES || a[1] < 16 || a[1] % 16 || (long long)a[0] * a[1] > 227 * 1024 || a[2] < 1 || a[3] < 1) return false;
  *v = {a[0], a[1], a[2], a[3], a[4] ? 1 : 0};
  return true;
}

// Default ring, from measurements on B200 (read+write GB/s of the fetch / insert copies on the bench workload):
//   32 KiB chunks: 3 x 32 KiB x 1 CTA per SM 6.65 / 6.46 TB/s (deeper rings and more CTAs lose 3-7 %: few bytes in flight win)
//   16 KiB chunks: 3 x 16 KiB x 2 CTAs       6.54 / 6.25       (1 CTA: 5.80 / 5.37 - one issuing thread per SM is too slow)
//    8 KiB chunks: 3 x  8 KiB x 3 CTAs       6.47 / 6.21       (9 x 8 KiB x 1 CTA: 5.43 / 4.61)
//    4 KiB chunks: 5 x  4 KiB x 4 CTAs       6.48 / 5.69
// i.e. about 64 KiB of loads in flight per SM, spread over enough issuing threads that none has less than ~1 us per piece.
BulkVariant auto_bulk(u64 chunk_bytes) {
  const int stage = (int)(chunk_bytes < 32768 ? chunk_bytes : 32768);
  const int ctas = stage >= 32768 ? 1 : stage >= 16384 ? 2 : stage >= 8192 ? 3 : 4;
  const int stages = stage >= 8192 ? 3 : 5;
  return {stages, stage, ctas, 1, 0};
}

template <int MODE>
int launch_bulk(ptstore* h, const Paged& pc, cudaStream_t s, const BulkVariant& v, int ctas_per_sm) {
  const int smem = v.stages * v.stage_bytes;
  if (smem > h->bulk_smem_set[MODE]) {
    if (cudaFuncSetAttribute(copy_bulk_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
      h->last_cuda = (int)cudaGetLastError();
      return PTSTORE_E_CUDA;
    }
    h->bulk_smem_set[MODE] = smem;
  }
  BulkTune t = {v.stages, v.stage_bytes, v.group, v.hint};
  copy_bulk_kernel<MODE><<<h->sms * ctas_per_sm, 32, smem, s>>>(h->st, pc, h->desc, &h->st.ctrl->n_pairs, t);
  PTS_CHECK_LAUNCH(h);
  return PTSTORE_OK;
}

// multi-destination fetch: dynamic dealing of `group`-piece units (default: a quarter of a source block)
int launch_bulk_multi(ptstore* h, const Paged& pc, cudaStream_t s, BulkVariant v, int ctas_per_sm) {
  const int smem = v.stages * v.stage_bytes;
  if (smem > h->bulk_multi_smem_set) {
    if (cudaFuncSetAttribute(copy_bulk_multi_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
      h->last_cuda = (int)cudaGetLastError();
      return PTSTORE_E_CUDA;
    }
    h->bulk_multi_smem_set = smem;
  }
  const u32 ppc = (u32)((h->st.chunk_bytes + v.stage_bytes - 1) / v.stage_bytes);
  const u32 per_pair = 2u * h->st.layers * ppc;
  int group = v.group > 1 ? v.group : (int)(per_pair >= 4 ? per_pair / 4 : per_pair);
  BulkTune t = {v.stages, v.stage_bytes, group, 0};
  copy_bulk_multi_kernel<<<h->sms * ctas_per_sm, 32, smem, s>>>(h->st, pc, h->desc, &h->st.ctrl->n_pairs, &h->st.ctrl->work_counter, t);
  PTS_CHECK_LAUNCH(h);
  return PTSTORE_OK;
}

template <int MODE>
int launch_copy(ptstore* h, const Paged& pc, bool host_side_possible, cudaStream_t s, const int2* desc = nullptr,
                const u32* n_pairs = nullptr, int grid = 0) {
  if (!desc) { desc = h->desc; n_pairs = &h->st.ctrl->n_pairs; }
  if (grid > 0) {       // host-link copies: fixed small grid, vector engine
    copy_vector_kernel<MODE, 256, 8><<<grid, 256, 0, s>>>(h->st, pc, desc, n_pairs);
    PTS_CHECK_LAUNCH(h);
    return PTSTORE_OK;
  }
  const u32 variant = (h->cfg.flags >> 16) & 0xFu;
  int per_sm = (int)((h->cfg.flags >> 20) & 0xFFu);
  if (!(h->cfg.flags & PTSTORE_COPY_VECTOR) && !host_side_possible) {
    BulkVariant v = kBulkVariants[variant < (u32)kNumBulkVariants ? variant : 0];
    if (v.stages == 0) v = auto_bulk(h->st.chunk_bytes);
    if (h->has_env_tune) v = h->env_tune;
    if (MODE == COPY_FETCH_MULTI && !v.hint) return launch_bulk_multi(h, pc, s, v, per_sm ? per_sm : v.ctas_per_sm);
    return launch_bulk<MODE>(h, pc, s, v, per_sm ? per_sm : v.ctas_per_sm);
  }
  switch (variant) {
    case 1:
      copy_vector_kernel<MODE, 256, 8><<<h->sms * (per_sm ? per_sm : 8), 256, 0, s>>>(h->st, pc, desc, n_pairs);
      break;
    case 2:
      copy_vector_kernel<MODE, 512, 4><<<h->sms * (per_sm ? per_sm : 4), 512, 0, s>>>(h->st, pc, desc, n_pairs);
      break;
    default:
      copy_vector_kernel<MODE, 256, 4><<<h->sms * (per_sm ? per_sm : 16), 256, 0, s>>>(h->st, pc, desc, n_pairs);
      break;
  }
  PTS_CHECK_LAUNCH(h);
  return PTSTORE_OK;
}

// ---- radix sort of the eviction candidates ----------------------------------------------------------------------
int bytes_needed(u64 max_value) {
  int b = 0;
  while (max_value) { ++b; max_value >>= 8; }
  return b ? b : 1;
}

// sorts sort_buf[0][0..ev_cand) ; returns the index of the buffer that holds the result in *result
int launch_sort(ptstore* h, cudaStream_t s, int* result) {
  const u32 nt = h->lay.n_tiles;
  const bool small = sort_steps_for((u64)h->cfg.hbm_blocks + h->cfg.host_blocks) == 2;
  int cur = 0;
  struct Pass { int word, shift; } passes[16];
  int np = 0;
  const int id_bytes = bytes_needed((u64)h->cfg.hbm_blocks + h->cfg.host_blocks - 1);
  for (int b = 0; b < id_bytes; ++b) passes[np++] = {0, 8 * b};
  passes[np++] = {0, 32};
  passes[np++] = {0, 40};
  // LRU: stamps are at most the epoch.  GDSF: a priority H = L + F has no bound the host knows (L accumulates the
  // priorities of earlier victims), so the whole word is sorted
  const int st_bytes = h->st.policy ? 8 : bytes_needed(h->epoch);
  for (int b = 0; b < st_bytes; ++b) passes[np++] = {1, 8 * b};
  for (int p = 0; p < np; ++p) {
    if (small) sort_hist_kernel<2><<<nt, SORT_THREADS, 0, s>>>(h->sort_buf[cur], &h->st.ctrl->ev_cand, passes[p].word, passes[p].shift, h->hist, nt);
    else sort_hist_kernel<8><<<nt, SORT_THREADS, 0, s>>>(h->sort_buf[cur], &h->st.ctrl->ev_cand, passes[p].word, passes[p].shift, h->hist, nt);
    PTS_CHECK_LAUNCH(h);
    sort_scan_kernel<<<1, 1024, 0, s>>>(h->hist, 256u * nt);
    PTS_CHECK_LAUNCH(h);
    if (small) sort_scatter_kernel<2><<<nt, SORT_THREADS, 0, s>>>(h->sort_buf[cur], h->sort_buf[cur ^ 1], &h->st.ctrl->ev_cand, passes[p].word,
                                                                passes[p].shift, h->hist, nt);
    else sort_scatter_kernel<8><<<nt, SORT_THREADS, 0, s>>>(h->sort_buf[cur], h->sort_buf[cur ^ 1], &h->st.ctrl->ev_cand, passes[p].word,
                                                     passes[p].shift, h->hist, nt);
    PTS_CHECK_LAUNCH(h);
    cur ^= 1;
  }
  *result = cur;
  return PTSTORE_OK;
}

// deleted markers are reclaimed at the start of an insert once they exceed 1/8 of the table (device-side decision)
inline u32 rebuild_threshold(const ptstore* h) { return (u32)(h->cfg.table_slots / 8); }

int maybe_rebuild(ptstore* h, cudaStream_t s) {
  const int cap = h->sms * 8;
  table_stash_kernel<<<grid_for((long long)h->cfg.table_slots, 256, cap), 256, 0, s>>>(h->st, h->stash, rebuild_threshold(h));
  PTS_CHECK_LAUNCH(h);
  table_rebuild_kernel<<<grid_for((long long)h->cfg.table_slots, 256, cap), 256, 0, s>>>(h->st, h->stash, rebuild_threshold(h));
  PTS_CHECK_LAUNCH(h);
  return PTSTORE_OK;
}

// drop phase: tier, mode EV_DROP (victims -> caller) or EV_HOST_ROOM (victims -> scratch)
int run_drop(ptstore* h, int tier, int mode, u32 n, int* n_evicted, int* victims, cudaStream_t s) {
  const int cap = h->sms * 8;
  const bool two_tier = h->cfg.host_blocks > 0;
  evict_begin_kernel<<<1, 1, 0, s>>>(h->st, mode, n);
  PTS_CHECK_LAUNCH(h);
  unsigned char* blocked = nullptr;
  if (tier == 1 && two_tier) {
    blocked = h->blocked;
    if (cudaMemsetAsync(blocked, 0, (size_t)h->cfg.hbm_blocks + h->cfg.host_blocks, s) != cudaSuccess) {
      h->last_cuda = (int)cudaGetLastError();
      return PTSTORE_E_CUDA;
    }
    mark_blocked_kernel<<<grid_for(h->cfg.hbm_blocks, 256, cap), 256, 0, s>>>(h->st, blocked);
    PTS_CHECK_LAUNCH(h);
  }
  const u32 span = tier ? h->cfg.host_blocks : h->cfg.hbm_blocks;
  collect_kernel<<<grid_for(span, 256, cap), 256, 0, s>>>(h->st, tier, blocked, h->sort_buf[0]);
  PTS_CHECK_LAUNCH(h);
  int res;
  int rc = launch_sort(h, s, &res);
  if (rc) return rc;
  apply_drop_kernel<<<grid_for(n ? n : 1, 256, cap), 256, 0, s>>>(h->st, tier, h->sort_buf[res], mode == EV_DROP ? victims : h->room);
  PTS_CHECK_LAUNCH(h);
  drop_finish_kernel<<<1, 1, 0, s>>>(h->st, tier, mode, h->sort_buf[res], n_evicted);
  PTS_CHECK_LAUNCH(h);
  return PTSTORE_OK;
}

// make `s` wait for a demotion copy that ptstore_evict_async left running on the side stream
int join_tier(ptstore* h, cudaStream_t s) {
  if (!h->tier_pending) return PTSTORE_OK;
  if (cudaStreamWaitEvent(s, h->ev_copy, 0) != cudaSuccess) { h->last_cuda = (int)cudaGetLastError(); return PTSTORE_E_CUDA; }
  h->tier_pending = false;
  return PTSTORE_OK;
}

int evict_impl(ptstore* h, int32_t tier, int32_t n_blocks, int32_t* n_evicted, int32_t* victim_ids, cudaStream_t s, bool async_copy) {
  if (!h || n_blocks < 0 || (tier != PTSTORE_TIER_HBM && tier != PTSTORE_TIER_HOST) || !n_evicted) return PTSTORE_E_INVAL;
  if (tier == PTSTORE_TIER_HOST && h->cfg.host_blocks == 0) return PTSTORE_E_INVAL;
  int rc = join_tier(h, s);
  if (rc) return rc;
  const u32 n = (u32)n_blocks;
  if (tier == PTSTORE_TIER_HOST || h->cfg.host_blocks == 0) return run_drop(h, tier, EV_DROP, n, n_evicted, victim_ids, s);
  // HBM tier with a host tier behind it: make room in the host ring, then demote
  rc = run_drop(h, 1, EV_HOST_ROOM, n, nullptr, nullptr, s);
  if (rc) return rc;
  const int cap = h->sms * 8;
  evict_begin_kernel<<<1, 1, 0, s>>>(h->st, EV_DEMOTE, n);
  PTS_CHECK_LAUNCH(h);
  collect_kernel<<<grid_for(h->cfg.hbm_blocks, 256, cap), 256, 0, s>>>(h->st, 0, nullptr, h->sort_buf[0]);
  PTS_CHECK_LAUNCH(h);
  int res;
  rc = launch_sort(h, s, &res);
  if (rc) return rc;
  apply_demote_kernel<<<grid_for(n ? n : 1, 256, cap), 256, 0, s>>>(h->st, h->sort_buf[res], h->desc_tier, victim_ids);
  PTS_CHECK_LAUNCH(h);
  demote_finish_kernel<<<1, 256, 0, s>>>(h->st, h->sort_buf[res], n_evicted, victim_ids, h->room);
  PTS_CHECK_LAUNCH(h);
  Paged none = {};
  if (!async_copy) return launch_copy<COPY_POOL>(h, none, true, s, h->desc_tier, &h->st.ctrl->n_pairs_tier, h->host_ctas);
  // the copy HBM -> host goes to the side stream, ordered after the metadata kernels above
  if (!h->tier_ready) {
    if (cudaStreamCreateWithFlags(&h->tier_stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_meta, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_copy, cudaEventDisableTiming) != cudaSuccess) {
      h->last_cuda = (int)cudaGetLastError();
      return PTSTORE_E_CUDA;
    }
    h->tier_ready = true;
  }
  if (cudaEventRecord(h->ev_meta, s) != cudaSuccess || cudaStreamWaitEvent(h->tier_stream, h->ev_meta, 0) != cudaSuccess) {
    h->last_cuda = (int)cudaGetLastError();
    return PTSTORE_E_CUDA;
  }
  rc = launch_copy<COPY_POOL>(h, none, true, h->tier_stream, h->desc_tier, &h->st.ctrl->n_pairs_tier, h->host_ctas);
  if (rc) return rc;
  if (cudaEventRecord(h->ev_copy, h->tier_stream) != cudaSuccess) { h->last_cuda = (int)cudaGetLastError(); return PTSTORE_E_CUDA; }
  h->tier_pending = true;
  return PTSTORE_OK;
}

}  // namespace

extern "C" {

uint64_t ptstore_workspace_bytes(const ptstore_config_t* cfg) {
  if (!geometry_ok(cfg)) return 0;
  return make_layout(cfg).total;
}

int ptstore_create(const ptstore_config_t* cfg, ptstore_t** out, ptstore_stream_t stream) {
  if (!out) return PTSTORE_E_INVAL;
  *out = nullptr;
  if (!geometry_ok(cfg)) return PTSTORE_E_INVAL;
  if (!cfg->hbm_pool || !aligned16(cfg->hbm_pool) || !cfg->workspace || (reinterpret_cast<uintptr_t>(cfg->workspace) % ALIGN)) return PTSTORE_E_INVAL;
  if (cfg->host_blocks && (!cfg->host_pool || !aligned16(cfg->host_pool))) return PTSTORE_E_INVAL;
  const Layout lay = make_layout(cfg);
  if (cfg->workspace_bytes < lay.total) return PTSTORE_E_NOMEM;
  ptstore* h = new (std::nothrow) ptstore();
  if (!h) return PTSTORE_E_NOMEM;
  std::memset(h, 0, sizeof(*h));
  h->cfg = *cfg;
  h->lay = lay;
  if (cudaSetDevice(cfg->device) != cudaSuccess) { h->last_cuda = (int)cudaGetLastError(); delete h; return PTSTORE_E_CUDA; }
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess || sms <= 0) {
    (void)cudaGetLastError(); delete h; return PTSTORE_E_CUDA;
  }
  h->sms = sms;
  h->has_env_tune = env_bulk_tune(&h->env_tune);
  unsigned char* w = static_cast<unsigned char*>(cfg->workspace);
  h->stash = reinterpret_cast<Slot*>(w + lay.table[1]);
  Store& st = h->st;
  st.table = reinterpret_cast<Slot*>(w + lay.table[0]);
  st.slots = cfg->table_slots;
  st.m_key = reinterpret_cast<u64*>(w + lay.m_key);
  st.m_parent = reinterpret_cast<u64*>(w + lay.m_parent);
  st.m_last = reinterpret_cast<u64*>(w + lay.m_last);
  st.m_freq = reinterpret_cast<u32*>(w + lay.m_freq);
  st.m_ref = reinterpret_cast<u32*>(w + lay.m_ref);
  st.m_depth = reinterpret_cast<u32*>(w + lay.m_depth);
  st.ring_ids[0] = reinterpret_cast<int*>(w + lay.ring[0]);
  st.ring_ids[1] = reinterpret_cast<int*>(w + lay.ring[1]);
  st.n[0] = cfg->hbm_blocks; st.n[1] = cfg->host_blocks;
  st.ctrl = reinterpret_cast<Ctrl*>(w + lay.ctrl);
  st.pool[0] = static_cast<unsigned char*>(cfg->hbm_pool);
  st.pool[1] = static_cast<unsigned char*>(cfg->host_pool);
  st.chunk_bytes = (u64)cfg->block_tokens * cfg->num_kv_heads * cfg->head_dim * cfg->elem_bytes;
  st.block_bytes = 2ull * cfg->num_layers * st.chunk_bytes;
  st.layers = cfg->num_layers;
  st.block_tokens = cfg->block_tokens;
  st.root_key = hroot(cfg->salt);
  st.policy = (cfg->flags & PTSTORE_EVICT_GDSF) ? 1u : 0u;
  h->blocked = w + lay.blocked;
  h->sort_buf[0] = reinterpret_cast<Key2*>(w + lay.sort[0]);
  h->sort_buf[1] = reinterpret_cast<Key2*>(w + lay.sort[1]);
  h->hist = reinterpret_cast<u32*>(w + lay.hist);
  h->room = reinterpret_cast<int*>(w + lay.room);
  h->desc = reinterpret_cast<int2*>(w + lay.desc);
  h->keys = reinterpret_cast<u64*>(w + lay.keys);
  h->eslot = reinterpret_cast<u32*>(w + lay.eslot);
  h->cta_sums = reinterpret_cast<u32*>(w + lay.cta_sums);
  h->prefix = reinterpret_cast<u32*>(w + lay.prefix);
  h->promo_first = reinterpret_cast<u32*>(w + lay.promo_first);
  h->promo_cnt = reinterpret_cast<u32*>(w + lay.promo_cnt);
  h->links = reinterpret_cast<int2*>(w + lay.links);
  h->desc_tier = reinterpret_cast<int2*>(w + lay.desc_tier);
  h->desc_host = reinterpret_cast<int2*>(w + lay.desc_host);
  {
    // a few CTAs saturate the host link; keeping these grids small leaves the SMs to kernels that run beside them
    const char* e = std::getenv("PTSTORE_HOST_CTAS");
    const int v = e ? std::atoi(e) : 0;
    h->host_ctas = v > 0 ? v : 32;
  }

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int cap = sms * 8;
  auto fail = [&](int code) { delete h; return code; };
  table_clear_kernel<<<grid_for((long long)cfg->table_slots, 256, cap), 256, 0, s>>>(st.table, cfg->table_slots);
  if (cudaGetLastError() != cudaSuccess) return fail(PTSTORE_E_CUDA);
  store_init_kernel<<<grid_for((long long)cfg->hbm_blocks + cfg->host_blocks, 256, cap), 256, 0, s>>>(st);
  if (cudaGetLastError() != cudaSuccess) return fail(PTSTORE_E_CUDA);
  ctrl_init_kernel<<<1, 1, 0, s>>>(st);
  if (cudaGetLastError() != cudaSuccess) return fail(PTSTORE_E_CUDA);
  h->launches = 3;
  *out = h;
  return PTSTORE_OK;
}

int ptstore_destroy(ptstore_t* h) {
  if (!h) return PTSTORE_E_INVAL;
  if (h->tier_ready) {
    cudaStreamSynchronize(h->tier_stream);
    cudaEventDestroy(h->ev_meta);
    cudaEventDestroy(h->ev_copy);
    cudaStreamDestroy(h->tier_stream);
  }
  delete h;
  return PTSTORE_OK;
}

int ptstore_hash(ptstore_t* h, const int32_t* tokens, const int64_t* offsets, int32_t R, int32_t max_blocks, uint64_t* keys_out,
                 ptstore_stream_t stream) {
  int rc = check_batch(h, R, max_blocks);
  if (rc) return rc;
  if (R == 0) return PTSTORE_OK;
  if (!offsets || !keys_out) return PTSTORE_E_INVAL;      // tokens may be NULL when every request is empty
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const long long* off = reinterpret_cast<const long long*>(offsets);
  u64* ko = reinterpret_cast<u64*>(keys_out);
  if (split_path(h, R, max_blocks)) return launch_hash_split(h, tokens, off, R, max_blocks, ko, s);
  switch (lanes_for(h, R, max_blocks)) {
    case 4: return launch_hash<4>(h, tokens, off, R, max_blocks, ko, s);
    case 8: return launch_hash<8>(h, tokens, off, R, max_blocks, ko, s);
    case 16: return launch_hash<16>(h, tokens, off, R, max_blocks, ko, s);
    default: return launch_hash<32>(h, tokens, off, R, max_blocks, ko, s);
  }
}

int ptstore_lookup(ptstore_t* h, const int32_t* tokens, const int64_t* offsets, int32_t R, int32_t max_blocks, uint32_t flags,
                   int32_t* matched_blocks, int32_t* block_ids, ptstore_stream_t stream) {
  int rc = check_batch(h, R, max_blocks);
  if (rc) return rc;
  if (R > 0 && (!offsets || !matched_blocks || !block_ids)) return PTSTORE_E_INVAL;
  h->epoch += 1;
  if (R == 0) return PTSTORE_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const long long* off = reinterpret_cast<const long long*>(offsets);
  if (split_path(h, R, max_blocks)) {
    rc = launch_content(h, tokens, off, R, max_blocks, h->keys, s);
    if (rc) return rc;
    lookup_chain_kernel<<<(R + 3) / 4, 128, 0, s>>>(h->st, h->keys, off, R, max_blocks, flags, h->epoch, matched_blocks, block_ids);
    PTS_CHECK_LAUNCH(h);
    return PTSTORE_OK;
  }
  switch (lanes_for(h, R, max_blocks)) {
    case 4: return launch_lookup<4>(h, tokens, off, R, max_blocks, flags, matched_blocks, block_ids, s);
    case 8: return launch_lookup<8>(h, tokens, off, R, max_blocks, flags, matched_blocks, block_ids, s);
    case 16: return launch_lookup<16>(h, tokens, off, R, max_blocks, flags, matched_blocks, block_ids, s);
    default: return launch_lookup<32>(h, tokens, off, R, max_blocks, flags, matched_blocks, block_ids, s);
  }
}

int ptstore_fetch(ptstore_t* h, const int32_t* block_ids, const int32_t* matched_blocks, int32_t R, int32_t max_blocks,
                  const ptstore_paged_cache_t* dst, const int32_t* block_tables, ptstore_stream_t stream) {
  int rc = check_batch(h, R, max_blocks);
  if (rc) return rc;
  if (R == 0) return PTSTORE_OK;
  if (!block_ids || !matched_blocks || !block_tables) return PTSTORE_E_INVAL;
  rc = check_cache(h, dst);
  if (rc) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // one descriptor per distinct source block, each with the list of its destinations (promo_first doubles as the list heads)
  const u32 n_blocks = h->cfg.hbm_blocks + h->cfg.host_blocks;
  const int cap = h->sms * 8;
  fetch_begin_kernel<<<grid_for(n_blocks, 256, cap), 256, 0, s>>>(h->st, h->promo_first, n_blocks);
  PTS_CHECK_LAUNCH(h);
  fetch_link_kernel<<<grid_for((long long)R * max_blocks, 256, cap), 256, 0, s>>>(h->st, block_ids, matched_blocks, block_tables, R, max_blocks,
                                                                                 dst->num_blocks, h->promo_first, h->links, h->desc, h->desc_host);
  PTS_CHECK_LAUNCH(h);
  Paged pc = to_paged(dst);
  pc.head = h->promo_first;
  pc.node = h->links;
  rc = launch_copy<COPY_FETCH_MULTI>(h, pc, false, s);                    // HBM-tier sources: every SM
  if (rc || h->cfg.host_blocks == 0) return rc;
  return launch_copy<COPY_FETCH_MULTI>(h, pc, true, s, h->desc_host, &h->st.ctrl->n_pairs_host, h->host_ctas);   // host-tier sources
}

int ptstore_insert(ptstore_t* h, const int32_t* tokens, const int64_t* offsets, int32_t R, int32_t max_blocks,
                   const ptstore_paged_cache_t* src, const int32_t* block_tables, int32_t* block_ids, int32_t* new_blocks,
                   ptstore_stream_t stream) {
  int rc = check_batch(h, R, max_blocks);
  if (rc) return rc;
  if (R > 0 && (!offsets || !block_ids || !new_blocks)) return PTSTORE_E_INVAL;
  const bool copy = src != nullptr && R > 0;
  if (copy) {
    rc = check_cache(h, src);
    if (rc) return rc;
    if (!block_tables) return PTSTORE_E_INVAL;
  }
  h->epoch += 1;
  if (R == 0) return PTSTORE_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  rc = join_tier(h, s);        // new blocks may reuse HBM ids whose demotion copy is still running
  if (rc) return rc;
  rc = maybe_rebuild(h, s);
  if (rc) return rc;
  const long long* off = reinterpret_cast<const long long*>(offsets);
  if (split_path(h, R, max_blocks)) rc = launch_hash_split(h, tokens, off, R, max_blocks, h->keys, s);
  else switch (lanes_for(h, R, max_blocks)) {
    case 4: rc = launch_hash<4>(h, tokens, off, R, max_blocks, h->keys, s); break;
    case 8: rc = launch_hash<8>(h, tokens, off, R, max_blocks, h->keys, s); break;
    case 16: rc = launch_hash<16>(h, tokens, off, R, max_blocks, h->keys, s); break;
    default: rc = launch_hash<32>(h, tokens, off, R, max_blocks, h->keys, s); break;
  }
  if (rc) return rc;
  const long long total = (long long)R * max_blocks;
  const int cap = h->sms * 8;
  insert_claim_kernel<<<grid_for(total, 256, cap), 256, 0, s>>>(h->st, h->keys, R, max_blocks, h->eslot, new_blocks);
  PTS_CHECK_LAUNCH(h);
  const u32 n_ctas = (u32)((total + INS_THREADS - 1) / INS_THREADS);
  insert_count_kernel<<<n_ctas, INS_THREADS, 0, s>>>(h->st, h->eslot, total, max_blocks, h->cta_sums);
  PTS_CHECK_LAUNCH(h);
  insert_plan_kernel<<<1, INS_THREADS, 0, s>>>(h->st, h->cta_sums, n_ctas, rebuild_threshold(h));
  PTS_CHECK_LAUNCH(h);
  insert_assign_kernel<<<n_ctas, INS_THREADS, 0, s>>>(h->st, h->keys, h->eslot, total, max_blocks, h->cta_sums,
                                                       copy ? block_tables : nullptr, copy ? src->num_blocks : 0, h->epoch, h->desc,
                                                       new_blocks);
  PTS_CHECK_LAUNCH(h);
  insert_finish_kernel<<<grid_for(total, 256, cap), 256, 0, s>>>(h->st, h->eslot, total, h->epoch, block_ids);
  PTS_CHECK_LAUNCH(h);
  if (copy) return launch_copy<COPY_INSERT>(h, to_paged(src), false, s);
  return PTSTORE_OK;
}

int ptstore_release(ptstore_t* h, const int32_t* block_ids, const int32_t* matched_blocks, int32_t R, int32_t max_blocks,
                    ptstore_stream_t stream) {
  int rc = check_batch(h, R, max_blocks);
  if (rc) return rc;
  if (R == 0) return PTSTORE_OK;
  if (!block_ids || !matched_blocks) return PTSTORE_E_INVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  release_kernel<<<grid_for((long long)R * max_blocks, 256, h->sms * 8), 256, 0, s>>>(h->st, block_ids, matched_blocks, R, max_blocks);
  PTS_CHECK_LAUNCH(h);
  return PTSTORE_OK;
}

int ptstore_evict(ptstore_t* h, int32_t tier, int32_t n_blocks, int32_t* n_evicted, int32_t* victim_ids, ptstore_stream_t stream) {
  return evict_impl(h, tier, n_blocks, n_evicted, victim_ids, static_cast<cudaStream_t>(stream), false);
}

int ptstore_evict_async(ptstore_t* h, int32_t tier, int32_t n_blocks, int32_t* n_evicted, int32_t* victim_ids, ptstore_stream_t stream) {
  return evict_impl(h, tier, n_blocks, n_evicted, victim_ids, static_cast<cudaStream_t>(stream), true);
}

int ptstore_join(ptstore_t* h, ptstore_stream_t stream) {
  if (!h) return PTSTORE_E_INVAL;
  return join_tier(h, static_cast<cudaStream_t>(stream));
}

int ptstore_promote(ptstore_t* h, int32_t* block_ids, const int32_t* matched_blocks, int32_t R, int32_t max_blocks, uint32_t flags,
                    int32_t max_promote, int32_t* n_promoted, ptstore_stream_t stream) {
  int rc = check_batch(h, R, max_blocks);
  if (rc) return rc;
  if (h->cfg.host_blocks == 0 || max_promote < 0) return PTSTORE_E_INVAL;
  if (R > 0 && (!block_ids || !matched_blocks)) return PTSTORE_E_INVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  rc = join_tier(h, s);
  if (rc) return rc;
  const u64 N = (u64)h->cfg.hbm_blocks + h->cfg.host_blocks;
  if (cudaMemsetAsync(h->promo_first, 0xFF, N * 4, s) != cudaSuccess || cudaMemsetAsync(h->promo_cnt, 0, N * 4, s) != cudaSuccess) {
    h->last_cuda = (int)cudaGetLastError();
    return PTSTORE_E_CUDA;
  }
  const long long total = (long long)R * max_blocks;
  const int cap = h->sms * 8;
  const u32 pinned = (flags & PTSTORE_PINNED_LIST) ? 1u : 0u;
  const u32 n_ctas = (u32)((total + INS_THREADS - 1) / INS_THREADS);
  if (total > 0) {
    promote_mark_kernel<<<grid_for(total, 256, cap), 256, 0, s>>>(h->st, block_ids, matched_blocks, total, max_blocks, h->promo_first, h->promo_cnt);
    PTS_CHECK_LAUNCH(h);
    promote_count_kernel<<<n_ctas, INS_THREADS, 0, s>>>(h->st, block_ids, matched_blocks, total, max_blocks, h->promo_first, h->promo_cnt,
                                                        pinned, h->cta_sums);
    PTS_CHECK_LAUNCH(h);
  }
  promote_plan_kernel<<<1, INS_THREADS, 0, s>>>(h->st, h->cta_sums, total > 0 ? n_ctas : 0, (u32)max_promote, n_promoted);
  PTS_CHECK_LAUNCH(h);
  if (total == 0) return PTSTORE_OK;
  promote_assign_kernel<<<n_ctas, INS_THREADS, 0, s>>>(h->st, block_ids, matched_blocks, total, max_blocks, h->promo_first, h->promo_cnt,
                                                       pinned, h->cta_sums, h->desc);
  PTS_CHECK_LAUNCH(h);
  promote_rewrite_kernel<<<grid_for(total, 256, cap), 256, 0, s>>>(h->st, block_ids, matched_blocks, total, max_blocks, h->promo_first);
  PTS_CHECK_LAUNCH(h);
  Paged none = {};
  return launch_copy<COPY_POOL>(h, none, true, s, nullptr, nullptr, h->host_ctas);      // host -> HBM at host-link speed
}

int ptstore_status(ptstore_t* h, ptstore_stream_t stream, uint32_t* status_out) {
  if (!h || !status_out) return PTSTORE_E_INVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(status_out, &h->st.ctrl->status, sizeof(u32), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaMemsetAsync(&h->st.ctrl->status, 0, sizeof(u32), s) != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess) {
    h->last_cuda = (int)cudaGetLastError();
    return PTSTORE_E_CUDA;
  }
  return PTSTORE_OK;
}

int ptstore_stats(ptstore_t* h, ptstore_stream_t stream, ptstore_stats_t* out) {
  if (!h || !out) return PTSTORE_E_INVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  Ctrl c;
  if (cudaMemcpyAsync(&c, h->st.ctrl, sizeof(Ctrl), cudaMemcpyDeviceToHost, s) != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess) {
    h->last_cuda = (int)cudaGetLastError();
    return PTSTORE_E_CUDA;
  }
  std::memset(out, 0, sizeof(*out));
  out->epoch = h->epoch;
  for (int t = 0; t < 2; ++t) {
    out->live_nodes[t] = c.live[t];
    out->free_blocks[t] = c.ring[t].count;
    out->blocks_fetched[t] = c.blocks_fetched[t];
    out->blocks_dropped[t] = c.blocks_dropped[t];
  }
  out->tombstones = c.tombstones;
  out->query_blocks = c.query_blocks;
  out->probes_issued = c.probes_issued;
  out->slots_visited = c.slots_visited;
  out->blocks_matched = c.blocks_matched;
  for (int i = 0; i < LOOKUP_STRIPES; ++i) {
    out->query_blocks += c.lookup_stripes[i][0];
    out->probes_issued += c.lookup_stripes[i][1];
    out->slots_visited += c.lookup_stripes[i][2];
    out->blocks_matched += c.lookup_stripes[i][3];
  }
  out->blocks_inserted = c.blocks_inserted;
  out->blocks_denied = c.blocks_denied;
  out->blocks_demoted = c.blocks_demoted;
  out->rebuilds = c.rebuilds;
  out->blocks_promoted = c.blocks_promoted;
  out->gdsf_clock = c.inflation;
  out->blocks_fetched_distinct = c.blocks_fetched_distinct;
  return PTSTORE_OK;
}

int ptstore_stats_enqueue(ptstore_t* h, ptstore_stats_t* out, ptstore_stream_t stream) {
  static_assert(sizeof(StatsOut) == sizeof(ptstore_stats_t), "device and host views of the counters must match");
  if (!h || !out) return PTSTORE_E_INVAL;
  stats_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(h->st, h->epoch, reinterpret_cast<StatsOut*>(out));
  PTS_CHECK_LAUNCH(h);
  return PTSTORE_OK;
}

uint64_t ptstore_launch_count(const ptstore_t* h) { return h ? h->launches : 0; }
int ptstore_last_cuda_error(const ptstore_t* h) { return h ? h->last_cuda : 0; }

const char* ptstore_strerror(int code) {
  switch (code) {
    case PTSTORE_OK: return "ok";
    case PTSTORE_E_INVAL: return "invalid argument";
    case PTSTORE_E_CUDA: return "CUDA call failed";
    case PTSTORE_E_NOMEM: return "handle allocation failed or workspace too small";
    case PTSTORE_E_LIMIT: return "batch exceeds the limits given at create";
    default: return "unknown error";
  }
}

}  // extern "C"
