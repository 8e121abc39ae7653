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
#include "fused.cuh"

using namespace pts;

namespace {

constexpr u64 ALIGN = 256;
inline u64 align_up(u64 x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }

struct Layout {            // byte offsets into the workspace
  u64 table, m_key, m_parent, m_last, m_freq, m_ref, m_depth, m_flight, ring[2], ctrl, blocked, sort[2], hist, tile_stats, room, desc,
      keys, eslot, cta_sums, prefix, promo_first, promo_cnt, heads, links, desc_tier, desc_host, progress, total;
};

constexpr u32 MAX_COOP_GRID = 256;      // cooperative kernels use at most this many CTAs (and at most one per SM)
constexpr u64 MIN_SLOTS = 2 * PROBE_WINDOW;   // the windowed probe wraps an index once, so a table is never smaller than this

inline u64 effective_slots(const ptstore_config_t* c) { return c->table_slots < MIN_SLOTS ? MIN_SLOTS : c->table_slots; }

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
  const u64 N = (u64)c->hbm_blocks + c->host_blocks, M = c->max_batch_blocks, S = effective_slots(c);
  u64 o = 0;
  auto take = [&](u64 bytes) { u64 at = o; o = align_up(o + (bytes ? bytes : 1)); return at; };
  L.table = take(S * sizeof(Slot));
  L.m_key = take(N * 8); L.m_parent = take(N * 8); L.m_last = take(N * 8);
  L.m_freq = take(N * 4); L.m_ref = take(N * 4); L.m_depth = take(N * 4); L.m_flight = take(N * 4);
  L.ring[0] = take((u64)c->hbm_blocks * 4); L.ring[1] = take((u64)c->host_blocks * 4);
  L.ctrl = take(sizeof(Ctrl));
  L.blocked = take(N);
  // eviction: one sort record per block id of a tier, padded to whole tiles of the largest grid
  const u64 recs = N + (u64)MAX_COOP_GRID * EV_THREADS + 8192;
  L.sort[0] = take(recs * sizeof(Key2)); L.sort[1] = take(recs * sizeof(Key2));
  L.hist = take((u64)256 * MAX_COOP_GRID * 4);
  L.tile_stats = take((u64)MAX_COOP_GRID * 4 * 8);
  L.room = take((u64)c->host_blocks * 4);
  L.desc = take((M > N ? M : N) * sizeof(int2));
  L.keys = take(M * 8);
  L.eslot = take(M * 4);
  L.cta_sums = take(((M + INS_THREADS - 1) / INS_THREADS + 1) * 4);
  L.prefix = take(((u64)c->max_requests + 1) * 4);
  L.promo_first = take(N * 4);
  L.promo_cnt = take(N * 4);
  L.heads = take(N * 8);
  L.links = take(M * sizeof(int2));
  L.desc_tier = take((u64)c->hbm_blocks * sizeof(int2));
  L.desc_host = take((c->host_blocks ? (M < c->host_blocks ? M : (u64)c->host_blocks) : 1) * sizeof(int2));
  L.progress = take((u64)FUSED_MAX_REQUESTS * 24);      // per request: two progress words and a unit counter
  L.total = o;
  return L;
}

}  // namespace

struct BulkVariant { int stages, stage_bytes, ctas_per_sm, group, hint; };

struct ptstore {
  ptstore_config_t cfg;
  Layout lay;
  Store st;
  unsigned char* blocked;
  Key2* sort_buf[2];
  u32* hist;
  u64* tile_stats;
  int* room;
  int2* desc;
  u64* keys;
  u32* eslot;
  u32* cta_sums;
  u32* prefix;
  u32* promo_first;
  u32* promo_cnt;
  u64* heads;            // fetch: tagged heads of the destination lists, one per block id
  int2* links;           // fetch: destination list nodes, one per (request, block) entry
  int2* desc_tier;       // demotion: {HBM id, host id} pairs
  int2* desc_host;       // fetch: descriptors of distinct host-tier source blocks
  u64* progress;         // fused lookup + gather, per request: lookup progress word, owned-list progress word, unit counter
  int fused_smem_set;    // dynamic shared memory already granted to the fused kernel
  int host_ctas;         // grid of the copies that run at host-link speed
  cudaStream_t tier_stream;   // side stream of the asynchronous demotion copy (created on first use)
  cudaEvent_t ev_meta, ev_copy;
  bool tier_ready, tier_pending;
  u32 flight_seq;        // tag of the demotion copy that may still be running (valid while tier_pending)
  u32 fetch_seq;         // sequence number of the last fetch call (tags the list heads; never 0)
  u32 coop_seq;          // cooperative launches with grid barriers so far (selects the barrier counter)
  u32 gather_seq;        // launches of the fused lookup + gather so far (the tag of its progress words)
  u32 wait_limit;        // polls per bounded wait in the copy kernels' main loop
  // the batch whose chained keys the last lookup left in `keys` / `prefix` (for ptstore_insert_after_lookup)
  const void* lk_tokens; const void* lk_offsets; int lk_R, lk_max_blocks; bool lk_valid;
  u64 inserts_resumed;   // inserts that resumed hashing behind a lookup's keys
  cudaEvent_t time_before, time_after;   // one-shot: recorded around the next HBM copy kernel (ptstore_time_next_copy)
  int coop_grid;         // CTAs a cooperative kernel may use: one per SM, at most MAX_COOP_GRID
  u64 epoch;
  u64 launches;
  int last_cuda;
  int sms;
  int bulk_smem_set[4];
  int bulk_multi_smem_set;  // dynamic shared memory already granted to the bulk kernel of each mode
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

// A kernel whose CTAs wait for one another: all of them must be resident at once.  Kernels that meet at grid-wide barriers
// are numbered by coop_seq, which selects the barrier's counter, and every one of them clears the counter of a later launch,
// so a kernel that has no barrier must not take a number from that sequence: it gets its own (`barrier` false).
template <typename Kernel, typename Args>
int launch_coop(ptstore* h, Kernel kernel, int grid, int threads, Args& args, cudaStream_t s, size_t smem = 0, bool barrier = true) {
  args.launch_seq = barrier ? ++h->coop_seq : ++h->gather_seq;
  void* params[2] = {&h->st, &args};
  cudaError_t e = cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(kernel), dim3(grid), dim3(threads), params, smem, s);
  h->launches += 1;
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    h->last_cuda = (int)e;
    if (barrier) --h->coop_seq; else --h->gather_seq;      // the number was not used: the kernel that clears a later counter never ran
    return PTSTORE_E_CUDA;
  }
  return PTSTORE_OK;
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
                  int* ids, const FetchLink& fl, cudaStream_t s) {
  const long long warps = ((long long)R + (32 / L) - 1) / (32 / L);
  const int grid = (int)((warps * 32 + 255) / 256);
  lookup_kernel<L><<<grid, 256, 0, s>>>(h->st, tokens, offsets, R, max_blocks, flags, h->epoch, matched, ids, fl, h->keys, h->prefix);
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
// Ring geometries selectable with PTSTORE_COPY_VARIANT (see include/ptstore.h); 0 sizes the ring from the chunk size.
const BulkVariant kBulkVariants[] = {
    {0, 0, 1, 1, 0},       // 0: default, sized by auto_bulk() from the chunk size
    {8, 8192, 3, 1, 0},    // 1: 8 stages of 8 KiB, 3 CTAs per SM
    {3, 32768, 1, 1, 0},   // 2: 3 stages of 32 KiB
    {4, 16384, 3, 1, 0},   // 3: 4 stages of 16 KiB, 3 CTAs per SM
    {12, 16384, 1, 1, 0},  // 4: 12 stages of 16 KiB
    {6, 16384, 1, 2, 0},   // 5: 6 stages of 16 KiB, a CTA takes two consecutive pieces at a time
    {6, 16384, 1, 1, 1},   // 6: 6 stages of 16 KiB, loads and stores marked evict-first in L2
    {3, 65536, 1, 1, 0},   // 7: 3 stages of 64 KiB
};
constexpr int kNumBulkVariants = (int)(sizeof(kBulkVariants) / sizeof(kBulkVariants[0]));

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
int launch_bulk(ptstore* h, const Paged& pc, cudaStream_t s, const BulkVariant& v, int ctas_per_sm, const int2* desc, const u32* n_pairs) {
  const int smem = v.stages * v.stage_bytes;
  if (smem > h->bulk_smem_set[MODE]) {
    if (cudaFuncSetAttribute(copy_bulk_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
      h->last_cuda = (int)cudaGetLastError();
      return PTSTORE_E_CUDA;
    }
    h->bulk_smem_set[MODE] = smem;
  }
  BulkTune t = {v.stages, v.stage_bytes, v.group, v.hint, h->wait_limit};
  copy_bulk_kernel<MODE><<<h->sms * ctas_per_sm, 32, smem, s>>>(h->st, pc, desc, n_pairs, t);
  PTS_CHECK_LAUNCH(h);
  return PTSTORE_OK;
}

// multi-destination fetch: dynamic dealing of `group`-piece units (default: a quarter of a source block)
int launch_bulk_multi(ptstore* h, const Paged& pc, cudaStream_t s, BulkVariant v, int ctas_per_sm, const int2* desc, const u32* n_pairs,
                      u32* work_counter) {
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
  BulkTune t = {v.stages, v.stage_bytes, group, 0, h->wait_limit};
  copy_bulk_multi_kernel<<<h->sms * ctas_per_sm, 32, smem, s>>>(h->st, pc, desc, n_pairs, work_counter, t);
  PTS_CHECK_LAUNCH(h);
  return PTSTORE_OK;
}

// desc / n_pairs: the descriptor list to copy; grid > 0: a copy at host-link speed (fixed small grid, vector engine)
template <int MODE>
int launch_copy(ptstore* h, const Paged& pc, bool host_side_possible, cudaStream_t s, const int2* desc, const u32* n_pairs, int grid = 0,
                u32* work_counter = nullptr) {
  if (grid > 0) {
    copy_vector_kernel<MODE, 256, 8><<<grid, 256, 0, s>>>(h->st, pc, desc, n_pairs);
    PTS_CHECK_LAUNCH(h);
    return PTSTORE_OK;
  }
  // a caller who asked for it gets its two events recorded around this kernel (one shot)
  struct Timer {
    ptstore* h; cudaStream_t s; cudaEvent_t after;
    Timer(ptstore* h_, cudaStream_t s_) : h(h_), s(s_), after(h_->time_after) {
      if (h->time_before) cudaEventRecord(h->time_before, s);
      h->time_before = nullptr; h->time_after = nullptr;
    }
    ~Timer() { if (after) cudaEventRecord(after, s); }
  } timer(h, s);
  const u32 variant = (h->cfg.flags >> 16) & 0xFu;
  int per_sm = (int)((h->cfg.flags >> 20) & 0xFFu);
  if (!(h->cfg.flags & PTSTORE_COPY_VECTOR) && !host_side_possible) {
    BulkVariant v = kBulkVariants[variant < (u32)kNumBulkVariants ? variant : 0];
    if (v.stages == 0) v = auto_bulk(h->st.chunk_bytes);
    if (MODE == COPY_FETCH_MULTI && !v.hint) return launch_bulk_multi(h, pc, s, v, per_sm ? per_sm : v.ctas_per_sm, desc, n_pairs, work_counter);
    return launch_bulk<MODE>(h, pc, s, v, per_sm ? per_sm : v.ctas_per_sm, desc, n_pairs);
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

// make `s` wait for a demotion copy left running on the side stream
int join_tier(ptstore* h, cudaStream_t s) {
  if (!h->tier_pending) return PTSTORE_OK;
  if (cudaStreamWaitEvent(s, h->ev_copy, 0) != cudaSuccess) { h->last_cuda = (int)cudaGetLastError(); return PTSTORE_E_CUDA; }
  h->tier_pending = false;
  return PTSTORE_OK;
}

// one phase of an eviction: a single cooperative launch
int launch_evict(ptstore* h, int tier, int mode, EvictArgs a, cudaStream_t s) {
  const u32 span = tier ? h->cfg.host_blocks : h->cfg.hbm_blocks;
  // CTAs: measured on B200, a pass over 512 records per CTA costs about as much as its two barriers, and barriers get
  // slower with more CTAs: 512 records per CTA up to 64 CTAs, then 2048 per CTA up to one CTA per SM, then whatever it takes
  int grid = (int)((span + 511) / 512);
  if (grid > 64) { grid = (int)((span + 2047) / 2048); if (grid < 64) grid = 64; }
  if (grid < 1) grid = 1;
  if (grid > h->coop_grid) grid = h->coop_grid;
  const u32 per = (span + grid - 1) / grid;
  a.tier = tier;
  a.mode = mode;
  a.tile_elems = (per + EV_THREADS - 1) / EV_THREADS * EV_THREADS;
  a.room = h->room;
  a.buf[0] = h->sort_buf[0]; a.buf[1] = h->sort_buf[1];
  a.hist = h->hist;
  a.tile_stats = h->tile_stats;
  a.blocked = (tier == 1 && h->cfg.host_blocks) ? h->blocked : nullptr;
  a.desc_tier = h->desc_tier;
  return launch_coop(h, evict_kernel, grid, EV_THREADS, a, s);
}

// n victims (want_free < 0) or as many as bring the HBM free count to want_free - sum(minus) (decided on the device)
int evict_impl(ptstore* h, int32_t tier, u32 n, long long want_free, const int* minus, int n_minus, int32_t* n_evicted,
               int32_t* victim_ids, u32 max_victims, cudaStream_t s, bool async_copy) {
  int rc = join_tier(h, s);
  if (rc) return rc;
  EvictArgs a = {};
  a.n = n; a.want_free = want_free; a.minus = minus; a.n_minus = n_minus; a.max_victims = max_victims;
  a.n_evicted = n_evicted; a.victims = victim_ids;
  if (tier == PTSTORE_TIER_HOST || h->cfg.host_blocks == 0) return launch_evict(h, tier, EV_DROP, a, s);
  // HBM tier with a host tier behind it: make room in the host ring, then demote
  EvictArgs room = a;
  room.n_evicted = nullptr; room.victims = nullptr;
  rc = launch_evict(h, 1, EV_HOST_ROOM, room, s);
  if (rc) return rc;
  if (async_copy) {
    if (++h->flight_seq == 0) h->flight_seq = 1;
    a.flight_seq = h->flight_seq;
  }
  rc = launch_evict(h, 0, EV_DEMOTE, a, s);
  if (rc) return rc;
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

// the linking record of the next fetch call
int next_fetch_link(ptstore* h, const ptstore_paged_cache_t* dst, const int32_t* block_tables, cudaStream_t s, FetchLink* fl) {
  if (++h->fetch_seq == 0) {          // the tag wrapped: heads written 2^32 calls ago would look current
    const u64 N = (u64)h->cfg.hbm_blocks + h->cfg.host_blocks;
    if (cudaMemsetAsync(h->heads, 0, N * 8, s) != cudaSuccess || cudaMemsetAsync(h->st.ctrl->f_pairs, 0, 6 * sizeof(u32), s) != cudaSuccess) {
      h->last_cuda = (int)cudaGetLastError();
      return PTSTORE_E_CUDA;
    }
    h->fetch_seq = 1;
  }
  fl->bt = block_tables;
  fl->cache_blocks = dst->num_blocks;
  fl->seq = h->fetch_seq;
  fl->pending_seq = h->tier_pending ? h->flight_seq : 0;
  fl->heads = h->heads;
  fl->node = h->links;
  fl->desc = h->desc;
  fl->desc_host = h->desc_host;
  return PTSTORE_OK;
}

// the copies of a fetch whose lists have been linked under tag `seq`
int launch_fetch_copies(ptstore* h, const ptstore_paged_cache_t* dst, u32 seq, cudaStream_t s) {
  Paged pc = to_paged(dst);
  pc.head = h->heads;
  pc.node = h->links;
  Ctrl* c = h->st.ctrl;
  const u32 slot = seq & 1u;
  int rc = launch_copy<COPY_FETCH_MULTI>(h, pc, false, s, h->desc, &c->f_pairs[slot], 0, &c->f_work[slot]);     // HBM-tier sources: every SM
  if (rc || h->cfg.host_blocks == 0) return rc;
  return launch_copy<COPY_FETCH_MULTI>(h, pc, true, s, h->desc_host, &c->f_pairs_host[slot], h->host_ctas);       // host-tier sources
}

int lookup_impl(ptstore* h, const int32_t* tokens, const int64_t* offsets, int32_t R, int32_t max_blocks, uint32_t flags,
                int32_t* matched_blocks, int32_t* block_ids, const FetchLink& fl, cudaStream_t s) {
  const long long* off = reinterpret_cast<const long long*>(offsets);
  h->lk_tokens = tokens; h->lk_offsets = offsets; h->lk_R = R; h->lk_max_blocks = max_blocks; h->lk_valid = true;
  if (split_path(h, R, max_blocks)) {      // few long requests: one CTA per request does content hashes, chain and list linking
    lookup_long_kernel<<<R, LONG_THREADS, 0, s>>>(h->st, tokens, h->keys, off, R, max_blocks, flags, h->epoch, matched_blocks, block_ids, fl,
                                                  h->prefix);
    PTS_CHECK_LAUNCH(h);
    return PTSTORE_OK;
  }
  switch (lanes_for(h, R, max_blocks)) {
    case 4: return launch_lookup<4>(h, tokens, off, R, max_blocks, flags, matched_blocks, block_ids, fl, s);
    case 8: return launch_lookup<8>(h, tokens, off, R, max_blocks, flags, matched_blocks, block_ids, fl, s);
    case 16: return launch_lookup<16>(h, tokens, off, R, max_blocks, flags, matched_blocks, block_ids, fl, s);
    default: return launch_lookup<32>(h, tokens, off, R, max_blocks, flags, matched_blocks, block_ids, fl, s);
  }
}

// A handful of long prompts, HBM tier only, default copy ring: lookup and gather as one cooperative launch in which the
// copies of a prompt's first blocks start while its hash chain is still running.  Not taken when the caller asked for
// events around the copy kernel (there is no separate one).
bool fused_small_batch(const ptstore* h, int R, int max_blocks) {
  return split_path(h, R, max_blocks) && R <= FUSED_MAX_REQUESTS && max_blocks <= FUSED_MAX_BLOCKS && h->cfg.host_blocks == 0 && !(h->cfg.flags & PTSTORE_COPY_VECTOR) &&
         ((h->cfg.flags >> 16) & 0xFu) == 0 && ((h->cfg.flags >> 20) & 0xFFu) == 0 && h->time_before == nullptr;
}

int launch_lookup_gather(ptstore* h, const int32_t* tokens, const int64_t* offsets, int R, int max_blocks, u32 flags,
                         const ptstore_paged_cache_t* dst, const int32_t* block_tables, int32_t* matched, int32_t* ids, cudaStream_t s) {
  const BulkVariant v = auto_bulk(h->st.chunk_bytes);
  const int smem = v.stages * v.stage_bytes;
  if (smem > h->fused_smem_set) {
    if (cudaFuncSetAttribute(lookup_gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
      h->last_cuda = (int)cudaGetLastError();
      return PTSTORE_E_CUDA;
    }
    h->fused_smem_set = smem;
  }
  const u32 ppc = (u32)((h->st.chunk_bytes + v.stage_bytes - 1) / v.stage_bytes);
  const u32 per_block = 2u * h->st.layers * ppc;
  FusedArgs a = {};
  a.tokens = tokens;
  a.offsets = reinterpret_cast<const long long*>(offsets);
  a.R = R; a.max_blocks = max_blocks; a.flags = flags; a.epoch = h->epoch;
  a.matched = matched; a.ids_out = ids;
  a.scratch = h->keys; a.hashed = h->prefix;
  a.bt = block_tables;
  a.pc = to_paged(dst);
  a.progress = h->progress;
  a.owned_progress = h->progress + FUSED_MAX_REQUESTS;
  a.taken = reinterpret_cast<u32*>(h->progress + 2 * FUSED_MAX_REQUESTS);
  a.owned = h->eslot;                  // scratch of the insert kernel, free between inserts
  a.owned_src = h->links;              // list nodes of the list-based fetch, which this call replaces
  if (++h->fetch_seq == 0) {          // keep the fetch calls' alternation of counters (and their tag wrap) in step
    const u64 N = (u64)h->cfg.hbm_blocks + h->cfg.host_blocks;
    if (cudaMemsetAsync(h->heads, 0, N * 8, s) != cudaSuccess || cudaMemsetAsync(h->st.ctrl->f_pairs, 0, 6 * sizeof(u32), s) != cudaSuccess) {
      h->last_cuda = (int)cudaGetLastError();
      return PTSTORE_E_CUDA;
    }
    h->fetch_seq = 1;
  }
  a.fetch_seq = h->fetch_seq;
  // units of an eighth of a block: with so few blocks the last units decide the time (measured on B200, batch 1 / 4 / 16,
  // whole step: a quarter 210 / 712 / 2681 us, an eighth 207 / 705 / 2681, a sixteenth 209 / 724 / 2764)
  a.tune = {v.stages, v.stage_bytes, (int)(per_block >= 8 ? per_block / 8 : per_block), 0, h->wait_limit};
  h->lk_tokens = tokens; h->lk_offsets = offsets; h->lk_R = R; h->lk_max_blocks = max_blocks; h->lk_valid = true;
  return launch_coop(h, lookup_gather_kernel, h->coop_grid, LONG_THREADS, a, s, (size_t)smem, false);
}

template <int L>
int launch_insert(ptstore* h, InsertArgs& a, int grid, cudaStream_t s) { return launch_coop(h, insert_kernel<L>, grid, INS_THREADS, a, s); }

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
  int sms = 0, coop = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess || sms <= 0 ||
      cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, cfg->device) != cudaSuccess || !coop) {
    (void)cudaGetLastError(); delete h; return PTSTORE_E_CUDA;
  }
  h->sms = sms;
  h->coop_grid = sms < (int)MAX_COOP_GRID ? sms : (int)MAX_COOP_GRID;
  h->wait_limit = BULK_POLL_LIMIT;
  unsigned char* w = static_cast<unsigned char*>(cfg->workspace);
  Store& st = h->st;
  st.table = reinterpret_cast<Slot*>(w + lay.table);
  st.slots = effective_slots(cfg);
  st.m_key = reinterpret_cast<u64*>(w + lay.m_key);
  st.m_parent = reinterpret_cast<u64*>(w + lay.m_parent);
  st.m_last = reinterpret_cast<u64*>(w + lay.m_last);
  st.m_freq = reinterpret_cast<u32*>(w + lay.m_freq);
  st.m_ref = reinterpret_cast<u32*>(w + lay.m_ref);
  st.m_depth = reinterpret_cast<u32*>(w + lay.m_depth);
  st.m_flight = reinterpret_cast<u32*>(w + lay.m_flight);
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
  h->tile_stats = reinterpret_cast<u64*>(w + lay.tile_stats);
  h->room = reinterpret_cast<int*>(w + lay.room);
  h->desc = reinterpret_cast<int2*>(w + lay.desc);
  h->keys = reinterpret_cast<u64*>(w + lay.keys);
  h->eslot = reinterpret_cast<u32*>(w + lay.eslot);
  h->cta_sums = reinterpret_cast<u32*>(w + lay.cta_sums);
  h->prefix = reinterpret_cast<u32*>(w + lay.prefix);
  h->promo_first = reinterpret_cast<u32*>(w + lay.promo_first);
  h->promo_cnt = reinterpret_cast<u32*>(w + lay.promo_cnt);
  h->heads = reinterpret_cast<u64*>(w + lay.heads);
  h->links = reinterpret_cast<int2*>(w + lay.links);
  h->desc_tier = reinterpret_cast<int2*>(w + lay.desc_tier);
  h->desc_host = reinterpret_cast<int2*>(w + lay.desc_host);
  h->progress = reinterpret_cast<u64*>(w + lay.progress);
  h->host_ctas = 32;     // a few CTAs saturate the host link; a small grid leaves the SMs to kernels that run beside it

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int cap = sms * 8;
  auto fail = [&](int code) { delete h; return code; };
  table_clear_kernel<<<grid_for((long long)st.slots, 256, cap), 256, 0, s>>>(st.table, st.slots);
  if (cudaGetLastError() != cudaSuccess) return fail(PTSTORE_E_CUDA);
  store_init_kernel<<<grid_for((long long)cfg->hbm_blocks + cfg->host_blocks, 256, cap), 256, 0, s>>>(st, h->heads);
  if (cudaGetLastError() != cudaSuccess) return fail(PTSTORE_E_CUDA);
  ctrl_init_kernel<<<1, 1, 0, s>>>(st, h->progress, 2 * FUSED_MAX_REQUESTS);
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
  FetchLink none = {};
  return lookup_impl(h, tokens, offsets, R, max_blocks, flags, matched_blocks, block_ids, none, static_cast<cudaStream_t>(stream));
}

int ptstore_lookup_fetch(ptstore_t* h, const int32_t* tokens, const int64_t* offsets, int32_t R, int32_t max_blocks, uint32_t flags,
                         const ptstore_paged_cache_t* dst, const int32_t* block_tables, int32_t* matched_blocks, int32_t* block_ids,
                         ptstore_stream_t stream) {
  int rc = check_batch(h, R, max_blocks);
  if (rc) return rc;
  if (R > 0 && (!offsets || !matched_blocks || !block_ids || !block_tables)) return PTSTORE_E_INVAL;
  if (R > 0) {
    rc = check_cache(h, dst);
    if (rc) return rc;
  }
  h->epoch += 1;
  if (R == 0) return PTSTORE_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (fused_small_batch(h, R, max_blocks)) return launch_lookup_gather(h, tokens, offsets, R, max_blocks, flags, dst, block_tables, matched_blocks, block_ids, s);
  FetchLink fl;
  rc = next_fetch_link(h, dst, block_tables, s, &fl);
  if (rc) return rc;
  rc = lookup_impl(h, tokens, offsets, R, max_blocks, flags, matched_blocks, block_ids, fl, s);
  if (rc) return rc;
  return launch_fetch_copies(h, dst, fl.seq, s);
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
  // one descriptor per distinct source block, each with the list of its destinations
  FetchLink fl;
  rc = next_fetch_link(h, dst, block_tables, s, &fl);
  if (rc) return rc;
  fetch_link_kernel<<<grid_for((long long)R * max_blocks, 256, h->sms * 8), 256, 0, s>>>(h->st, block_ids, matched_blocks, R, max_blocks, fl);
  PTS_CHECK_LAUNCH(h);
  return launch_fetch_copies(h, dst, fl.seq, s);
}

static int insert_entry(ptstore_t* h, const int32_t* tokens, const int64_t* offsets, int32_t R, int32_t max_blocks,
                        const ptstore_paged_cache_t* src, const int32_t* block_tables, int32_t* block_ids, int32_t* new_blocks,
                        ptstore_stream_t stream, bool after_lookup) {
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
  const long long total = (long long)R * max_blocks;
  InsertArgs a = {};
  a.tokens = tokens;
  a.offsets = reinterpret_cast<const long long*>(offsets);
  a.R = R; a.max_blocks = max_blocks;
  a.split = split_path(h, R, max_blocks) ? 1 : 0;
  a.keys = h->keys; a.eslot = h->eslot; a.cta_sums = h->cta_sums;
  const int lanes = a.split ? 32 : lanes_for(h, R, max_blocks);
  // the keys of this very batch, left by the last lookup: with a warp per request the chain resumes behind them
  const bool resume = after_lookup && h->lk_valid && lanes == 32 && h->lk_tokens == tokens && h->lk_offsets == offsets && h->lk_R == R &&
                      h->lk_max_blocks == max_blocks;
  a.hashed = resume ? h->prefix : nullptr;
  h->lk_valid = false;                        // this call overwrites the key scratch
  if (resume) h->inserts_resumed += 1;
  a.bt = copy ? block_tables : nullptr;
  a.cache_blocks = copy ? src->num_blocks : 0;
  a.epoch = h->epoch;
  a.desc = h->desc;
  a.ids_out = block_ids; a.new_blocks = new_blocks;
  // CTAs: enough for one element per thread and for one sub-warp per request, at most one per SM
  const long long by_elems = (total + INS_THREADS - 1) / INS_THREADS;
  const long long by_reqs = ((long long)R * lanes + INS_THREADS - 1) / INS_THREADS;
  long long g = by_elems > by_reqs ? by_elems : by_reqs;
  const int grid = (int)(g < 1 ? 1 : (g > h->coop_grid ? h->coop_grid : g));
  switch (lanes) {
    case 4: rc = launch_insert<4>(h, a, grid, s); break;
    case 8: rc = launch_insert<8>(h, a, grid, s); break;
    case 16: rc = launch_insert<16>(h, a, grid, s); break;
    default: rc = launch_insert<32>(h, a, grid, s); break;
  }
  if (rc) return rc;
  if (copy) return launch_copy<COPY_INSERT>(h, to_paged(src), false, s, h->desc, &h->st.ctrl->n_pairs);
  return PTSTORE_OK;
}

int ptstore_insert(ptstore_t* h, const int32_t* tokens, const int64_t* offsets, int32_t R, int32_t max_blocks,
                   const ptstore_paged_cache_t* src, const int32_t* block_tables, int32_t* block_ids, int32_t* new_blocks,
                   ptstore_stream_t stream) {
  return insert_entry(h, tokens, offsets, R, max_blocks, src, block_tables, block_ids, new_blocks, stream, false);
}

int ptstore_insert_after_lookup(ptstore_t* h, const int32_t* tokens, const int64_t* offsets, int32_t R, int32_t max_blocks,
                                const ptstore_paged_cache_t* src, const int32_t* block_tables, int32_t* block_ids, int32_t* new_blocks,
                                ptstore_stream_t stream) {
  return insert_entry(h, tokens, offsets, R, max_blocks, src, block_tables, block_ids, new_blocks, stream, true);
}

uint64_t ptstore_resumed_inserts(const ptstore_t* h) { return h ? h->inserts_resumed : 0; }

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

static int evict_entry(ptstore_t* h, int32_t tier, int32_t n_blocks, int32_t* n_evicted, int32_t* victim_ids, ptstore_stream_t stream, bool async_copy) {
  if (!h || n_blocks < 0 || (tier != PTSTORE_TIER_HBM && tier != PTSTORE_TIER_HOST) || !n_evicted) return PTSTORE_E_INVAL;
  if (tier == PTSTORE_TIER_HOST && h->cfg.host_blocks == 0) return PTSTORE_E_INVAL;
  return evict_impl(h, tier, (u32)n_blocks, -1, nullptr, 0, n_evicted, victim_ids, 0xFFFFFFFFu, static_cast<cudaStream_t>(stream), async_copy);
}

int ptstore_evict(ptstore_t* h, int32_t tier, int32_t n_blocks, int32_t* n_evicted, int32_t* victim_ids, ptstore_stream_t stream) {
  return evict_entry(h, tier, n_blocks, n_evicted, victim_ids, stream, false);
}

int ptstore_evict_async(ptstore_t* h, int32_t tier, int32_t n_blocks, int32_t* n_evicted, int32_t* victim_ids, ptstore_stream_t stream) {
  return evict_entry(h, tier, n_blocks, n_evicted, victim_ids, stream, true);
}

int ptstore_reserve(ptstore_t* h, int64_t want_free, int32_t headroom, const int32_t* minus, int32_t n_minus, uint32_t flags,
                    int32_t* n_evicted, int32_t* victim_ids, int32_t max_victims, ptstore_stream_t stream) {
  if (!h || want_free < 0 || headroom < 0 || n_minus < 0 || (n_minus > 0 && !minus) || !n_evicted || max_victims < 0) return PTSTORE_E_INVAL;
  if ((u32)n_minus > h->cfg.max_requests) return PTSTORE_E_LIMIT;
  const u32 cap = victim_ids ? (u32)max_victims : 0x7FFFFFFFu;
  return evict_impl(h, PTSTORE_TIER_HBM, (u32)headroom, (long long)want_free, minus, n_minus, n_evicted, victim_ids, cap,
                    static_cast<cudaStream_t>(stream), (flags & PTSTORE_ASYNC_COPY) != 0);
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
  return launch_copy<COPY_POOL>(h, none, true, s, h->desc, &h->st.ctrl->n_pairs, h->host_ctas);      // host -> HBM at host-link speed
}

int ptstore_time_next_copy(ptstore_t* h, void* before, void* after) {
  if (!h || !before || !after) return PTSTORE_E_INVAL;
  h->time_before = static_cast<cudaEvent_t>(before);
  h->time_after = static_cast<cudaEvent_t>(after);
  return PTSTORE_OK;
}

int ptstore_set_wait_limit(ptstore_t* h, uint32_t polls) {
  if (!h) return PTSTORE_E_INVAL;
  h->wait_limit = polls ? polls : BULK_POLL_LIMIT;
  return PTSTORE_OK;
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
  out->max_displacement = c.max_disp;
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
  out->far_keys = c.far_keys;
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

#ifdef PTS_PHASE_TIMERS
// diagnostic build only: copies the phase time stamps of the last cooperative kernel to the host (synchronises)
extern "C" int ptstore_debug_phases(ptstore_t* h, uint64_t* out16) {
  cudaDeviceSynchronize();
  return cudaMemcpy(out16, h->st.ctrl->phase_ns, 16 * sizeof(uint64_t), cudaMemcpyDeviceToHost) == cudaSuccess ? 0 : PTSTORE_E_CUDA;
}
#endif

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
