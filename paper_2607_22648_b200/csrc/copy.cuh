// Copy engine: moves chunks between the store pool and a vLLM-style paged cache (load / store of
// tensors through application-supplied pointers, paper Section 4.1), or between two pool blocks
// (flush of owned tensors to a slower tier, Section 4.1 "Access pattern-aware eviction policy").
//
// The paper moves all scattered (offset,size) segments of a request "in parallel in a single RDMA RPC"
// without packing them first (Section 4.1 "RDMA-aware consolidation").  The analogue here is ONE
// kernel launch over a descriptor list {pool block, cache block}: no staging buffer, every chunk is
// contiguous on both sides, and a pool block is one contiguous region.
//
// Two engines:
//   vector: every thread moves 16-byte pieces with several independent loads in flight; works for any
//           device-visible memory (also mapped pinned host memory).
//   bulk  : one elected thread per CTA drives bulk-async copies global -> shared -> global through a
//           ring of shared-memory stages tracked by mbarriers; HBM to HBM only.
// Pure data movement: bounded by HBM bandwidth (or by the host link for the host tier); algorithmic
// bytes per pool block moved = 2 * block_bytes (read once, write once).
#pragma once
#include "common.cuh"

namespace pts {

struct Paged {                 // device view of ptstore_paged_cache_t
  unsigned char* const* layer_base;
  u64 kv_stride, block_stride;
  u32 num_blocks;
  // COPY_FETCH_MULTI only: destination lists, one per distinct source block
  const u64* head = nullptr;   // low half of head[block id] = first node of the block's list (the block is in the
                               // descriptor list, so the head was written by this call)
  const int2* node = nullptr;  // node[e] = {next node or LINK_NIL, cache block}
};

// COPY_FETCH_MULTI: a batch of prompts over popular documents names the same pool block many times (a block is
// a trie node, so equal ids always sit at the same depth of different requests).  Descriptors are then one per
// DISTINCT source block; a piece is read once and written to every destination of the block's list, which
// removes the repeated reads from DRAM (on the bench workload only ~40 % of the fetched blocks are distinct).
enum CopyMode { COPY_FETCH = 0, COPY_INSERT = 1, COPY_POOL = 2, COPY_FETCH_MULTI = 3 };

__device__ __forceinline__ unsigned char* cache_addr(const Paged& pc, u32 ls, u32 cache_block, u64 off) {
  return pc.layer_base[ls >> 1] + (u64)(ls & 1) * pc.kv_stride + (u64)cache_block * pc.block_stride + off;
}

// address of piece (ls, off) on both sides of descriptor d
template <int MODE>
__device__ __forceinline__ void piece_addr(const Store& st, const Paged& pc, int2 d, u32 ls, u64 off,
                                           const unsigned char*& src, unsigned char*& dst) {
  unsigned char* pool_side = block_ptr(st, (u32)d.x) + (u64)ls * st.chunk_bytes + off;
  if (MODE == COPY_FETCH_MULTI) {
    src = pool_side;
    dst = nullptr;                       // destinations come from the block's list
  } else if (MODE == COPY_POOL) {
    src = pool_side;
    dst = block_ptr(st, (u32)d.y) + (u64)ls * st.chunk_bytes + off;
  } else {
    unsigned char* cache_side = cache_addr(pc, ls, (u32)d.y, off);
    if (MODE == COPY_FETCH) { src = pool_side; dst = cache_side; }
    else { src = cache_side; dst = pool_side; }
  }
}

__device__ __forceinline__ uint4 ld_stream(const unsigned char* p) {
  uint4 v;
  asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(unsigned char* p, uint4 v) {
  asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// ---- vector engine ------------------------------------------------------------------------------------
// A CTA of THREADS threads moves one piece of THREADS*16*UNROLL bytes per iteration; consecutive CTAs take
// consecutive pieces, so a pool block is read (or written) front to back by neighbouring CTAs.
template <int MODE, int THREADS, int UNROLL>
__global__ void __launch_bounds__(THREADS) copy_vector_kernel(Store st, Paged pc, const int2* __restrict__ desc,
                                                              const u32* __restrict__ n_pairs_ptr) {
  constexpr u64 PIECE = (u64)THREADS * 16 * UNROLL;
  const u32 n_pairs = *n_pairs_ptr;
  const u32 ppc = (u32)((st.chunk_bytes + PIECE - 1) / PIECE);       // pieces per chunk
  const u64 per_pair = (u64)2 * st.layers * ppc;
  const u64 total = (u64)n_pairs * per_pair;
  for (u64 u = blockIdx.x; u < total; u += gridDim.x) {
    const u32 pair = (u32)(u / per_pair);
    const u32 rem = (u32)(u % per_pair);
    const u32 ls = rem / ppc, piece = rem % ppc;
    const int2 d = desc[pair];
    if (d.x < 0) continue;
    const u64 off = (u64)piece * PIECE;
    const unsigned char* src;
    unsigned char* dst;
    piece_addr<MODE>(st, pc, d, ls, off, src, dst);
    const u64 left = st.chunk_bytes - off;                           // bytes of this chunk from `off` on
    uint4 v[UNROLL];
#pragma unroll
    for (int k = 0; k < UNROLL; ++k) {
      const u64 o = ((u64)k * THREADS + threadIdx.x) * 16;
      if (o < left) v[k] = ld_stream(src + o);
    }
    if (MODE == COPY_FETCH_MULTI) {
      u32 e = (u32)pc.head[d.x];
      for (u32 guard = 0; e != LINK_NIL && guard < 0x7FFFFFFFu; ++guard) {      // every thread walks the same list
        const int2 nd = pc.node[e];
        unsigned char* to = cache_addr(pc, ls, (u32)nd.y, off);
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) {
          const u64 o = ((u64)k * THREADS + threadIdx.x) * 16;
          if (o < left) st_stream(to + o, v[k]);
        }
        e = (u32)nd.x;
      }
    } else {
#pragma unroll
      for (int k = 0; k < UNROLL; ++k) {
        const u64 o = ((u64)k * THREADS + threadIdx.x) * 16;
        if (o < left) st_stream(dst + o, v[k]);
      }
    }
  }
}

// ---- bulk engine --------------------------------------------------------------------------------------
__device__ __forceinline__ u32 smem_u32(const void* p) { return (u32)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(u64* bar, u32 count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(u64* bar, u32 bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(u64* bar, u32 parity) {
  u32 ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(u64* bar, u32 parity) {
  u32 ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// bounded wait: gives up after `limit` polls and reports false.  A poll may suspend the thread for a short,
// hardware-defined time; a limit of 1 is a single test that does not suspend at all.
__device__ __forceinline__ bool mbar_wait_bounded(u64* bar, u32 parity, u32 limit) {
  if (limit <= 1) return mbar_test_wait(bar, parity);
  for (u32 i = 0; i < limit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gsrc, u32 bytes, u64* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_s2g(void* gdst, const void* smem_src, u32 bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

constexpr u32 BULK_POLL_LIMIT = 1u << 22;   // polls per wait before the kernel gives up (each poll may suspend briefly)
constexpr int BULK_MAX_STAGES = 32;

struct BulkTune {
  int stages;        // ring depth
  int stage_bytes;   // bytes per stage (multiple of 16)
  int group;         // consecutive pieces a CTA takes before striding to its next group
  int hint;          // 1: mark loads and stores evict-first in L2
  u32 wait_limit;    // polls per wait for a load in the main loop before the CTA gives up (draining keeps BULK_POLL_LIMIT)
};

__device__ __forceinline__ u64 l2_evict_first_policy() {
  u64 p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void bulk_g2s_hint(void* smem_dst, const void* gsrc, u32 bytes, u64* bar, u64 policy) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(policy) : "memory");
}
__device__ __forceinline__ void bulk_s2g_hint(void* gdst, const void* smem_src, u32 bytes, u64 policy) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
               ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes), "l"(policy) : "memory");
}

// One warp per CTA; lane 0 runs the whole pipeline over a ring of `stages` shared-memory stages.
// The pieces of the launch are dealt to CTAs in groups of `group` consecutive pieces.  The load of piece
// i+stages-1 is issued once the store of piece i-1 has finished reading its stage, so stages-1 loads are
// in flight per CTA.  Every wait is bounded; on expiry the CTA raises S_TIMEOUT, drains and returns.
// The issuing thread is the only instruction stream of the SM, so its per-piece work is kept short: the
// piece index is decomposed incrementally (no 64-bit divisions in the loop) and each piece is resolved
// once, at load time; its destination and size wait in a small shared-memory ring for the store.
struct PieceCursor {       // walks the pieces of one CTA in order
  u32 pair, rem;           // piece u = pair * per_pair + rem
  u32 in_group;            // position inside the current group
  u32 per_pair, group;
  u32 step_div, step_mod;  // (grid - 1) * group + 1 decomposed by per_pair: jump to the CTA's next group
  __device__ __forceinline__ void advance() {
    u32 add_div = 0, add_mod = 1;
    if (++in_group == group) { in_group = 0; add_div = step_div; add_mod = step_mod; }
    rem += add_mod;
    pair += add_div;
    if (rem >= per_pair) { rem -= per_pair; pair += 1; }
  }
};

template <int MODE>
__global__ void __launch_bounds__(32) copy_bulk_kernel(Store st, Paged pc, const int2* __restrict__ desc,
                                                       const u32* __restrict__ n_pairs_ptr, BulkTune tune) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) u64 bars[BULK_MAX_STAGES];
  __shared__ unsigned char* s_dst[BULK_MAX_STAGES];
  __shared__ u32 s_bytes[BULK_MAX_STAGES];
  // COPY_FETCH_MULTI: the first BULK_DST_CACHE destinations of the piece in each stage, resolved at load time while
  // the load is in flight; longer lists continue from s_more at store time
  constexpr int BULK_DST_CACHE = MODE == COPY_FETCH_MULTI ? 8 : 1;
  __shared__ unsigned char* s_multi[MODE == COPY_FETCH_MULTI ? BULK_MAX_STAGES : 1][BULK_DST_CACHE];
  __shared__ u32 s_ndst[BULK_MAX_STAGES], s_more[BULK_MAX_STAGES], s_ls[BULK_MAX_STAGES], s_off[BULK_MAX_STAGES];
  if (threadIdx.x != 0) return;
  const int STAGES = tune.stages;
  const u32 SB = (u32)tune.stage_bytes;
  const u32 G = (u32)tune.group;
  const u32 n_pairs = *n_pairs_ptr;
  const u32 ppc = (u32)((st.chunk_bytes + SB - 1) / SB);
  const u32 per_pair = 2u * st.layers * ppc;
  const u64 total = (u64)n_pairs * per_pair;
  // pieces of this CTA: groups blockIdx, blockIdx+grid, ... of G pieces each
  const u64 n_groups = (total + G - 1) / G;
  if (blockIdx.x >= n_groups) return;
  const u64 my_groups = (n_groups - blockIdx.x + gridDim.x - 1) / gridDim.x;
  u64 mine = my_groups * G;
  {   // the very last group of the launch may be short
    const u64 last_group = blockIdx.x + (my_groups - 1) * gridDim.x;
    if (last_group == n_groups - 1) mine -= n_groups * G - total;
  }
  const u64 policy = tune.hint ? l2_evict_first_policy() : 0;
  const u32 chunk = (u32)st.chunk_bytes;

  for (int s = 0; s < STAGES; ++s) mbar_init(&bars[s], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  fence_async_smem();

  PieceCursor cur;
  {
    const u64 first = (u64)blockIdx.x * G;
    const u64 step = (u64)(gridDim.x - 1) * G + 1;
    cur.pair = (u32)(first / per_pair); cur.rem = (u32)(first % per_pair);
    cur.in_group = 0; cur.per_pair = per_pair; cur.group = G;
    cur.step_div = (u32)(step / per_pair); cur.step_mod = (u32)(step % per_pair);
  }
  // issue the load of the piece under the cursor into stage s, remember where it goes, move the cursor on
  auto issue_load = [&](int s) {
    const int2 d = desc[cur.pair];
    const u32 ls = cur.rem / ppc, piece = cur.rem - ls * ppc;
    cur.advance();
    if (d.x < 0) {                               // skipped descriptor: complete the phase with no bytes
      s_bytes[s] = 0;
      mbar_expect_tx(&bars[s], 0);
      return;
    }
    const u32 off = piece * SB;
    const unsigned char* src; unsigned char* dst;
    piece_addr<MODE>(st, pc, d, ls, off, src, dst);
    const u32 left = chunk - off;
    const u32 bytes = left < SB ? left : SB;
    s_dst[s] = dst;
    s_bytes[s] = bytes;
    mbar_expect_tx(&bars[s], bytes);
    if (tune.hint) bulk_g2s_hint(smem + (size_t)s * SB, src, bytes, &bars[s], policy);
    else bulk_g2s(smem + (size_t)s * SB, src, bytes, &bars[s]);
    if (MODE == COPY_FETCH_MULTI) {              // resolve destinations while the load flies
      u32 e = (u32)pc.head[d.x];
      u32 n = 0;
      while (e != LINK_NIL && n < (u32)BULK_DST_CACHE) {
        const int2 nd = pc.node[e];
        s_multi[s][n++] = cache_addr(pc, ls, (u32)nd.y, off);
        e = (u32)nd.x;
      }
      s_ndst[s] = n; s_more[s] = e; s_ls[s] = ls; s_off[s] = off;
    }
  };

  const u64 pre = mine < (u64)(STAGES - 1) ? mine : (u64)(STAGES - 1);
  u64 issued = 0;
  int ls_stage = 0;                              // stage the next load goes to
  for (; issued < pre; ++issued) { issue_load(ls_stage); ls_stage = ls_stage + 1 == STAGES ? 0 : ls_stage + 1; }
  bool ok = true;
  int s = 0;                                     // stage of piece i
  u32 parity = 0;
  u64 i = 0;
  for (; i < mine; ++i) {
    if (!mbar_wait_bounded(&bars[s], parity, tune.wait_limit)) { ok = false; break; }
    const u32 bytes = s_bytes[s];
    if (bytes) {
      if (MODE == COPY_FETCH_MULTI) {
        const u32 n = s_ndst[s];
        for (u32 k = 0; k < n; ++k) bulk_s2g(s_multi[s][k], smem + (size_t)s * SB, bytes);
        u32 e = s_more[s];
        for (u32 guard = 0; e != LINK_NIL && guard < 0x7FFFFFFFu; ++guard) {
          const int2 nd = pc.node[e];
          bulk_s2g(cache_addr(pc, s_ls[s], (u32)nd.y, s_off[s]), smem + (size_t)s * SB, bytes);
          e = (u32)nd.x;
        }
      } else if (tune.hint) bulk_s2g_hint(s_dst[s], smem + (size_t)s * SB, bytes, policy);
      else bulk_s2g(s_dst[s], smem + (size_t)s * SB, bytes);
    }
    bulk_commit();
    // the stage of piece i-1 is free once its store has read it: at most one newer group may be pending
    if (issued < mine) {
      bulk_wait_read<1>();
      issue_load(ls_stage);
      ls_stage = ls_stage + 1 == STAGES ? 0 : ls_stage + 1;
      ++issued;
    }
    if (++s == STAGES) { s = 0; parity ^= 1u; }
  }
  if (!ok) {
    raise(st, S_TIMEOUT);
    // drain loads already issued (bounded), so no copy lands in shared memory after exit
    for (u64 k = i; k < issued; ++k) {
      mbar_wait_bounded(&bars[s], parity, BULK_POLL_LIMIT);
      if (++s == STAGES) { s = 0; parity ^= 1u; }
    }
  }
  bulk_wait_all();
}

// ---- bulk engine, one read and many writes per piece (COPY_FETCH_MULTI) --------------------------------------------
// Same ring as copy_bulk_kernel, two differences.  (1) Work is dealt dynamically: a unit is `group` consecutive
// pieces of one source block, taken from an atomic counter, because units now differ in cost (one read plus one
// write per destination).  (2) The destination list of the unit's source block is walked once per unit into a
// small shared-memory record, so the per-piece work of the issuing thread stays free of dependent global loads.
constexpr int MULTI_KMAX = 16;                       // destinations cached per record; longer lists continue in global memory
constexpr int MULTI_NREC = BULK_MAX_STAGES + 1;      // every piece in flight may belong to a different unit

__global__ void __launch_bounds__(32) copy_bulk_multi_kernel(Store st, Paged pc, const int2* __restrict__ desc,
                                                             const u32* __restrict__ n_pairs_ptr, u32* __restrict__ work_counter,
                                                             BulkTune tune) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) u64 bars[BULK_MAX_STAGES];
  __shared__ u32 s_rec[BULK_MAX_STAGES], s_ls[BULK_MAX_STAGES], s_off[BULK_MAX_STAGES], s_bytes[BULK_MAX_STAGES];
  __shared__ const unsigned char* rec_src[MULTI_NREC];
  __shared__ u32 rec_n[MULTI_NREC], rec_more[MULTI_NREC];
  __shared__ u32 rec_dst[MULTI_NREC][MULTI_KMAX];
  if (threadIdx.x != 0) return;
  const int STAGES = tune.stages;
  const u32 SB = (u32)tune.stage_bytes;
  const u32 n_pairs = *n_pairs_ptr;
  const u32 chunk = (u32)st.chunk_bytes;
  const u32 ppc = (chunk + SB - 1) / SB;
  const u32 per_pair = 2u * st.layers * ppc;
  const u32 G = (u32)tune.group < per_pair ? (u32)tune.group : per_pair;
  const u32 units_per_pair = (per_pair + G - 1) / G;
  const u64 total_units = (u64)n_pairs * units_per_pair;

  for (int s = 0; s < STAGES; ++s) mbar_init(&bars[s], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  fence_async_smem();

  // cursor over the pieces of the current unit
  u32 rec = 0, unit_pieces = 0, in_unit = 0, ls = 0, piece = 0;
  bool exhausted = false;
  auto grab = [&]() {
    const u64 w = (u64)atomicAdd(work_counter, 1u);
    if (w >= total_units) { exhausted = true; return; }
    const u32 pair = (u32)(w / units_per_pair), sub = (u32)(w % units_per_pair);
    const u32 base_piece = sub * G;
    unit_pieces = per_pair - base_piece < G ? per_pair - base_piece : G;
    in_unit = 0;
    ls = base_piece / ppc;
    piece = base_piece - ls * ppc;
    rec = rec + 1 == (u32)MULTI_NREC ? 0 : rec + 1;
    const u32 id = (u32)desc[pair].x;
    rec_src[rec] = block_ptr(st, id);
    u32 e = (u32)pc.head[id], n = 0;
    while (e != LINK_NIL && n < (u32)MULTI_KMAX) {
      const int2 nd = pc.node[e];
      rec_dst[rec][n++] = (u32)nd.y;
      e = (u32)nd.x;
    }
    rec_n[rec] = n;
    rec_more[rec] = e;
  };
  auto issue_load = [&](int s) -> bool {
    if (in_unit == unit_pieces) {
      grab();
      if (exhausted) return false;
    }
    const u32 off = piece * SB;
    const u32 left = chunk - off;
    const u32 bytes = left < SB ? left : SB;
    s_rec[s] = rec; s_ls[s] = ls; s_off[s] = off; s_bytes[s] = bytes;
    mbar_expect_tx(&bars[s], bytes);
    bulk_g2s(smem + (size_t)s * SB, rec_src[rec] + (u64)ls * chunk + off, bytes, &bars[s]);
    ++in_unit;
    if (++piece == ppc) { piece = 0; ++ls; }
    return true;
  };

  u64 issued = 0, stored = 0;
  int load_stage = 0;
  for (int k = 0; k < STAGES - 1 && !exhausted; ++k)
    if (issue_load(load_stage)) { ++issued; load_stage = load_stage + 1 == STAGES ? 0 : load_stage + 1; }
  int s = 0;
  u32 parity = 0;
  bool ok = true;
  while (stored < issued) {
    if (!mbar_wait_bounded(&bars[s], parity, tune.wait_limit)) { ok = false; break; }
    const u32 r = s_rec[s], lsx = s_ls[s], off = s_off[s], bytes = s_bytes[s];
    unsigned char* base = pc.layer_base[lsx >> 1] + (u64)(lsx & 1) * pc.kv_stride + off;
    const unsigned char* from = smem + (size_t)s * SB;
    const u32 n = rec_n[r];
    for (u32 k = 0; k < n; ++k) bulk_s2g(base + (u64)rec_dst[r][k] * pc.block_stride, from, bytes);
    u32 e = rec_more[r];
    for (u32 guard = 0; e != LINK_NIL && guard < 0x7FFFFFFFu; ++guard) {
      const int2 nd = pc.node[e];
      bulk_s2g(base + (u64)(u32)nd.y * pc.block_stride, from, bytes);
      e = (u32)nd.x;
    }
    bulk_commit();
    ++stored;
    if (!exhausted) {
      bulk_wait_read<1>();                       // the stage of the previous piece has been read out
      if (issue_load(load_stage)) { ++issued; load_stage = load_stage + 1 == STAGES ? 0 : load_stage + 1; }
    }
    if (++s == STAGES) { s = 0; parity ^= 1u; }
  }
  if (!ok) {
    raise(st, S_TIMEOUT);
    for (u64 k = stored; k < issued; ++k) {      // drain loads in flight (bounded)
      mbar_wait_bounded(&bars[s], parity, BULK_POLL_LIMIT);
      if (++s == STAGES) { s = 0; parity ^= 1u; }
    }
  }
  bulk_wait_all();
}

// ---- descriptor lists -----------------------------------------------------------------------------------
// prefix[r] = sum of min(matched[r'], max_blocks) for r' < r; prefix[R] = total, also stored in ctrl->n_pairs.
__global__ void __launch_bounds__(1024) scan_matched_kernel(Store st, const int* __restrict__ matched, int R, int max_blocks,
                                                            u32* __restrict__ prefix) {
  __shared__ u32 warp_sums[32];
  __shared__ u32 carry;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (int base = 0; base < R; base += 1024) {
    const int r = base + threadIdx.x;
    int mr = r < R ? matched[r] : 0;
    mr = mr < 0 ? 0 : (mr > max_blocks ? max_blocks : mr);
    u32 x = (u32)mr;
    for (int o = 1; o < 32; o <<= 1) { u32 y = __shfl_up_sync(FULL, x, o); if (lane >= o) x += y; }
    if (lane == 31) warp_sums[wid] = x;
    __syncthreads();
    if (wid == 0) {
      u32 w = warp_sums[lane];
      for (int o = 1; o < 32; o <<= 1) { u32 y = __shfl_up_sync(FULL, w, o); if (lane >= o) w += y; }
      warp_sums[lane] = w;
    }
    __syncthreads();
    const u32 incl = x + (wid ? warp_sums[wid - 1] : 0) + carry;
    if (r < R) prefix[r] = incl - (u32)mr;
    __syncthreads();
    if (threadIdx.x == 1023) carry = incl;
    __syncthreads();
  }
  if (threadIdx.x == 0) { prefix[R] = carry; st.ctrl->n_pairs = carry; }
}

// desc[prefix[r] + j] = {pool block, cache block} for j < matched[r]; bad entries become {-1,-1}
__global__ void __launch_bounds__(256) build_pairs_kernel(Store st, const int* __restrict__ ids, const int* __restrict__ matched,
                                                          const int* __restrict__ bt, int R, int max_blocks, u32 cache_blocks,
                                                          const u32* __restrict__ prefix, int2* __restrict__ desc) {
  const long long total = (long long)R * max_blocks;
  u32 cnt0 = 0, cnt1 = 0;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    const int r = (int)(e / max_blocks), j = (int)(e % max_blocks);
    int mr = matched[r];
    mr = mr > max_blocks ? max_blocks : mr;
    if (j >= mr) continue;
    const int id = ids[e], cb = bt[e];
    int2 d;
    if (id < 0 || (u32)id >= st.n[0] + st.n[1] || cb < 0 || (u32)cb >= cache_blocks) {
      raise(st, S_BOUNDS);
      d = make_int2(-1, -1);
    } else {
      d = make_int2(id, cb);
      if ((u32)id < st.n[0]) ++cnt0; else ++cnt1;
    }
    desc[prefix[r] + j] = d;
  }
  cnt0 = __reduce_add_sync(FULL, cnt0);
  cnt1 = __reduce_add_sync(FULL, cnt1);
  if ((threadIdx.x & 31) == 0) {
    if (cnt0) atomicAdd(&st.ctrl->blocks_fetched[0], (u64)cnt0);
    if (cnt1) atomicAdd(&st.ctrl->blocks_fetched[1], (u64)cnt1);
  }
}

}  // namespace pts
