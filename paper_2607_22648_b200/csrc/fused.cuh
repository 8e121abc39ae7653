// Lookup and gather of a small batch in ONE cooperative launch (the load of the paper, Section 4.1: find the longest
// common prefix, then bring each of its tensors to the GPU pointers the application supplies; what the application waits
// for is the pair, Sections 6.1 and 6.3-6.4: time to first token).
//
// With a handful of long prompts the lookup is one serial hash chain per prompt (tens of microseconds) and the gather a
// copy of a few hundred microseconds; run one after the other, the copy engine idles while the chain runs.  Here the
// first R CTAs look their request up exactly as lookup_long_kernel does (warp 0) and publish, after every chunk of 32
// blocks, how many blocks have matched so far; every CTA (those R too, once they are done) drives a copy ring and starts on
// a block as soon as it is known to be matched.  The CTAs of a cooperative launch are all resident, so CTAs may wait for
// one another; every wait is bounded (S_TIMEOUT, then drain and return), and only lookups are ever waited for, which
// themselves wait for nothing.
//
// Prompts of one batch often share a prefix, and a pool block named by several requests should be read once (Section 4:
// shared prefixes are stored once).  A block id is a trie node, so equal ids sit at the same depth j of different
// requests: warp 1 of the CTA that looks request r up follows the progress of ALL requests chunk by chunk, compares
// ids[r][j] with ids[r2][j] and makes r the OWNER of block j unless a lower request names the same block.  It appends the
// owned blocks, each with the set of higher requests that share it, to r's owned list and publishes the list's length.
// Work units - part q of the k-th owned block of request r - are dealt per request from a counter of units taken; a
// copier goes round the requests, one unit at a time, waits until r's owned list covers the unit, and drops a request
// whose counter has passed the end of its list.  A unit is loaded once and stored to every request that shares it.
#pragma once
#include "common.cuh"
#include "lookup.cuh"
#include "copy.cuh"

namespace pts {

constexpr int FUSED_MAX_REQUESTS = 16;
constexpr int FUSED_MAX_BLOCKS = 1 << 16;         // an owned-list entry holds the depth in 16 bits
constexpr u32 PROGRESS_POLL_LIMIT = 1u << 21;

struct FusedArgs {
  const int* tokens;
  const long long* offsets;
  int R, max_blocks;
  u32 flags;
  u64 epoch;
  int* matched;
  int* ids_out;
  u64* scratch;             // content hashes / chained keys [R*max_blocks]
  u32* hashed;
  const int* bt;            // destination block tables
  Paged pc;
  u64* progress;            // [FUSED_MAX_REQUESTS] lookup progress: (launch tag << 32) | (done << 31) | blocks matched
  u64* owned_progress;      // [FUSED_MAX_REQUESTS] the same for the owned lists: entries appended so far
  u32* taken;               // [FUSED_MAX_REQUESTS] units of each request handed out so far; request r's is reset by the warp
                            // that builds r's owned list, before that warp's first owned_progress word of this launch
  u32* owned;               // [R*max_blocks] owned lists: (sharing higher requests, a bit each) << 16 | depth j
  int2* owned_src;          // [R*max_blocks] ... and {pool block, the owner's own destination block} of the same entry, so
                            // that a copier has all it needs for an unshared block after one round of loads
  u32 fetch_seq;            // sequence number of this call among the handle's fetch calls: as in every fetch, the next
                            // call's list scalars are cleared here
  BulkTune tune;
  u32 launch_seq;           // this kernel's own launch count, from 1: the tag of the progress words
};

// All lanes: reads a progress word until it carries `tag` and covers `need` blocks (or entries) or is final.
// Returns false when the wait ran out.  `count` and `fin` are what the word said last (0 / false if it never had the tag).
__device__ __forceinline__ bool await_progress(const u64* word, u32 tag, int need, int& count, bool& fin) {
  u32 polls = 0;
  count = 0; fin = false;
  while (true) {
    u64 v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(word) : "memory");
    if ((u32)(v >> 32) == tag) {
      count = (int)(v & 0x7FFFFFFFull);
      fin = (v & 0x80000000ull) != 0;
      if (fin || count >= need) return true;
    }
    if (++polls >= PROGRESS_POLL_LIMIT) return false;
    __nanosleep(64);
  }
}

// One warp: the owned list of request r (see the head of this file).  Follows the lookups of all requests through their
// progress words; returns the number of owned blocks.
__device__ __forceinline__ int build_owned_list(const Store& st, const FusedArgs& a, int r, u32 tag, int lane) {
  const int R = a.R, max_blocks = a.max_blocks;
  if (lane == 0) a.taken[r] = 0;                  // ordered before this lane's release of the first owned_progress word
  int k = 0;
  bool timed_out = false;
  for (int base = 0;; base += 32) {
    const int j = base + lane;
    const int my_cb = j < max_blocks ? a.bt[(long long)r * max_blocks + j] : -1;   // in flight while the lookups are awaited
    int m_r; bool fin_r;
    if (!await_progress(a.progress + r, tag, base + 32, m_r, fin_r)) { timed_out = true; break; }
    const int lim = m_r < base + 32 ? m_r : base + 32;          // blocks [base, lim) of r are matched and not yet listed
    const bool active = j < lim;
    const int my_id = active ? __ldcg(a.ids_out + (long long)r * max_blocks + j) : -1;
    bool lower = false;
    u32 sharers = 0;
    for (int r2 = 0; r2 < R && lim > base; ++r2) {
      if (r2 == r) continue;
      int m2; bool fin2;
      if (!await_progress(a.progress + r2, tag, lim, m2, fin2)) { timed_out = true; break; }
      const int other = (active && j < m2) ? __ldcg(a.ids_out + (long long)r2 * max_blocks + j) : -2;
      if (other == my_id) { if (r2 < r) lower = true; else sharers |= 1u << r2; }
    }
    if (timed_out) break;
    const bool own = active && !lower;
    const unsigned om = __ballot_sync(FULL, own);
    if (own) {
      const long long at = (long long)r * max_blocks + k + __popc(om & ((1u << lane) - 1u));
      a.owned[at] = (sharers << 16) | (u32)j;
      a.owned_src[at] = make_int2(my_id, my_cb);
    }
    k += __popc(om);
    const bool last = fin_r && lim == m_r;
    __syncwarp();
    if (lane == 0 && (om || last)) { __threadfence(); publish_progress(a.owned_progress, r, tag, (u32)k, last); }
    if (last) break;
  }
  if (timed_out) {                                 // let the copiers finish with what is listed
    if (lane == 0) { raise(st, S_TIMEOUT); __threadfence(); publish_progress(a.owned_progress, r, tag, (u32)k, true); }
  }
  if (lane == 0 && k) atomicAdd(&st.ctrl->blocks_fetched_distinct, (u64)k);
  return k;
}

__global__ void __launch_bounds__(LONG_THREADS) lookup_gather_kernel(Store st, FusedArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) u64 bars[BULK_MAX_STAGES];
  __shared__ u32 s_bytes[BULK_MAX_STAGES], s_n[BULK_MAX_STAGES];
  __shared__ unsigned char* s_plane[BULK_MAX_STAGES];              // address of the piece in cache block 0 of its plane
  __shared__ u32 s_blk[BULK_MAX_STAGES][FUSED_MAX_REQUESTS];      // destination cache blocks of the piece in each stage
  __shared__ u32 s_unit_blk[FUSED_MAX_REQUESTS];                   // ... of the unit being loaded
  __shared__ int s_known[FUSED_MAX_REQUESTS], s_final[FUSED_MAX_REQUESTS];
  __shared__ int s_m;
  const int lane = threadIdx.x & 31;
  const int R = a.R, max_blocks = a.max_blocks;
  const u32 tag = a.launch_seq;

  if (blockIdx.x == 0 && threadIdx.x == 0) {
    FetchLink seq_only = {};
    seq_only.seq = a.fetch_seq;
    link_prepare_next(st, seq_only);
  }
  // ---- the lookup of request blockIdx.x (warp 0) and its owned list (warp 1) -----------------------------------------
  if ((int)blockIdx.x < R) {
    const long long r = blockIdx.x;
    const int nblk = full_blocks(a.offsets, (int)r, st.block_tokens, max_blocks);
    u64* crow = a.scratch + r * max_blocks;
    {
      const int* t0 = a.tokens + a.offsets[r];
      for (int j = threadIdx.x; j < nblk; j += LONG_THREADS) crow[j] = content_block(t0 + (long long)j * st.block_tokens, st.block_tokens);
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      if (R == 1 && lane == 0) a.taken[0] = 0;       // a single request owns all it matches: the copiers follow the lookup itself
      const int m = chain_probe_request(st, crow, nblk, r, max_blocks, a.flags, a.epoch, a.matched, a.ids_out, a.hashed, a.progress, tag, lane);
      if (lane == 0) {
        s_m = m;
        if (m) atomicAdd(&st.ctrl->blocks_fetched[0], (u64)m);
        if (m && R == 1) atomicAdd(&st.ctrl->blocks_fetched_distinct, (u64)m);
      }
    } else if (threadIdx.x < 64 && R > 1) {
      build_owned_list(st, a, (int)r, tag, lane);
    }
    __syncthreads();
    const int m = s_m;
    for (int j = m + threadIdx.x; j < max_blocks; j += LONG_THREADS) a.ids_out[r * max_blocks + j] = -1;
  }
  if (threadIdx.x != 0) return;

  // ---- the copy ring, driven by one thread ----------------------------------------------------------------------------
  const int STAGES = a.tune.stages;
  const u32 SB = (u32)a.tune.stage_bytes;
  const u32 chunk = (u32)st.chunk_bytes;
  const u32 ppc = (chunk + SB - 1) / SB;
  const u32 per_block = 2u * st.layers * ppc;                      // pieces of one block
  const u32 G = (u32)a.tune.group < per_block ? (u32)a.tune.group : per_block;
  const u32 U = (per_block + G - 1) / G;                           // units per block
  for (int s = 0; s < STAGES; ++s) mbar_init(&bars[s], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  fence_async_smem();

  // what this copier knows of each request's owned list: entries so far, and whether that is final
  for (int r = 0; r < FUSED_MAX_REQUESTS; ++r) { s_known[r] = 0; s_final[r] = 0; }
  bool ok = true;
  auto await_owned = [&](int r, int need) -> bool {          // false when the wait ran out
    int count; bool fin;
    const bool got = await_progress((R == 1 ? a.progress : a.owned_progress) + r, tag, need, count, fin);
    s_known[r] = count; s_final[r] = fin ? 1 : 0;
    if (!got) { ok = false; raise(st, S_TIMEOUT); }
    return got;
  };

  // generator of pieces: goes round the requests that may still have units and takes one unit at a time
  u32 alive = (1u << R) - 1u;
  int cur = (int)(blockIdx.x % (unsigned)R);
  u32 in_unit = 0, unit_pieces = 0, unit_n = 0, ls = 0, piece = 0;
  const unsigned char* src_block = nullptr;
  bool exhausted = false;
  auto next_unit = [&]() -> bool {                  // positions the cursor on the next unit that exists
    while (ok && alive) {
      int r = cur;
      while (!((alive >> r) & 1u)) r = r + 1 == R ? 0 : r + 1;
      cur = r + 1 == R ? 0 : r + 1;
      // the counter of r may be touched only after an owned_progress word of this launch has been seen (it is reset before)
      if (s_known[r] == 0 && !s_final[r] && !await_owned(r, 1)) return false;
      if (s_known[r] == 0) { alive &= ~(1u << r); continue; }            // final with nothing owned
      const u32 u = atomicAdd(a.taken + r, 1u);
      const int k = (int)(u / U);
      const u32 q = u - (u32)k * U;
      if (k >= s_known[r] && !s_final[r] && !await_owned(r, k + 1)) return false;
      if (k >= s_known[r]) { alive &= ~(1u << r); continue; }            // final and shorter: nothing left of r
      u32 w;
      int2 src;
      if (R == 1) {                                                       // the k-th matched block, owned, unshared
        w = (u32)k;
        src = make_int2(__ldcg(a.ids_out + k), a.bt[k]);
      } else {
        w = __ldcg(a.owned + (long long)r * max_blocks + k);              // lists are written during this launch: not
        src = __ldcg(a.owned_src + (long long)r * max_blocks + k);        // through L1
      }
      const int j = (int)(w & 0xFFFFu);
      const int id = src.x;
      if (id < 0 || (u32)id >= st.n[0]) { if (q == 0) raise(st, S_BOUNDS); continue; }
      u32 n = 0, bad = 0;
      if (src.y < 0 || (u32)src.y >= a.pc.num_blocks) ++bad;
      else s_unit_blk[n++] = (u32)src.y;
      for (u32 set = w >> 16; set; set &= set - 1) {                      // the higher requests that share the block
        const int r2 = __ffs(set) - 1;
        const int cb = a.bt[(long long)r2 * max_blocks + j];
        if (cb < 0 || (u32)cb >= a.pc.num_blocks) ++bad;
        else s_unit_blk[n++] = (u32)cb;
      }
      if (bad && q == 0) {                         // once per block: flag it, and take the skipped entries out of the count
        raise(st, S_BOUNDS);
        atomicAdd(&st.ctrl->blocks_fetched[0], 0ull - (u64)bad);
      }
      if (n == 0) continue;
      unit_n = n;
      const u32 base_piece = q * G;
      unit_pieces = per_block - base_piece < G ? per_block - base_piece : G;
      in_unit = 0;
      ls = base_piece / ppc;
      piece = base_piece - ls * ppc;
      src_block = st.pool[0] + (u64)(u32)id * st.block_bytes;
      return true;
    }
    return false;
  };
  auto issue_load = [&](int s) -> bool {
    if (in_unit == unit_pieces) {
      if (exhausted || !next_unit()) { exhausted = true; return false; }
    }
    const u32 off = piece * SB;
    const u32 left = chunk - off;
    const u32 bytes = left < SB ? left : SB;
    s_plane[s] = cache_addr(a.pc, ls, 0, off); s_bytes[s] = bytes; s_n[s] = unit_n;
    for (u32 i = 0; i < unit_n; ++i) s_blk[s][i] = s_unit_blk[i];
    mbar_expect_tx(&bars[s], bytes);
    bulk_g2s(smem + (size_t)s * SB, src_block + (u64)ls * chunk + off, bytes, &bars[s]);
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
  while (stored < issued) {
    if (!mbar_wait_bounded(&bars[s], parity, a.tune.wait_limit)) { ok = false; raise(st, S_TIMEOUT); break; }
    for (u32 i = 0; i < s_n[s]; ++i) bulk_s2g(s_plane[s] + (u64)s_blk[s][i] * a.pc.block_stride, smem + (size_t)s * SB, s_bytes[s]);
    bulk_commit();
    ++stored;
    if (!exhausted && ok) {
      bulk_wait_read<1>();                       // the stage of the previous piece has been read out
      if (issue_load(load_stage)) { ++issued; load_stage = load_stage + 1 == STAGES ? 0 : load_stage + 1; }
    }
    if (++s == STAGES) { s = 0; parity ^= 1u; }
  }
  if (stored < issued) {                         // gave up: drain loads in flight (bounded)
    for (u64 k = stored; k < issued; ++k) {
      mbar_wait_bounded(&bars[s], parity, BULK_POLL_LIMIT);
      if (++s == STAGES) { s = 0; parity ^= 1u; }
    }
  }
  bulk_wait_all();
}

}  // namespace pts
