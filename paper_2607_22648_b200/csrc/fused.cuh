// Lookup and gather of a small batch in ONE cooperative launch (the load of the paper, Section 4.1: find the longest
// common prefix, then bring each of its tensors to the GPU pointers the application supplies; what the application waits
// for is the pair, Sections 6.1 and 6.3-6.4: time to first token).
//
// With a handful of long prompts the lookup is one serial hash chain per prompt (tens of microseconds) and the gather a
// copy of a few hundred microseconds; run one after the other, the copy engine idles while the chain runs.  Here the
// first R CTAs look their request up exactly as lookup_long_kernel does and publish, after every chunk of 32 blocks,
// how many blocks have matched so far; every CTA (those R too, once they are done) drives a copy ring and starts on a
// block as soon as its request's progress word says it is matched.  The CTAs of a cooperative launch are all resident,
// so the copiers may wait for the lookups; every wait is bounded (S_TIMEOUT, then drain and return).
//
// Work units - part q of block j of request r - are dealt per request: every request has a counter of units taken (in the
// order of its blocks, so the blocks that match first are copied first), and a copier goes round the requests, one unit
// at a time, dropping a request once its counter has passed the end of what matched.  A batch of one long prompt and
// fifteen that miss therefore costs a copier fifteen wasted counter reads, not fifteen of every sixteen.  Every (request,
// block) entry is copied on its own - no sharing of reads between requests that name the same pool block - which is why
// the host only takes this path for small batches.
#pragma once
#include "common.cuh"
#include "lookup.cuh"
#include "copy.cuh"

namespace pts {

constexpr int FUSED_MAX_REQUESTS = 16;
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
  u64* progress;            // [FUSED_MAX_REQUESTS] progress words
  u32* taken;               // [FUSED_MAX_REQUESTS] units of each request handed out so far; request r's is reset by the CTA
                            // that looks r up, before that CTA's first progress word of this launch
  u32 fetch_seq;            // sequence number of this call among the handle's fetch calls: as in every fetch, the next
                            // call's list scalars are cleared here
  BulkTune tune;
  u32 launch_seq;           // this kernel's own launch count, from 1: the tag of the progress words
};

__global__ void __launch_bounds__(LONG_THREADS) lookup_gather_kernel(Store st, FusedArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) u64 bars[BULK_MAX_STAGES];
  __shared__ unsigned char* s_dst[BULK_MAX_STAGES];
  __shared__ u32 s_bytes[BULK_MAX_STAGES];
  __shared__ int s_m;
  const int lane = threadIdx.x & 31;
  const int R = a.R, max_blocks = a.max_blocks;
  const u32 tag = a.launch_seq;

  if (blockIdx.x == 0 && threadIdx.x == 0) {
    FetchLink seq_only = {};
    seq_only.seq = a.fetch_seq;
    link_prepare_next(st, seq_only);
  }
  // ---- the lookup of request blockIdx.x ---------------------------------------------------------------------------------
  if ((int)blockIdx.x < R) {
    const long long r = blockIdx.x;
    const int nblk = full_blocks(a.offsets, (int)r, st.block_tokens, max_blocks);
    u64* crow = a.scratch + r * max_blocks;
    if (threadIdx.x == 0) a.taken[r] = 0;        // ordered before this thread's release of the first progress word
    {
      const int* t0 = a.tokens + a.offsets[r];
      for (int j = threadIdx.x; j < nblk; j += LONG_THREADS) crow[j] = content_block(t0 + (long long)j * st.block_tokens, st.block_tokens);
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      const int m = chain_probe_request(st, crow, nblk, r, max_blocks, a.flags, a.epoch, a.matched, a.ids_out, a.hashed, a.progress, tag, lane);
      if (lane == 0) {
        s_m = m;
        atomicAdd(&st.ctrl->blocks_fetched[0], (u64)m);
        atomicAdd(&st.ctrl->blocks_fetched_distinct, (u64)m);
      }
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

  // what this copier knows of each request: blocks matched so far, and whether that is final (used by thread 0 only)
  __shared__ int s_known[FUSED_MAX_REQUESTS];
  __shared__ int s_final[FUSED_MAX_REQUESTS];
  for (int r = 0; r < FUSED_MAX_REQUESTS; ++r) { s_known[r] = 0; s_final[r] = 0; }
  bool ok = true;
  // Reads request r's progress word until it covers block j or is final (j < 0: until it carries this launch's tag with
  // something to copy, or is final).  False when the wait ran out.
  auto await = [&](int r, int j) -> bool {
    u32 polls = 0;
    while (true) {
      u64 v;
      asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(a.progress + r) : "memory");
      if ((u32)(v >> 32) == tag) {
        const int kn = (int)(v & 0x7FFFFFFFull);
        const int fin = (v & 0x80000000ull) != 0;
        s_known[r] = kn; s_final[r] = fin;
        if (fin || (j < 0 ? kn > 0 : j < kn)) return true;
      }
      if (++polls >= PROGRESS_POLL_LIMIT) { ok = false; raise(st, S_TIMEOUT); return false; }
      __nanosleep(64);
    }
  };

  // generator of pieces: goes round the requests that may still have units and takes one unit at a time
  u32 alive = R >= 32 ? 0xFFFFFFFFu : ((1u << R) - 1u);
  int cur = (int)(blockIdx.x % (unsigned)R);
  u32 in_unit = 0, unit_pieces = 0, ls = 0, piece = 0;
  const unsigned char* src_block = nullptr;
  u32 dst_block = 0;
  bool exhausted = false;
  auto next_unit = [&]() -> bool {                  // positions the cursor on the next unit that exists
    while (ok && alive) {
      int r = cur;
      while (!((alive >> r) & 1u)) r = r + 1 == R ? 0 : r + 1;
      cur = r + 1 == R ? 0 : r + 1;
      // the counter of r may be touched only after a progress word of this launch has been seen (it is reset before)
      if (s_known[r] == 0 && !s_final[r] && !await(r, -1)) return false;
      if (s_known[r] == 0) { alive &= ~(1u << r); continue; }            // final with nothing matched
      const u32 u = atomicAdd(a.taken + r, 1u);
      const int j = (int)(u / U);
      const u32 q = u - (u32)j * U;
      if (j >= s_known[r] && !s_final[r] && !await(r, j)) return false;
      if (j >= s_known[r]) { alive &= ~(1u << r); continue; }            // final and shorter: nothing left of r
      const long long e = (long long)r * max_blocks + j;
      const int id = __ldcg(a.ids_out + e), cb = a.bt[e];      // ids are written during this launch: not through L1
      if (id < 0 || (u32)id >= st.n[0] || cb < 0 || (u32)cb >= a.pc.num_blocks) {
        if (q == 0) raise(st, S_BOUNDS);
        continue;
      }
      const u32 base_piece = q * G;
      unit_pieces = per_block - base_piece < G ? per_block - base_piece : G;
      in_unit = 0;
      ls = base_piece / ppc;
      piece = base_piece - ls * ppc;
      src_block = st.pool[0] + (u64)(u32)id * st.block_bytes;
      dst_block = (u32)cb;
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
    s_dst[s] = cache_addr(a.pc, ls, dst_block, off);
    s_bytes[s] = bytes;
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
    bulk_s2g(s_dst[s], smem + (size_t)s * SB, s_bytes[s]);
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
