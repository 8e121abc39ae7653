// Hash kernel and batched longest-common-prefix lookup (one-shot LCP query, paper Section 1
// contributions and Section 4.1 "Co-optimized compact metadata and fast prefix queries").
//
// Mapping: a sub-warp of L lanes owns one request and walks it in chunks of L blocks; a warp holds
// 32/L requests.  Per chunk: every lane hashes the tokens of its block (independent), the chained keys
// are produced by a short serial scan over the sub-warp, every lane probes its key, and the ballot of
// the "found" flags gives the first miss, which ends the request.  Lanes of different requests that
// hold the same key (hot documents) are grouped with __match_any_sync so that one lane probes for the
// group; pins are merged the same way into one atomicAdd per distinct block.
#pragma once
#include "common.cuh"

namespace pts {

// chained keys of one chunk of L blocks for each sub-warp.  `parent` is uniform inside a sub-warp,
// `c` the content hash of the lane's block.  steps = warp-uniform number of chain steps needed.
template <int L>
__device__ __forceinline__ u64 chain_chunk(u64& parent, u64 c, int lane, int steps) {
  const int sl = lane & (L - 1), base_lane = lane & ~(L - 1);
  u64 mine = 0;
  // the chain itself is serial (three dependent 64-bit multiplies per step); the shuffle that brings the next
  // block's content hash is issued one step ahead so that its latency hides behind the arithmetic.  The remap of
  // the reserved keys is kept off the dependent path: with x the un-remapped value, fix(x) * C1 = x * C1 + (x < 2 ?
  // 2 * C1 : 0), so the multiply starts as soon as x exists and the compare runs beside it.
  u64 x = parent;                                  // parent is a finished key (>= 2), so it is its own un-remapped value
  u64 ci = __shfl_sync(FULL, c, base_lane);
  for (int i = 0; i < steps; ++i) {
    const u64 cn = __shfl_sync(FULL, c, base_lane + ((i + 1) & (L - 1)));
    const u64 corr = x < 2 ? 2 * HC1 : 0;
    x = hmix(x * HC1 + corr + ci);
    if (sl == i) mine = hfix(x);
    ci = cn;
  }
  return mine;
}

// ---- destination lists of a fetch --------------------------------------------------------------------------------
// A batch of prompts over popular documents names the same pool block many times (a block is a trie node, so equal
// ids always sit at the same depth of different requests).  A fetch therefore reads each DISTINCT source block once
// and writes it to every destination: each (request, block) entry pushes its cache block on the list of its source
// block, and the entry that finds the list empty appends the block to a descriptor list (HBM-tier sources and
// host-tier sources separately, so that each gets the copy engine and the grid that suit it).  List heads carry the
// sequence number of the fetch call in their upper half: a head written by an earlier call reads as "empty", so
// nothing has to be cleared between calls.
struct FetchLink {
  const int* bt;        // block tables of the destination cache; null = no fetch attached to this lookup
  u32 cache_blocks;
  u32 seq;              // sequence number of this fetch call (never 0)
  u32 pending_seq;      // tag of a demotion copy still running on the side stream, 0 if none
  u64* heads;           // [block id] = seq << 32 | entry index of the first list node
  int2* node;           // [entry] = {next entry or LINK_NIL, cache block}
  int2* desc;           // distinct HBM-tier source blocks
  int2* desc_host;      // distinct host-tier source blocks
};

// one entry: returns 1 if it opened the list of an HBM-tier block, 2 for a host-tier block, 0 otherwise
__device__ __forceinline__ int link_entry(const Store& st, const FetchLink& fl, long long e, int id, u32& cnt0, u32& cnt1) {
  const int cb = fl.bt[e];
  if (id < 0 || (u32)id >= st.n[0] + st.n[1] || cb < 0 || (u32)cb >= fl.cache_blocks) { raise(st, S_BOUNDS); return 0; }
  if (fl.pending_seq && (u32)id >= st.n[0] && st.m_flight[id] == fl.pending_seq) { raise(st, S_INFLIGHT); return 0; }
  const u64 old = atomicExch(&fl.heads[id], ((u64)fl.seq << 32) | (u64)(u32)e);
  const bool fresh = (u32)(old >> 32) != fl.seq;
  fl.node[e] = make_int2(fresh ? (int)LINK_NIL : (int)(u32)old, cb);
  if ((u32)id < st.n[0]) ++cnt0; else ++cnt1;
  return fresh ? ((u32)id < st.n[0] ? 1 : 2) : 0;
}
// all 32 lanes: append the blocks whose lists were opened to the descriptor lists (one atomic per warp and list)
__device__ __forceinline__ void link_append(const Store& st, const FetchLink& fl, int opened, int id, int lane) {
  const unsigned m = __ballot_sync(FULL, opened == 1);
  const unsigned mh = __ballot_sync(FULL, opened == 2);
  const u32 slot = fl.seq & 1u;
  if (m) {
    u32 base = 0;
    if (lane == __ffs(m) - 1) base = atomicAdd(&st.ctrl->f_pairs[slot], (u32)__popc(m));
    base = __shfl_sync(FULL, base, __ffs(m) - 1);
    if (opened == 1) fl.desc[base + __popc(m & ((1u << lane) - 1u))] = make_int2(id, 0);
  }
  if (mh) {
    u32 base = 0;
    if (lane == __ffs(mh) - 1) base = atomicAdd(&st.ctrl->f_pairs_host[slot], (u32)__popc(mh));
    base = __shfl_sync(FULL, base, __ffs(mh) - 1);
    if (opened == 2) fl.desc_host[base + __popc(mh & ((1u << lane) - 1u))] = make_int2(id, 0);
  }
  if ((m | mh) && lane == 0) atomicAdd(&st.ctrl->blocks_fetched_distinct, (u64)(__popc(m) + __popc(mh)));
}
// once per linking kernel: clear the per-call scalars of the NEXT fetch call
__device__ __forceinline__ void link_prepare_next(const Store& st, const FetchLink& fl) {
  const u32 nxt = (fl.seq & 1u) ^ 1u;
  st.ctrl->f_pairs[nxt] = 0; st.ctrl->f_pairs_host[nxt] = 0; st.ctrl->f_work[nxt] = 0;
}
__device__ __forceinline__ void link_count(const Store& st, u32 cnt0, u32 cnt1, int lane) {
  cnt0 = __reduce_add_sync(FULL, cnt0);
  cnt1 = __reduce_add_sync(FULL, cnt1);
  if (lane == 0) {
    if (cnt0) atomicAdd(&st.ctrl->blocks_fetched[0], (u64)cnt0);
    if (cnt1) atomicAdd(&st.ctrl->blocks_fetched[1], (u64)cnt1);
  }
}

// keys_out[r*max_blocks + j] = chained key of block j, 0 beyond the request's full blocks
template <int L>
__global__ void __launch_bounds__(256) hash_kernel(Store st, const int* __restrict__ tokens,
                                                   const long long* __restrict__ offsets, int R, int max_blocks,
                                                   u64* __restrict__ keys_out) {
  constexpr int G = 32 / L;
  const int lane = threadIdx.x & 31, sl = lane & (L - 1), sub = lane / L;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long r = warp * G + sub;
  const bool valid = r < R;
  const int nblk = valid ? full_blocks(offsets, (int)r, st.block_tokens, max_blocks) : 0;
  const long long tok0 = valid ? offsets[r] : 0;
  u64 parent = st.root_key;
  int most = __reduce_max_sync(FULL, nblk);
  for (int base = 0; base < most; base += L) {
    const int j = base + sl;
    const bool active = j < nblk;
    u64 c = active ? content_block(tokens + tok0 + (long long)j * st.block_tokens, st.block_tokens) : 0;
    int steps = most - base < L ? most - base : L;
    u64 key = chain_chunk<L>(parent, c, lane, steps);
    if (active) keys_out[r * max_blocks + j] = key;
    parent = __shfl_sync(FULL, key, (lane & ~(L - 1)) + L - 1);
  }
  if (valid)
    for (int j = nblk + sl; j < max_blocks; j += L) keys_out[r * max_blocks + j] = 0;
}

template <int L>
__global__ void __launch_bounds__(256, 4) lookup_kernel(Store st, const int* __restrict__ tokens,
                                                     const long long* __restrict__ offsets, int R, int max_blocks,
                                                     u32 flags, u64 epoch, int* __restrict__ matched,
                                                     int* __restrict__ ids_out, FetchLink fl, u64* __restrict__ keys_out,
                                                     u32* __restrict__ hashed) {
  constexpr int G = 32 / L;
  constexpr unsigned SUBMASK = (L == 32) ? FULL : ((1u << L) - 1u);
  const int lane = threadIdx.x & 31, sl = lane & (L - 1), sub = lane / L;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long r = warp * G + sub;
  const bool valid = r < R;
  const int nblk = valid ? full_blocks(offsets, (int)r, st.block_tokens, max_blocks) : 0;
  const long long tok0 = valid ? offsets[r] : 0;
  u64 parent = st.root_key;
  const u64 inflation = st.policy ? st.ctrl->inflation : 0;
  int m = 0;
  bool done = nblk == 0;
  u32 my_probes = 0, my_visited = 0;
  u32 cnt0 = 0, cnt1 = 0;
  int n_hashed = 0;
  if (fl.bt && blockIdx.x == 0 && threadIdx.x == 0) link_prepare_next(st, fl);

  for (int base = 0;; base += L) {
    const unsigned going = __ballot_sync(FULL, !done);
    if (!going) break;
    const int j = base + sl;
    const bool active = !done && j < nblk;
    u64 c = active ? content_block(tokens + tok0 + (long long)j * st.block_tokens, st.block_tokens) : 0;
    const int left = done ? 0 : (nblk - base < L ? nblk - base : L);
    const int steps = __reduce_max_sync(FULL, left);
    const u64 key = chain_chunk<L>(parent, c, lane, steps);
    if (active) keys_out[r * max_blocks + j] = key;              // kept for an insert of the same batch
    if (!done) n_hashed = nblk < base + L ? nblk : base + L;

    // one probe per distinct key in the warp
    u32 id = NO_ID;
    const unsigned act = __ballot_sync(FULL, active);
    unsigned peers = 0;
    int leader = lane;
    if (active) {
      peers = __match_any_sync(act, key);
      leader = __ffs(peers) - 1;
    }
    {
      const bool probing = active && lane == leader;
      u32 visited;
      find_slot_warp(st, probing, key, &visited, &id);          // all lanes: the rare long way is walked by the whole warp
      if (probing) { my_probes += 1; my_visited += visited; }
    }
    if (active) id = __shfl_sync(peers, id, leader);
    // first miss inside each sub-warp
    const unsigned found = __ballot_sync(FULL, active && id != NO_ID);
    const unsigned mine = (found >> (sub * L)) & SUBMASK;
    const int nf = (mine == SUBMASK) ? L : (__ffs(~mine) - 1);
    const bool hit = active && sl < nf;
    const unsigned hm = __ballot_sync(FULL, hit);
    if (hit) {
      ids_out[r * max_blocks + j] = (int)id;
      const bool touch = !(flags & F_NO_TOUCH);
      if (touch && st.policy == 0) st.m_last[id] = epoch;
      if ((flags & F_PIN) || (touch && st.policy)) {           // one atomic per distinct block in the warp
        const unsigned same = __match_any_sync(hm, id);
        if (lane == __ffs(same) - 1) {
          const u32 cnt = (u32)__popc(same);
          if (flags & F_PIN) atomicAdd(&st.m_ref[id], cnt);
          if (touch && st.policy) touch_block(st, id, epoch, inflation, cnt);
        }
      }
    }
    if (fl.bt) {                                                 // fetch attached: link the hits to their source blocks
      const int opened = hit ? link_entry(st, fl, r * max_blocks + j, (int)id, cnt0, cnt1) : 0;
      link_append(st, fl, opened, (int)id, lane);
    }
    if (!done) {
      m += nf;
      if (nf < L || base + L >= nblk) done = true;
    }
    parent = __shfl_sync(FULL, key, (lane & ~(L - 1)) + L - 1);
  }
  if (fl.bt) link_count(st, cnt0, cnt1, lane);

  if (valid) {
    for (int j = m + sl; j < max_blocks; j += L) ids_out[r * max_blocks + j] = -1;
    if (sl == 0) { matched[r] = m; hashed[r] = (u32)n_hashed; }
  }
  // counters: warp sums, then fire-and-forget adds into one of LOOKUP_STRIPES stripes (no block barrier)
  u32 qb = (valid && sl == 0) ? (u32)nblk : 0, mb = (valid && sl == 0) ? (u32)m : 0;
  qb = __reduce_add_sync(FULL, qb);
  mb = __reduce_add_sync(FULL, mb);
  my_probes = __reduce_add_sync(FULL, my_probes);
  my_visited = __reduce_add_sync(FULL, my_visited);
  if (lane < 4) {
    const u32 v = lane == 0 ? qb : lane == 1 ? my_probes : lane == 2 ? my_visited : mb;
    if (v) atomicAdd(&st.ctrl->lookup_stripes[warp % LOOKUP_STRIPES][lane], (u64)v);
  }
}

// ---- split path for few, long requests ---------------------------------------------------------------------------
// With a whole warp per request the fused kernel above is one dependent chain per 32-block chunk: token loads ->
// content hashes -> 32 chain steps -> probe.  For long prompts (hundreds of blocks, a handful of requests) that
// serial latency is all there is.  Here the content hashes of ALL blocks are computed first by one thread per block
// (content_kernel for ptstore_hash, the first phase of lookup_long_kernel for lookups), and the per-request warp only
// chains and probes; the probe loads of a chunk are in flight while the keys of the next chunk are chained (the chain
// does not depend on the probe result; if the chunk then turns out to hold the first miss the extra chain is discarded).
__global__ void __launch_bounds__(256) content_kernel(Store st, const int* __restrict__ tokens, const long long* __restrict__ offsets,
                                                      int R, int max_blocks, u64* __restrict__ content_out) {
  const long long total = (long long)R * max_blocks;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    const int r = (int)(e / max_blocks), j = (int)(e % max_blocks);
    if (j >= full_blocks(offsets, r, st.block_tokens, max_blocks)) continue;
    content_out[e] = content_block(tokens + offsets[r] + (long long)j * st.block_tokens, st.block_tokens);
  }
}

// keys[r][j] = chained key from content[r][j]; may run in place (content == keys)
__global__ void __launch_bounds__(128) chain_kernel(Store st, const u64* content, const long long* __restrict__ offsets, int R,
                                                    int max_blocks, u64* keys_out) {
  const int lane = threadIdx.x & 31;
  const long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (r >= R) return;
  const int nblk = full_blocks(offsets, (int)r, st.block_tokens, max_blocks);
  u64 parent = st.root_key;
  u64 c_next = lane < nblk ? content[r * max_blocks + lane] : 0;          // loaded a chunk ahead of its use
  for (int base = 0; base < nblk; base += 32) {
    const int j = base + lane;
    const u64 c = c_next;
    c_next = j + 32 < nblk ? content[r * max_blocks + j + 32] : 0;
    const int steps = nblk - base < 32 ? nblk - base : 32;
    const u64 key = chain_chunk<32>(parent, c, lane, steps);
    if (j < nblk) keys_out[r * max_blocks + j] = key;
    parent = __shfl_sync(FULL, key, 31);
  }
  for (int j = nblk + lane; j < max_blocks; j += 32) keys_out[r * max_blocks + j] = 0;
}

// One CTA per request, three phases in one launch.
//   1. all threads: content hashes of the request's blocks into `scratch` (one thread per block);
//   2. warp 0: the chain, the probes and the first miss, as described above; the chained keys of every chunk that is
//      probed are written over the content hashes and hashed[r] says how many leading blocks of request r hold a key
//      afterwards (kept for an insert of the same batch);
//   3. all threads: the -1 padding of the ids and, with a fetch attached, the linking of the matched blocks to their
//      source blocks (one thread per entry: inside the chain loop the same work cost three dependent memory round
//      trips per chunk of a serial loop).
// Progress word of a request in the fused lookup + gather kernel: (launch tag << 32) | (done << 31) | blocks matched so far.
// A word with another tag was written by an earlier launch and reads as "nothing yet".
__device__ __forceinline__ void publish_progress(u64* progress, long long r, u32 tag, u32 count, bool done) {
  const u64 v = ((u64)tag << 32) | (done ? 0x80000000ull : 0ull) | (u64)count;
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(progress + r), "l"(v) : "memory");
}

// One warp: chain, probes, first miss, pins and stamps of request r, whose content hashes are in crow.  The chained keys
// of every chunk that is probed are written over the content hashes and hashed[r] says how many leading blocks hold a key
// afterwards (kept for an insert of the same batch).  With `progress` the number of blocks matched so far is published after
// every chunk, so that another CTA can start copying them.  Returns the matched length (in every lane).
__device__ __forceinline__ int chain_probe_request(const Store& st, u64* crow, int nblk, long long r, int max_blocks, u32 flags, u64 epoch,
                                                   int* __restrict__ matched, int* __restrict__ ids_out, u32* __restrict__ hashed,
                                                   u64* progress, u32 tag, int lane) {
  const u64 inflation = st.policy ? st.ctrl->inflation : 0;
  int m = 0, n_hashed = 0;
  u32 probes = 0, visited_sum = 0;
  u64 parent = st.root_key;
  u64 key = 0;
  u64 c_next = 0;                                  // content hashes of the chunk after the current one, loaded a chunk ahead
  if (nblk > 0) {
    const u64 c0 = lane < nblk ? crow[lane] : 0;
    c_next = 32 + lane < nblk ? crow[32 + lane] : 0;
    key = chain_chunk<32>(parent, c0, lane, nblk < 32 ? nblk : 32);
  }
  for (int base = 0; base < nblk; base += 32) {
    const int j = base + lane;
    const bool active = j < nblk;
    ProbeWindow w;
    if (active) probe_issue(st, key, w);          // loads in flight ...
    u64 next_key = 0;
    if (base + 32 < nblk) {                                       // ... while the next chunk is chained
      const u64 cn = c_next;
      c_next = base + 64 + lane < nblk ? crow[base + 64 + lane] : 0;
      u64 p = __shfl_sync(FULL, key, 31);
      const int left = nblk - base - 32;
      next_key = chain_chunk<32>(p, cn, lane, left < 32 ? left : 32);
    }
    if (active) crow[j] = key;                // the content hashes of this chunk and the next are in registers by now
    n_hashed = nblk < base + 32 ? nblk : base + 32;
    u32 id = NO_ID;
    {
      u32 visited;
      id = probe_finish_warp(st, active, key, w, &visited);       // all lanes: the rare long way is walked by the whole warp
      if (active) { probes += 1; visited_sum += visited; }
    }
    const unsigned found = __ballot_sync(FULL, active && id != NO_ID);
    const int nf = (found == FULL) ? 32 : (__ffs(~found) - 1);
    const bool hit = active && lane < nf;
    const unsigned hm = __ballot_sync(FULL, hit);
    if (hit) {
      ids_out[r * max_blocks + j] = (int)id;
      const bool touch = !(flags & F_NO_TOUCH);
      if (touch && st.policy == 0) st.m_last[id] = epoch;
      if ((flags & F_PIN) || (touch && st.policy)) {
        const unsigned same = __match_any_sync(hm, id);            // ids of one request are distinct: groups of one
        if (lane == __ffs(same) - 1) {
          const u32 cnt = (u32)__popc(same);
          if (flags & F_PIN) atomicAdd(&st.m_ref[id], cnt);
          if (touch && st.policy) touch_block(st, id, epoch, inflation, cnt);
        }
      }
    }
    m += nf;
    if (progress && nf == 32 && base + 32 < nblk) {              // more to come: let the copies of this chunk start
      __syncwarp();
      if (lane == 0) { __threadfence(); publish_progress(progress, r, tag, (u32)m, false); }
    }
    if (nf < 32) break;
    key = next_key;
  }
  if (lane == 0) { matched[r] = m; hashed[r] = (u32)n_hashed; }
  if (progress) {
    __syncwarp();
    if (lane == 0) { __threadfence(); publish_progress(progress, r, tag, (u32)m, true); }
  }
  u32 qb = lane == 0 ? (u32)nblk : 0, mb = lane == 0 ? (u32)m : 0;
  probes = __reduce_add_sync(FULL, probes);
  visited_sum = __reduce_add_sync(FULL, visited_sum);
  qb = __reduce_add_sync(FULL, qb);
  mb = __reduce_add_sync(FULL, mb);
  if (lane < 4) {
    const u32 v = lane == 0 ? qb : lane == 1 ? probes : lane == 2 ? visited_sum : mb;
    if (v) atomicAdd(&st.ctrl->lookup_stripes[r % LOOKUP_STRIPES][lane], (u64)v);
  }
  return m;
}

constexpr int LONG_THREADS = 256;
__global__ void __launch_bounds__(LONG_THREADS) lookup_long_kernel(Store st, const int* __restrict__ tokens, u64* scratch,
                                                                  const long long* __restrict__ offsets, int R, int max_blocks,
                                                                  u32 flags, u64 epoch, int* __restrict__ matched,
                                                                  int* __restrict__ ids_out, FetchLink fl, u32* __restrict__ hashed) {
  __shared__ int s_m;
  const int lane = threadIdx.x & 31;
  const long long r = blockIdx.x;
  if (fl.bt && blockIdx.x == 0 && threadIdx.x == 0) link_prepare_next(st, fl);
  const int nblk = full_blocks(offsets, (int)r, st.block_tokens, max_blocks);
  u64* crow = scratch + r * max_blocks;
  {
    const int* t0 = tokens + offsets[r];
    for (int j = threadIdx.x; j < nblk; j += LONG_THREADS) crow[j] = content_block(t0 + (long long)j * st.block_tokens, st.block_tokens);
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    const int m = chain_probe_request(st, crow, nblk, r, max_blocks, flags, epoch, matched, ids_out, hashed, nullptr, 0, lane);
    if (lane == 0) s_m = m;
  }
  __syncthreads();
  const int m = s_m;
  for (int j = m + threadIdx.x; j < max_blocks; j += LONG_THREADS) ids_out[r * max_blocks + j] = -1;
  if (fl.bt) {
    u32 cnt0 = 0, cnt1 = 0;
    for (int j0 = 0; j0 < m; j0 += LONG_THREADS) {
      const int j = j0 + threadIdx.x;
      const bool hit = j < m;
      const int id = hit ? ids_out[r * max_blocks + j] : -1;
      const int opened = hit ? link_entry(st, fl, r * max_blocks + j, id, cnt0, cnt1) : 0;
      link_append(st, fl, opened, id, lane);
    }
    link_count(st, cnt0, cnt1, lane);
  }
}

// the linking step on its own, for a fetch of ids the caller already holds: every (r, j < matched[r]) entry
__global__ void __launch_bounds__(256) fetch_link_kernel(Store st, const int* __restrict__ ids, const int* __restrict__ matched, int R,
                                                         int max_blocks, FetchLink fl) {
  const long long total = (long long)R * max_blocks;
  const long long rounded = (total + 31) & ~31ll;
  const int lane = threadIdx.x & 31;
  u32 cnt0 = 0, cnt1 = 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) link_prepare_next(st, fl);
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < rounded; e += (long long)gridDim.x * blockDim.x) {
    int opened = 0, id = -1;
    if (e < total) {
      const int r = (int)(e / max_blocks), j = (int)(e % max_blocks);
      int mr = matched[r];
      mr = mr > max_blocks ? max_blocks : mr;
      if (j < mr) {
        id = ids[e];
        opened = link_entry(st, fl, e, id, cnt0, cnt1);
      }
    }
    link_append(st, fl, opened, id, lane);
  }
  link_count(st, cnt0, cnt1, lane);
}

// refcount-- per (r, j < matched[r]) pair; a zero count stays zero and raises S_STATE
__global__ void __launch_bounds__(256) release_kernel(Store st, const int* __restrict__ ids,
                                                      const int* __restrict__ matched, int R, int max_blocks) {
  const long long total = (long long)R * max_blocks;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    const int r = (int)(e / max_blocks), j = (int)(e % max_blocks);
    int mr = matched[r];
    if (mr > max_blocks) mr = max_blocks;
    if (j >= mr) continue;
    const int id = ids[e];
    if (id < 0 || (u32)id >= st.n[0] + st.n[1] || st.m_key[id] == 0) { raise(st, S_BOUNDS); continue; }
    // decrement unless zero
    u32 old = st.m_ref[id];
    while (true) {
      if (old == 0) { raise(st, S_STATE); break; }
      u32 seen = atomicCAS(&st.m_ref[id], old, old - 1);
      if (seen == old) break;
      old = seen;
    }
  }
}

}  // namespace pts
