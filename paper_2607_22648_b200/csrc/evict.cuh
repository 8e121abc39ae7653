// LRU eviction of unreferenced leaves, demotion to the host tier, table rebuild.
// (Paper Section 1: blocks of finished requests are evicted least-recently-used first; Section 4.1
// "Access pattern-aware eviction policy": owned tensors are flushed to slower tiers, not dropped.)
//
// Order of victims: (LRU stamp ascending, deeper first, lower id first), leaves first, a parent may
// follow its last child in the same call.  Stamps are only written along whole chains, so a parent's
// stamp is never older than a child's, and pins are taken along whole chains, so a parent's count is
// never below a child's.  Under those two facts the greedy "take the best leaf, repeat" loop takes
// exactly the first n entries of the list of all unreferenced nodes of the tier sorted by that order
// (for the host tier: those without a live descendant in HBM).  The kernels build that list, sort it
// with a stable LSD radix sort and apply the first n entries in parallel.
#pragma once
#include "common.cuh"

namespace pts {

struct Key2 { u64 hi, lo; };     // hi = stamp; lo = (0xFFFF - depth) << 32 | block id

enum EvictMode { EV_DROP = 0, EV_HOST_ROOM = 1, EV_DEMOTE = 2 };

__global__ void evict_begin_kernel(Store st, int mode, u32 n) {
  Ctrl* c = st.ctrl;
  const u32 host_free = c->ring[1].count;
  u32 want = n;
  if (mode == EV_HOST_ROOM) want = n > host_free ? n - host_free : 0;
  if (mode == EV_DEMOTE) want = n < host_free ? n : host_free;
  c->ev_want = want;
  c->ev_cand = 0;
  if (mode != EV_DEMOTE) c->ev_host_dropped = 0;
}

// Host-tier nodes that still have a live descendant in HBM must stay.  Every live HBM node whose
// parent sits in the host tier walks up its chain and marks the host-tier ancestors, stopping at the
// first one already marked (whoever marked it goes on from there).
__global__ void __launch_bounds__(256) mark_blocked_kernel(Store st, unsigned char* __restrict__ blocked) {
  if (st.ctrl->ev_want == 0) return;
  for (u32 id = blockIdx.x * blockDim.x + threadIdx.x; id < st.n[0]; id += gridDim.x * blockDim.x) {
    if (st.m_key[id] == 0 || st.m_depth[id] == 0) continue;
    u64 pk = st.m_parent[id];
    bool climbing = false;
    for (u32 step = 0; step < 65536; ++step) {
      u32 visited, pid;
      if (find_slot(st.table, st.slots, pk, &visited, &pid) == NO_SLOT || pid == NO_ID) break;
      if (pid >= st.n[0]) {                                   // host-tier ancestor
        if (*reinterpret_cast<volatile unsigned char*>(&blocked[pid])) break;
        blocked[pid] = 1;
        climbing = true;
      } else if (!climbing) {
        break;                                                // parent in HBM: its own walk covers the rest
      }
      if (st.m_depth[pid] == 0) break;
      pk = st.m_parent[pid];
    }
  }
}

__global__ void __launch_bounds__(256) collect_kernel(Store st, int tier, const unsigned char* __restrict__ blocked, Key2* __restrict__ out) {
  if (st.ctrl->ev_want == 0) return;
  const u32 lo = tier ? st.n[0] : 0, hi = tier ? st.n[0] + st.n[1] : st.n[0];
  const u32 span = hi - lo;
  const u32 rounded = (span + 31u) & ~31u;
  for (u32 i = blockIdx.x * blockDim.x + threadIdx.x; i < rounded; i += gridDim.x * blockDim.x) {
    const u32 id = lo + i;
    const bool ok = i < span && st.m_key[id] != 0 && st.m_ref[id] == 0 && !(blocked && blocked[id]);
    const unsigned m = __ballot_sync(FULL, ok);
    if (!m) continue;
    const int lane = threadIdx.x & 31;
    u32 base = 0;
    if (lane == __ffs(m) - 1) base = atomicAdd(&st.ctrl->ev_cand, (u32)__popc(m));
    base = __shfl_sync(FULL, base, __ffs(m) - 1);
    if (ok) {
      Key2 k;
      k.hi = st.m_last[id];
      k.lo = ((u64)(0xFFFFu - (st.m_depth[id] & 0xFFFFu)) << 32) | id;
      out[base + __popc(m & ((1u << lane) - 1u))] = k;
    }
  }
}

// ---- stable LSD radix sort of Key2, 8 bits per pass --------------------------------------------------------
constexpr int SORT_THREADS = 256;
// elements per CTA = 256 threads x STEPS: 512 (STEPS 2) for stores up to 32k blocks, so that a sort of a few ten thousand
// candidates spreads over tens of SMs and each CTA's serial part stays short; 2048 (STEPS 8) beyond, to keep the
// digit-by-tile histogram small
constexpr int sort_steps_for(unsigned long long n_blocks) { return n_blocks <= (32u << 10) ? 2 : 8; }

__device__ __forceinline__ u32 digit_of(const Key2& k, int word, int shift) { return (u32)(((word ? k.hi : k.lo) >> shift) & 0xFFu); }

template <int STEPS>
__global__ void __launch_bounds__(SORT_THREADS) sort_hist_kernel(const Key2* __restrict__ in, const u32* __restrict__ n_ptr, int word,
                                                                 int shift, u32* __restrict__ hist, u32 n_tiles) {
  __shared__ u32 h[256];
  h[threadIdx.x] = 0;
  __syncthreads();
  const u32 n = *n_ptr;
  constexpr u32 SORT_TILE = SORT_THREADS * STEPS;
  const u32 base = blockIdx.x * SORT_TILE;
  for (u32 i = threadIdx.x; i < SORT_TILE; i += SORT_THREADS)
    if (base + i < n) atomicAdd(&h[digit_of(in[base + i], word, shift)], 1u);
  __syncthreads();
  hist[threadIdx.x * n_tiles + blockIdx.x] = h[threadIdx.x];
}

__global__ void __launch_bounds__(1024) sort_scan_kernel(u32* __restrict__ hist, u32 len) {
  __shared__ u32 warp_sums[32];
  __shared__ u32 carry;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (u32 base = 0; base < len; base += 1024) {
    const u32 i = base + threadIdx.x;
    const u32 v = i < len ? hist[i] : 0;
    u32 x = v;
    for (int o = 1; o < 32; o <<= 1) { u32 y = __shfl_up_sync(FULL, x, o); if (lane >= o) x += y; }
    if (lane == 31) warp_sums[wid] = x;
    __syncthreads();
    if (wid == 0) {
      u32 w = warp_sums[lane];
      for (int o = 1; o < 32; o <<= 1) { u32 y = __shfl_up_sync(FULL, w, o); if (lane >= o) w += y; }
      warp_sums[lane] = w;
    }
    __syncthreads();
    const u32 incl = x + (wid ? warp_sums[wid - 1] : 0);
    if (i < len) hist[i] = carry + incl - v;
    __syncthreads();
    if (threadIdx.x == 1023) carry += incl;
    __syncthreads();
  }
}

template <int STEPS>
__global__ void __launch_bounds__(SORT_THREADS) sort_scatter_kernel(const Key2* __restrict__ in, Key2* __restrict__ out,
                                                                    const u32* __restrict__ n_ptr, int word, int shift,
                                                                    const u32* __restrict__ hist, u32 n_tiles) {
  __shared__ u32 wh[SORT_THREADS / 32][256];     // per-warp digit counts, then per-warp output cursors
  constexpr u32 SORT_TILE = SORT_THREADS * STEPS;
  const u32 n = *n_ptr;
  const u32 tile0 = blockIdx.x * SORT_TILE;
  if (tile0 >= n) return;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  for (int i = lane; i < 256; i += 32) wh[w][i] = 0;
  __syncwarp();
  const u32 seg = tile0 + w * (SORT_TILE / (SORT_THREADS / 32));
  Key2 el[STEPS];
  u32 dg[STEPS];
#pragma unroll
  for (int s = 0; s < STEPS; ++s) {
    const u32 i = seg + s * 32 + lane;
    const bool ok = i < n;
    if (ok) { el[s] = in[i]; dg[s] = digit_of(el[s], word, shift); }
    const unsigned act = __ballot_sync(FULL, ok);
    if (ok) {
      const unsigned peers = __match_any_sync(act, dg[s]);
      if (lane == __ffs(peers) - 1) wh[w][dg[s]] += __popc(peers);
    }
    __syncwarp();
  }
  __syncthreads();
  {   // cursor of (warp, digit) = global offset of (digit, tile) + counts of earlier warps
    const int d = threadIdx.x;
    u32 run = hist[d * n_tiles + blockIdx.x];
    for (int ww = 0; ww < SORT_THREADS / 32; ++ww) { const u32 t = wh[ww][d]; wh[ww][d] = run; run += t; }
  }
  __syncthreads();
#pragma unroll
  for (int s = 0; s < STEPS; ++s) {
    const u32 i = seg + s * 32 + lane;
    const bool ok = i < n;
    const unsigned act = __ballot_sync(FULL, ok);
    if (ok) {
      const unsigned peers = __match_any_sync(act, dg[s]);
      const u32 pos = wh[w][dg[s]] + __popc(peers & ((1u << lane) - 1u));
      out[pos] = el[s];
      __syncwarp(peers);
      if (lane == __ffs(peers) - 1) wh[w][dg[s]] += __popc(peers);
    }
    __syncwarp();
  }
}

// ---- apply ----------------------------------------------------------------------------------------------
__device__ __forceinline__ u32 ev_take(const Ctrl* c) { return c->ev_want < c->ev_cand ? c->ev_want : c->ev_cand; }

// delete the first `take` sorted candidates: tombstone, free the id (back of the ring, in victim order)
__global__ void __launch_bounds__(256) apply_drop_kernel(Store st, int tier, const Key2* __restrict__ sorted, int* __restrict__ victims) {
  const Ctrl* c = st.ctrl;
  const u32 take = ev_take(c);
  const u32 cap = st.n[tier], head = c->ring[tier].head, count = c->ring[tier].count;
  for (u32 i = blockIdx.x * blockDim.x + threadIdx.x; i < take; i += gridDim.x * blockDim.x) {
    const u32 id = (u32)(sorted[i].lo & 0xFFFFFFFFu);
    u32 visited, sid;
    const u32 s = find_slot(st.table, st.slots, st.m_key[id], &visited, &sid);
    if (s != NO_SLOT) {
      st.table[s].id = NO_ID;
      st.table[s].aux = NO_ID;
      st.table[s].key = KEY_TOMB;
    }
    st.m_key[id] = 0;
    st.ring_ids[tier][(u32)(((u64)head + count + i) % cap)] = (int)id;
    if (victims) victims[i] = (int)id;
  }
}

__global__ void drop_finish_kernel(Store st, int tier, int mode, const Key2* __restrict__ sorted, int* __restrict__ n_evicted) {
  Ctrl* c = st.ctrl;
  const u32 take = ev_take(c);
  if (st.policy && take && sorted[take - 1].hi > c->inflation) c->inflation = sorted[take - 1].hi;   // GDSF clock
  c->ring[tier].count += take;
  c->live[tier] -= take;
  c->tombstones += take;
  c->blocks_dropped[tier] += take;
  if (mode == EV_DROP) { if (n_evicted) { n_evicted[0] = (int)take; n_evicted[1] = 0; } }
  else c->ev_host_dropped = take;
}

// move the first `take` sorted HBM candidates to host blocks popped from the front of the host ring
__global__ void __launch_bounds__(256) apply_demote_kernel(Store st, const Key2* __restrict__ sorted, int2* __restrict__ desc,
                                                           int* __restrict__ victims) {
  const Ctrl* c = st.ctrl;
  const u32 take = ev_take(c);
  const u32 head1 = c->ring[1].head, head0 = c->ring[0].head, count0 = c->ring[0].count;
  for (u32 i = blockIdx.x * blockDim.x + threadIdx.x; i < take; i += gridDim.x * blockDim.x) {
    const u32 old_id = (u32)(sorted[i].lo & 0xFFFFFFFFu);
    const u32 new_id = (u32)st.ring_ids[1][(u32)(((u64)head1 + i) % st.n[1])];
    u32 visited, sid;
    const u32 s = find_slot(st.table, st.slots, st.m_key[old_id], &visited, &sid);
    if (s != NO_SLOT) st.table[s].id = new_id;
    st.m_key[new_id] = st.m_key[old_id];
    st.m_parent[new_id] = st.m_parent[old_id];
    st.m_last[new_id] = st.m_last[old_id];
    st.m_freq[new_id] = st.m_freq[old_id];
    st.m_ref[new_id] = 0;
    st.m_depth[new_id] = st.m_depth[old_id];
    st.m_key[old_id] = 0;
    desc[i] = make_int2((int)old_id, (int)new_id);
    st.ring_ids[0][(u32)(((u64)head0 + count0 + i) % st.n[0])] = (int)old_id;
    if (victims) victims[i] = (int)old_id;
  }
}

__global__ void __launch_bounds__(256) demote_finish_kernel(Store st, const Key2* __restrict__ sorted, int* __restrict__ n_evicted,
                                                            int* __restrict__ victims, const int* __restrict__ room_victims) {
  Ctrl* c = st.ctrl;
  const u32 take = ev_take(c);
  const u32 dropped = c->ev_host_dropped;
  if (victims)
    for (u32 i = threadIdx.x; i < dropped; i += blockDim.x) victims[take + i] = room_victims[i];
  __syncthreads();
  if (threadIdx.x == 0) {
    c->ring[1].head = (u32)(((u64)c->ring[1].head + take) % st.n[1]);
    c->ring[1].count -= take;
    c->ring[0].count += take;
    c->live[0] -= take;
    c->live[1] += take;
    c->n_pairs_tier = take;
    c->blocks_demoted += take;
    if (st.policy && take && sorted[take - 1].hi > c->inflation) c->inflation = sorted[take - 1].hi;
    if (n_evicted) { n_evicted[0] = (int)take; n_evicted[1] = (int)dropped; }
  }
}

// ---- table maintenance ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) table_clear_kernel(Slot* __restrict__ table, u64 slots) {
  for (u64 s = (u64)blockIdx.x * blockDim.x + threadIdx.x; s < slots; s += (u64)gridDim.x * blockDim.x) {
    uint4 v = make_uint4(0u, 0u, NO_ID, NO_ID);
    *reinterpret_cast<uint4*>(table + s) = v;
  }
}

// Rebuild in place, decided on the device: when more than `threshold` slots hold deleted markers, the
// table is moved aside (stash), cleared, and its live entries are re-inserted.  Both kernels return at
// once otherwise.  The marker count is reset by the insert that follows (insert_plan_kernel).
__global__ void __launch_bounds__(256) table_stash_kernel(Store st, Slot* __restrict__ stash, u32 threshold) {
  if (st.ctrl->tombstones <= threshold) return;
  for (u64 s = (u64)blockIdx.x * blockDim.x + threadIdx.x; s < st.slots; s += (u64)gridDim.x * blockDim.x) {
    uint4* p = reinterpret_cast<uint4*>(st.table + s);
    *reinterpret_cast<uint4*>(stash + s) = *p;
    *p = make_uint4(0u, 0u, NO_ID, NO_ID);
  }
}
__global__ void __launch_bounds__(256) table_rebuild_kernel(Store st, const Slot* __restrict__ stash, u32 threshold) {
  if (st.ctrl->tombstones <= threshold) return;
  for (u64 s = (u64)blockIdx.x * blockDim.x + threadIdx.x; s < st.slots; s += (u64)gridDim.x * blockDim.x) {
    const Slot v = load_slot(stash + s);
    if (v.key < 2 || v.id == NO_ID) continue;
    u64 t = home_slot(v.key, st.slots);
    bool placed = false;
    for (u64 i = 0; i < st.slots; ++i) {
      if (atomicCAS(&st.table[t].key, KEY_EMPTY, v.key) == KEY_EMPTY) { st.table[t].id = v.id; placed = true; break; }
      t = (t + 1 == st.slots) ? 0 : t + 1;
    }
    if (!placed) raise(st, S_TABLE_FULL);
  }
}

__global__ void __launch_bounds__(256) store_init_kernel(Store st) {
  const u32 total = st.n[0] + st.n[1];
  for (u32 i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    st.m_key[i] = 0; st.m_parent[i] = 0; st.m_last[i] = 0; st.m_freq[i] = 0; st.m_ref[i] = 0; st.m_depth[i] = 0;
    if (i < st.n[0]) st.ring_ids[0][i] = (int)i;
    else st.ring_ids[1][i - st.n[0]] = (int)i;
  }
}
__global__ void ctrl_init_kernel(Store st) {
  Ctrl* c = st.ctrl;
  unsigned char* p = reinterpret_cast<unsigned char*>(c);
  for (size_t i = 0; i < sizeof(Ctrl); ++i) p[i] = 0;
  c->ring[0].count = st.n[0];
  c->ring[1].count = st.n[1];
}

// counters for a caller that does not want to block: written by the device to any device-accessible address
struct StatsOut {
  u64 epoch, live[2], free_blocks[2], tombstones, query_blocks, probes_issued, slots_visited, blocks_matched, blocks_fetched[2],
      blocks_inserted, blocks_denied, blocks_dropped[2], blocks_demoted, rebuilds, blocks_promoted, gdsf_clock, blocks_fetched_distinct;
};
__global__ void stats_kernel(Store st, u64 epoch, StatsOut* __restrict__ out) {
  const Ctrl* c = st.ctrl;
  StatsOut o;
  o.epoch = epoch;
  for (int t = 0; t < 2; ++t) {
    o.live[t] = c->live[t]; o.free_blocks[t] = c->ring[t].count;
    o.blocks_fetched[t] = c->blocks_fetched[t]; o.blocks_dropped[t] = c->blocks_dropped[t];
  }
  o.tombstones = c->tombstones;
  o.query_blocks = c->query_blocks; o.probes_issued = c->probes_issued; o.slots_visited = c->slots_visited; o.blocks_matched = c->blocks_matched;
  for (int i = 0; i < LOOKUP_STRIPES; ++i) {
    o.query_blocks += c->lookup_stripes[i][0]; o.probes_issued += c->lookup_stripes[i][1];
    o.slots_visited += c->lookup_stripes[i][2]; o.blocks_matched += c->lookup_stripes[i][3];
  }
  o.blocks_inserted = c->blocks_inserted; o.blocks_denied = c->blocks_denied; o.blocks_demoted = c->blocks_demoted;
  o.rebuilds = c->rebuilds; o.blocks_promoted = c->blocks_promoted; o.gdsf_clock = c->inflation;
  o.blocks_fetched_distinct = c->blocks_fetched_distinct;
  *out = o;
}

}  // namespace pts
