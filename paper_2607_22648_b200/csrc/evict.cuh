// Eviction of unreferenced leaves (LRU or GDSF order), demotion to the host tier.
// (Paper Section 1: blocks of finished requests are evicted least-recently-used first; Section 4.1
// "Access pattern-aware eviction policy": owned tensors are flushed to slower tiers, not dropped.)
//
// Order of victims: (stamp or priority ascending, deeper first, lower id first), leaves first, a parent may
// follow its last child in the same call.  Stamps are only written along whole chains, so a parent's
// stamp is never older than a child's, and pins are taken along whole chains, so a parent's count is
// never below a child's.  Under those two facts the greedy "take the best leaf, repeat" loop takes
// exactly the first n entries of the list of all unreferenced nodes of the tier sorted by that order
// (for the host tier: those without a live descendant in HBM).
//
// One cooperative kernel does a whole phase (drop, room-making drop, or demotion): it builds one sort record per
// block id of the tier (non-candidates get a sentinel that sorts last), orders the records with a stable LSD
// radix sort whose passes are separated by grid-wide barriers, applies the first n records in parallel and
// updates the rings.  Records start in id order and the sort is stable, so the id needs no pass of its own; the
// number of passes for the depth and for the stamp comes from the largest depth and the stamp range found among
// the candidates on the device (no host-side bound on stamps or priorities is involved).
#pragma once
#include "common.cuh"

namespace pts {

struct Key2 { u64 hi, lo; };     // hi = stamp / priority; lo = (0xFFFF - depth) << 32 | block id; lo = ~0 marks a non-candidate

enum EvictMode { EV_DROP = 0, EV_HOST_ROOM = 1, EV_DEMOTE = 2 };

constexpr int EV_THREADS = 256;
constexpr int EV_WARPS = EV_THREADS / 32;

struct EvictArgs {
  int tier;                 // tier the victims come from
  int mode;                 // EvictMode
  // number of victims asked for: n; or (reserve form, want_free >= 0) need = want_free - sum(minus[0..n_minus)) - free
  // blocks of tier 0, and need + n victims if need > 0, else none
  u32 n;
  long long want_free;      // < 0: plain form
  const int* minus;
  int n_minus;
  int* n_evicted;           // out [2] or null
  int* victims;             // out or null
  u32 max_victims;          // entries the caller's victim array can take per part (reserve form), else ~0
  int* room;                // scratch: victims of a room-making drop, consumed by the demotion that follows
  Key2* buf[2];
  u32* hist;                // [256][grid]
  u64* tile_stats;          // [grid][4]: candidates, max stamp, min stamp, max depth
  unsigned char* blocked;
  int2* desc_tier;          // demotion: {HBM id, host id} copy descriptors
  u32 flight_seq;           // demotion whose copy runs on the side stream: tag written to the new host blocks, else 0
  u32 tile_elems;           // records per CTA, multiple of EV_THREADS
  u32 launch_seq;
};

// Host-tier nodes that still have a live descendant in HBM must stay.  Every live HBM node whose
// parent sits in the host tier walks up its chain and marks the host-tier ancestors, stopping at the
// first one already marked (whoever marked it goes on from there).
__device__ __forceinline__ void mark_blocked_walk(const Store& st, unsigned char* __restrict__ blocked, u32 id) {
  if (st.m_key[id] == 0 || st.m_depth[id] == 0) return;
  u64 pk = st.m_parent[id];
  bool climbing = false;
  for (u32 step = 0; step < 65536; ++step) {
    u32 visited, pid;
    if (find_slot(st, pk, &visited, &pid) == NO_SLOT || pid == NO_ID) break;
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

__device__ __forceinline__ bool ev_is_candidate(const Key2& k) { return k.lo != ~0ull; }

// digit of one sort pass.  Passes 0..depth_passes-1 order by depth (deeper first), the rest by stamp - smin;
// non-candidates carry the value one above the largest candidate value in every stamp pass, so they end up last.
struct EvictPlan {
  u32 dmax;          // largest candidate depth
  u64 smin, srange;  // smallest candidate stamp, largest minus smallest
  int depth_passes, stamp_passes;
};
__device__ __forceinline__ u32 ev_digit(const Key2& k, const EvictPlan& pl, int pass) {
  if (pass < pl.depth_passes) {
    if (!ev_is_candidate(k)) return 0;
    const u32 depth = 0xFFFFu - (u32)((k.lo >> 32) & 0xFFFFu);
    return ((pl.dmax - depth) >> (8 * pass)) & 0xFFu;
  }
  const u64 v = ev_is_candidate(k) ? k.hi - pl.smin : pl.srange + 1;
  return (u32)(v >> (8 * (pass - pl.depth_passes))) & 0xFFu;
}
__device__ __forceinline__ int ev_bytes(u64 v) {
  int b = 1;
  while (v >>= 8) ++b;
  return b;
}

__global__ void __launch_bounds__(EV_THREADS) evict_kernel(Store st, EvictArgs a) {
  __shared__ u32 wh[EV_WARPS][256];        // per-warp digit counts of the CTA's tile, then per-warp output cursors
  __shared__ u64 red[EV_WARPS][4];
  Ctrl* c = st.ctrl;
  GridBarrier bar;
  bar.init(c, a.launch_seq);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int tier = a.tier;
  const u32 lo_id = tier ? st.n[0] : 0;
  const u32 span = st.n[tier];
  const u32 G = gridDim.x;

  // ---- what is wanted; ring positions are read now, before anything in this launch changes them ----------------------
  const u32 head0 = c->ring[0].head, count0 = c->ring[0].count, head1 = c->ring[1].head, count1 = c->ring[1].count;
  const u32 host_dropped = c->ev_host_dropped;
  u32 n = a.n;
  if (a.want_free >= 0) {                      // reserve form: every CTA sums the list for itself
    u64 part = 0;
    for (int i = threadIdx.x; i < a.n_minus; i += EV_THREADS) { const int m = a.minus[i]; part += m > 0 ? (u64)m : 0; }
    for (int o = 16; o; o >>= 1) part += __shfl_xor_sync(FULL, part, o);
    if (lane == 0) red[w][0] = part;
    __syncthreads();
    part = 0;
    for (int i = 0; i < EV_WARPS; ++i) part += red[i][0];
    __syncthreads();                             // red is used again below
    long long need = a.want_free - (long long)part;
    need -= (long long)count0;
    if (need > 0) need += (long long)a.n;                 // short of room: evict `n` blocks more than needed right now
    n = need > 0 ? (need > 0x7FFFFFFFll ? 0x7FFFFFFFu : (u32)need) : 0u;
    if (n > a.max_victims) n = a.max_victims;
  }
  u32 want = n;
  if (a.mode == EV_HOST_ROOM) want = n > count1 ? n - count1 : 0;
  if (a.mode == EV_DEMOTE) want = n < count1 ? n : count1;

  const u32 tile0 = blockIdx.x * a.tile_elems;
  const u32 seg = a.tile_elems / EV_WARPS;            // records per warp, multiple of 32
  u32 take = 0;
  int cur = 0;

  PHASE_MARK(st, 0);
  if (want > 0) {
    // ---- host tier: which nodes are pinned in place by HBM descendants -------------------------------------------------
    const bool use_blocked = tier == 1 && st.n[1] > 0 && a.blocked != nullptr;
    if (use_blocked) {
      for (u32 i = blockIdx.x * EV_THREADS + threadIdx.x; i < st.n[1]; i += G * EV_THREADS) a.blocked[st.n[0] + i] = 0;
      bar.sync(st);
      for (u32 id = blockIdx.x * EV_THREADS + threadIdx.x; id < st.n[0]; id += G * EV_THREADS) mark_blocked_walk(st, a.blocked, id);
      bar.sync(st);
    }
    // ---- one record per block id of the tier, in id order ----------------------------------------------------------------
    u64 cand = 0, smax = 0, smin = ~0ull, dmax = 0;
    for (u32 i = tile0 + threadIdx.x; i < tile0 + a.tile_elems && i < span; i += EV_THREADS) {
      const u32 id = lo_id + i;
      Key2 k;
      k.hi = ~0ull; k.lo = ~0ull;
      if (st.m_key[id] != 0 && st.m_ref[id] == 0 && !(use_blocked && a.blocked[id])) {
        const u32 depth = st.m_depth[id] & 0xFFFFu;
        k.hi = st.m_last[id];
        k.lo = ((u64)(0xFFFFu - depth) << 32) | id;
        ++cand;
        smax = k.hi > smax ? k.hi : smax;
        smin = k.hi < smin ? k.hi : smin;
        dmax = depth > dmax ? depth : dmax;
      }
      a.buf[0][i] = k;
    }
    cand = __reduce_add_sync(FULL, (u32)cand);
    for (int o = 16; o; o >>= 1) {
      const u64 x = __shfl_xor_sync(FULL, smax, o), y = __shfl_xor_sync(FULL, smin, o), z = __shfl_xor_sync(FULL, dmax, o);
      smax = x > smax ? x : smax; smin = y < smin ? y : smin; dmax = z > dmax ? z : dmax;
    }
    if (lane == 0) { red[w][0] = cand; red[w][1] = smax; red[w][2] = smin; red[w][3] = dmax; }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int i = 1; i < EV_WARPS; ++i) {
        cand += red[i][0];
        smax = red[i][1] > smax ? red[i][1] : smax; smin = red[i][2] < smin ? red[i][2] : smin; dmax = red[i][3] > dmax ? red[i][3] : dmax;
      }
      u64* t = a.tile_stats + 4ull * blockIdx.x;
      t[0] = cand; t[1] = smax; t[2] = smin; t[3] = dmax;
    }
    bar.sync(st);
    cand = 0; smax = 0; smin = ~0ull; dmax = 0;
    for (u32 b = lane; b < G; b += 32) {                // every warp reduces the per-CTA figures itself
      const u64* t = a.tile_stats + 4ull * b;
      cand += t[0];
      smax = t[1] > smax ? t[1] : smax; smin = t[2] < smin ? t[2] : smin; dmax = t[3] > dmax ? t[3] : dmax;
    }
    cand = __reduce_add_sync(FULL, (u32)cand);
    for (int o = 16; o; o >>= 1) {
      const u64 x = __shfl_xor_sync(FULL, smax, o), y = __shfl_xor_sync(FULL, smin, o), z = __shfl_xor_sync(FULL, dmax, o);
      smax = x > smax ? x : smax; smin = y < smin ? y : smin; dmax = z > dmax ? z : dmax;
    }
    take = want < (u32)cand ? want : (u32)cand;
    PHASE_MARK(st, 1);

    if (take > 0) {
      EvictPlan pl;
      pl.dmax = (u32)dmax; pl.smin = smin; pl.srange = smax - smin;
      pl.depth_passes = dmax ? ev_bytes(dmax) : 0;
      pl.stamp_passes = ev_bytes(pl.srange + 1);           // the value srange + 1 of the non-candidates must sort too
      const int passes = pl.depth_passes + pl.stamp_passes;
      for (int p = 0; p < passes && bar.ok; ++p) {
        const Key2* in = a.buf[cur];
        Key2* out = a.buf[cur ^ 1];
        // counts of every digit per warp segment (a warp's records are contiguous, taken 32 at a time in order)
        for (int i = lane; i < 256; i += 32) wh[w][i] = 0;
        __syncwarp();
        const u32 wseg = tile0 + w * seg;
        for (u32 s = 0; s < seg; s += 32) {
          const u32 i = wseg + s + lane;
          const bool ok = i < span;
          u32 dg = 0;
          if (ok) dg = ev_digit(in[i], pl, p);
          const unsigned act = __ballot_sync(FULL, ok);
          if (ok) {
            const unsigned peers = __match_any_sync(act, dg);
            if (lane == __ffs(peers) - 1) wh[w][dg] += __popc(peers);
          }
          __syncwarp();
        }
        __syncthreads();
        {
          const int d = threadIdx.x;                        // EV_THREADS == 256: one digit per thread
          u32 sum = 0;
          for (int ww = 0; ww < EV_WARPS; ++ww) sum += wh[ww][d];
          a.hist[(u32)d * G + blockIdx.x] = sum;
        }
        bar.sync(st);
        {   // cursor of (digit d, this tile) = records with a smaller digit anywhere + records with digit d in earlier tiles
          const int d = threadIdx.x;
          u32 total = 0, before = 0;
          const u32* row = a.hist + (u32)d * G;
          for (u32 b = 0; b < G; ++b) { const u32 v = row[b]; total += v; before += b < blockIdx.x ? v : 0; }
          // exclusive scan of the digit totals over the 256 threads
          u32 x = total;
          for (int o = 1; o < 32; o <<= 1) { const u32 y = __shfl_up_sync(FULL, x, o); if (lane >= o) x += y; }
          __shared__ u32 wsum[EV_WARPS];
          if (lane == 31) wsum[w] = x;
          __syncthreads();
          u32 base = x - total;
          for (int ww = 0; ww < w; ++ww) base += wsum[ww];
          u32 run = base + before;
          for (int ww = 0; ww < EV_WARPS; ++ww) { const u32 t = wh[ww][d]; wh[ww][d] = run; run += t; }
        }
        __syncthreads();
        for (u32 s = 0; s < seg; s += 32) {
          const u32 i = wseg + s + lane;
          const bool ok = i < span;
          Key2 el;
          u32 dg = 0;
          if (ok) { el = in[i]; dg = ev_digit(el, pl, p); }
          const unsigned act = __ballot_sync(FULL, ok);
          if (ok) {
            const unsigned peers = __match_any_sync(act, dg);
            const u32 pos = wh[w][dg] + __popc(peers & ((1u << lane) - 1u));
            out[pos] = el;
            __syncwarp(peers);
            if (lane == __ffs(peers) - 1) wh[w][dg] += __popc(peers);
          }
          __syncwarp();
        }
        bar.sync(st);
        cur ^= 1;
      }

      PHASE_MARK(st, 2);
      // ---- apply the first `take` records ------------------------------------------------------------------------------
      if (bar.ok) {
        const Key2* sorted = a.buf[cur];
        if (a.mode == EV_DEMOTE) {
          for (u32 i0 = blockIdx.x * EV_THREADS + (threadIdx.x & ~31u); i0 < take; i0 += G * EV_THREADS) {   // whole warps
            const u32 i = i0 + (threadIdx.x & 31u);
            const bool on = i < take;
            const u32 old_id = on ? (u32)(sorted[i].lo & 0xFFFFFFFFu) : 0;
            u32 visited, sid;
            const u32 s = find_slot_warp(st, on, on ? st.m_key[old_id] : 0, &visited, &sid);
            if (!on) continue;
            const u32 new_id = (u32)st.ring_ids[1][(u32)(((u64)head1 + i) % st.n[1])];
            if (s != NO_SLOT) st.table[s].id = new_id;
            st.m_key[new_id] = st.m_key[old_id];
            st.m_parent[new_id] = st.m_parent[old_id];
            st.m_last[new_id] = st.m_last[old_id];
            st.m_freq[new_id] = st.m_freq[old_id];
            st.m_ref[new_id] = 0;
            st.m_depth[new_id] = st.m_depth[old_id];
            st.m_flight[new_id] = a.flight_seq;
            st.m_key[old_id] = 0;
            a.desc_tier[i] = make_int2((int)old_id, (int)new_id);
            st.ring_ids[0][(u32)(((u64)head0 + count0 + i) % st.n[0])] = (int)old_id;
            if (a.victims) a.victims[i] = (int)old_id;
          }
        } else {
          int* victims = a.mode == EV_DROP ? a.victims : a.room;
          const u32 cap = st.n[tier], head = tier ? head1 : head0, count = tier ? count1 : count0;
          for (u32 i0 = blockIdx.x * EV_THREADS + (threadIdx.x & ~31u); i0 < take; i0 += G * EV_THREADS) {   // whole warps
            const u32 i = i0 + (threadIdx.x & 31u);
            const bool on = i < take;
            const u32 id = on ? (u32)(sorted[i].lo & 0xFFFFFFFFu) : 0;
            u32 visited, sid;
            const u64 key = on ? st.m_key[id] : 0;
            const u32 s = find_slot_warp(st, on, key, &visited, &sid);
            if (!on) continue;
            if (s != NO_SLOT) {                     // the slot is empty again; a group or far bit stays (lookups clear those)
              const u64 h = home_slot(key, st.slots);
              const u32 d = displacement(s, h, st.slots);
              st.table[s].id = NO_ID;
              st.table[s].key = KEY_EMPTY;
              if (d < HOP_EXACT) atomicAnd(&st.table[h].hop, ~(1u << d));
            }
            st.m_key[id] = 0;
            st.ring_ids[tier][(u32)(((u64)head + count + i) % cap)] = (int)id;
            if (victims) victims[i] = (int)id;
          }
        }
      }
    }
  }

  PHASE_MARK(st, 3);
  // ---- bookkeeping, by one thread.  Every CTA read the ring positions before its first barrier, or there was none ---------
  if (a.mode == EV_DEMOTE && a.victims && blockIdx.x == 0) {          // room-making drops are reported behind the demoted ids
    for (u32 i = threadIdx.x; i < host_dropped; i += EV_THREADS) a.victims[take + i] = a.room[i];
  }
  if (blockIdx.x == 0 && threadIdx.x == 0 && bar.ok) {
    if (st.policy && take) {                                           // GDSF clock: largest priority evicted so far
      const u64 top = a.buf[cur][take - 1].hi;
      if (top > c->inflation) c->inflation = top;
    }
    if (a.mode == EV_DEMOTE) {
      c->ring[1].head = (u32)(((u64)head1 + take) % (st.n[1] ? st.n[1] : 1));
      c->ring[1].count = count1 - take;
      c->ring[0].count = count0 + take;
      c->live[0] -= take;
      c->live[1] += take;
      c->n_pairs_tier = take;
      c->blocks_demoted += take;
      if (a.n_evicted) { a.n_evicted[0] = (int)take; a.n_evicted[1] = (int)host_dropped; }
    } else {
      c->ring[tier].count = (tier ? count1 : count0) + take;
      c->live[tier] -= take;
      c->blocks_dropped[tier] += take;
      if (a.mode == EV_DROP) { if (a.n_evicted) { a.n_evicted[0] = (int)take; a.n_evicted[1] = 0; } }
      else c->ev_host_dropped = take;
    }
  }
}

__global__ void __launch_bounds__(256) table_clear_kernel(Slot* __restrict__ table, u64 slots) {
  for (u64 s = (u64)blockIdx.x * blockDim.x + threadIdx.x; s < slots; s += (u64)gridDim.x * blockDim.x) {
    uint4 v = make_uint4(0u, 0u, NO_ID, 0u);
    *reinterpret_cast<uint4*>(table + s) = v;
  }
}

__global__ void __launch_bounds__(256) store_init_kernel(Store st, u64* __restrict__ heads) {
  const u32 total = st.n[0] + st.n[1];
  for (u32 i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    st.m_key[i] = 0; st.m_parent[i] = 0; st.m_last[i] = 0; st.m_freq[i] = 0; st.m_ref[i] = 0; st.m_depth[i] = 0; st.m_flight[i] = 0;
    heads[i] = 0;
    if (i < st.n[0]) st.ring_ids[0][i] = (int)i;
    else st.ring_ids[1][i - st.n[0]] = (int)i;
  }
}
// `progress`: the per-request progress words of the fused lookup + gather.  They carry the launch number as a tag, launch
// numbers start at 1, and the workspace may hold the words of an earlier handle: cleared here.
__global__ void ctrl_init_kernel(Store st, u64* __restrict__ progress, int n_progress) {
  Ctrl* c = st.ctrl;
  unsigned char* p = reinterpret_cast<unsigned char*>(c);
  for (size_t i = 0; i < sizeof(Ctrl); ++i) p[i] = 0;
  for (int i = 0; i < n_progress; ++i) progress[i] = 0;
  c->ring[0].count = st.n[0];
  c->ring[1].count = st.n[1];
}

// counters for a caller that does not want to block: written by the device to any device-accessible address
struct StatsOut {
  u64 epoch, live[2], free_blocks[2], max_displacement, query_blocks, probes_issued, slots_visited, blocks_matched, blocks_fetched[2],
      blocks_inserted, blocks_denied, blocks_dropped[2], blocks_demoted, far_keys, blocks_promoted, gdsf_clock, blocks_fetched_distinct;
};
__global__ void stats_kernel(Store st, u64 epoch, StatsOut* __restrict__ out) {
  const Ctrl* c = st.ctrl;
  StatsOut o;
  o.epoch = epoch;
  for (int t = 0; t < 2; ++t) {
    o.live[t] = c->live[t]; o.free_blocks[t] = c->ring[t].count;
    o.blocks_fetched[t] = c->blocks_fetched[t]; o.blocks_dropped[t] = c->blocks_dropped[t];
  }
  o.max_displacement = c->max_disp;
  o.query_blocks = c->query_blocks; o.probes_issued = c->probes_issued; o.slots_visited = c->slots_visited; o.blocks_matched = c->blocks_matched;
  for (int i = 0; i < LOOKUP_STRIPES; ++i) {
    o.query_blocks += c->lookup_stripes[i][0]; o.probes_issued += c->lookup_stripes[i][1];
    o.slots_visited += c->lookup_stripes[i][2]; o.blocks_matched += c->lookup_stripes[i][3];
  }
  o.blocks_inserted = c->blocks_inserted; o.blocks_denied = c->blocks_denied; o.blocks_demoted = c->blocks_demoted;
  o.far_keys = c->far_keys; o.blocks_promoted = c->blocks_promoted; o.gdsf_clock = c->inflation;
  o.blocks_fetched_distinct = c->blocks_fetched_distinct;
  *out = o;
}

}  // namespace pts
