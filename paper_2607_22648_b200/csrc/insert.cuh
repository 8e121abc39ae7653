// Scatter-insert of new blocks (store operation: only the increment after the longest common prefix
// is saved and appended to the trie, paper Section 4 summary paragraph and Section 4.1).
//
// The batch must behave as if requests were inserted one after the other in index order.  All the
// metadata work of a call runs in ONE cooperative kernel whose phases are separated by grid-wide
// barriers (elements e = (request r, block j), R*max_blocks of them):
//   hash    : chained block keys (content hashes first, by one thread per block, when requests are few
//             and long); serial along a request
//   claim   : find the key of e in the table or claim the first empty slot at or after its home slot
//             (atomicCAS on the key); every element that lands on a slot claimed in this call lowers
//             slot.id to ID_PENDING | its request index (atomicMin), so the lowest request presenting a
//             new prefix becomes its creator.
//   count   : flag(e) = "e creates a node"; sums per tile of 1024 elements.
//   assign  : every CTA derives the allocation plan from the tile sums (grants = min(new nodes, free HBM
//             blocks)); rank(e) among creators in (r, j) order; rank < grants gets ring[head + rank],
//             writes the slot value, flags the slot in its home slot's hop word, writes the node's
//             metadata and a copy descriptor; the others empty their slot again.
//   finish  : every element reads its slot's block id (or -1) and refreshes the LRU stamp.
// Ranking creators in (r, j) order and granting the first `free` of them equals the sequential rule:
// a denied node's descendants always rank higher, so denials are prefix-closed per request.
#pragma once
#include "common.cuh"
#include "lookup.cuh"
#include "evict.cuh"

namespace pts {

constexpr int INS_THREADS = 1024;

__device__ __forceinline__ u32 creator_flag(const Store& st, const u32* __restrict__ eslot, long long e, int max_blocks) {
  const u32 s = eslot[e];
  if (s == NO_SLOT) return 0;
  const Slot v = load_slot(st.table + s);
  return v.id == (ID_PENDING | (u32)(e / max_blocks)) ? 1u : 0u;
}

// block-wide inclusive scan of one value per thread (INS_THREADS threads); returns inclusive sum, total in *total
__device__ __forceinline__ u32 block_scan_incl(u32 x, u32* warp_sums, u32* total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
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
  *total = warp_sums[31];
  __syncthreads();                       // warp_sums may be reused by the caller's next scan
  return incl;
}

// Find `key` or claim a slot for it; the lowest request index presenting a key claimed in this call owns it.
// First the lookup proper (home slot, flagged slots): a key stored by an earlier call is found there and nowhere else.
// A new key then takes the first empty slot at or after its home slot.  The walk reads PROBE_WINDOW slots at a time
// and compares every key it passes, because another element of this call may be claiming the same key at the same
// time: all of them walk the same slots in the same order, an empty slot is never passed over but claimed with a
// compare-and-swap whose result says what the slot really holds, and during this phase a slot only ever changes from
// empty to a key - so the first claim is seen by everyone who comes later.  (Keys claimed in this call are flagged in
// their home slots only when they are granted a block, after the phase.)
// Called by all 32 lanes of a warp together (lanes without an element pass active = false).
__device__ __forceinline__ u32 claim_slot(const Store& st, bool active, u64 key, u32 r) {
  ProbeWindow w;
  if (active) probe_issue(st, key, w);
  u32 visited, got;
  const u32 id = probe_finish_warp(st, active, key, w, &visited, &got);
  if (!active) return NO_SLOT;
  if (id != NO_ID) return got;                       // an existing node
  got = NO_SLOT;
  u64 s = home_slot(key, st.slots);
  for (u64 i = 0; i < st.slots && got == NO_SLOT; i += PROBE_WINDOW) {
    u64 k[PROBE_WINDOW], idx[PROBE_WINDOW];
#pragma unroll
    for (int x = 0; x < PROBE_WINDOW; ++x) {
      idx[x] = wrap_slot(s + x, st.slots);
      k[x] = *reinterpret_cast<volatile u64*>(&st.table[idx[x]].key);
    }
    if (i == 0) { k[0] = slot_key(w.v0); k[1] = slot_key(w.v1); k[2] = slot_key(w.v2); k[3] = slot_key(w.v3); }   // read already
#pragma unroll
    for (int x = 0; x < PROBE_WINDOW; ++x) {
      if (got != NO_SLOT) break;
      u64 kk = k[x];
      if (kk == KEY_EMPTY) {
        kk = atomicCAS(&st.table[idx[x]].key, KEY_EMPTY, key);
        if (kk == KEY_EMPTY) kk = key;                 // claimed
      }
      if (kk == key) got = (u32)idx[x];
    }
    s = wrap_slot(s + PROBE_WINDOW, st.slots);
  }
  if (got == NO_SLOT) { raise(st, S_TABLE_FULL); return got; }
  atomicMin(&st.table[got].id, ID_PENDING | r);        // NO_ID or another request's mark: the lowest request stays
  return got;
}

struct InsertArgs {
  const int* tokens;
  const long long* offsets;
  int R, max_blocks;
  int split;                // 1: content hashes first, one thread per block (few long requests); needs L == 32
  const u32* hashed;        // non-null (L == 32 only): keys[r][0 .. hashed[r]) already hold the chained keys of request r,
                            // left there by the lookup of the same batch; hashing resumes behind them
  u64* keys;                // scratch [R*max_blocks]
  u32* eslot;               // scratch [R*max_blocks]
  u32* cta_sums;            // scratch [tiles]
  const int* bt;            // block tables of the source cache, or null (metadata only)
  u32 cache_blocks;
  u64 epoch;
  int2* desc;               // out: copy descriptors {pool block, cache block}, ctrl->n_pairs of them
  int* ids_out;
  int* new_blocks;
  u32 launch_seq;
};

template <int L>
__global__ void __launch_bounds__(INS_THREADS) insert_kernel(Store st, InsertArgs a) {
  __shared__ u32 warp_sums[32];
  constexpr int G = 32 / L;
  Ctrl* c = st.ctrl;
  GridBarrier bar;
  bar.init(c, a.launch_seq);
  const int lane = threadIdx.x & 31, sl = lane & (L - 1), sub = lane / L;
  const long long total = (long long)a.R * a.max_blocks;
  const int max_blocks = a.max_blocks;
  // plan inputs, read before anything in this launch changes them
  const u32 head0 = c->ring[0].head, count0 = c->ring[0].count;
  const u64 inflation = st.policy ? c->inflation : 0;
  const long long gthreads = (long long)gridDim.x * INS_THREADS;
  const long long gtid = (long long)blockIdx.x * INS_THREADS + threadIdx.x;

  PHASE_MARK(st, 0);
  PHASE_MARK(st, 1);

  // ---- hash + claim ----------------------------------------------------------------------------------------------------
  if (a.split) {
    for (long long e = gtid; e < total; e += gthreads) {
      const int r = (int)(e / max_blocks), j = (int)(e % max_blocks);
      if (j < full_blocks(a.offsets, r, st.block_tokens, max_blocks) && !(a.hashed && (u32)j < a.hashed[r]))
        a.keys[e] = content_block(a.tokens + a.offsets[r] + (long long)j * st.block_tokens, st.block_tokens);
    }
    bar.sync(st);
  }
  PHASE_MARK(st, 2);
  {
    // warp w of CTA b takes request groups w * gridDim + b, ...: consecutive groups go to different SMs, because a chain is
    // a long dependent instruction sequence and many of them on one SM queue for its issue slots
    const long long warps = gthreads >> 5, warp0 = (long long)(threadIdx.x >> 5) * gridDim.x + blockIdx.x;
    const long long groups = ((long long)a.R + G - 1) / G;
    for (long long grp = warp0; grp < groups && bar.ok; grp += warps) {
      const long long r = grp * G + sub;
      const bool valid = r < a.R;
      const int nblk = valid ? full_blocks(a.offsets, (int)r, st.block_tokens, max_blocks) : 0;
      const long long tok0 = valid ? a.offsets[r] : 0;
      u64 parent = st.root_key;
      const int most = __reduce_max_sync(FULL, nblk);
      int base0 = 0;
      if (L == 32 && a.hashed && valid) {               // a warp per request: resume behind the keys the lookup left
        const int have = (int)a.hashed[r];
        base0 = have < nblk ? have : nblk;              // a multiple of 32, or all of the request
        if (base0 > 0) parent = a.keys[r * max_blocks + base0 - 1];
      }
      for (int base = base0; base < most; base += L) {
        const int j = base + sl;
        const bool active = j < nblk;
        u64 cc = 0;
        if (active) cc = a.split ? a.keys[r * max_blocks + j] : content_block(a.tokens + tok0 + (long long)j * st.block_tokens, st.block_tokens);
        const int steps = most - base < L ? most - base : L;
        const u64 key = chain_chunk<L>(parent, cc, lane, steps);
        if (active) a.keys[r * max_blocks + j] = key;
        parent = __shfl_sync(FULL, key, (lane & ~(L - 1)) + L - 1);
      }
      if (valid) {
        for (int j = nblk + sl; j < max_blocks; j += L) a.keys[r * max_blocks + j] = 0;
        if (sl == 0) a.new_blocks[r] = 0;
      }
    }
  }
  bar.sync(st);
  PHASE_MARK(st, 3);
  // the chain is serial per request, the claims are not: one element per thread, so that the probe latencies overlap
  for (long long e0 = gtid - lane; e0 < total && bar.ok; e0 += gthreads) {        // whole warps: claim_slot wants all lanes
    const long long e = e0 + lane;
    const u64 key = e < total ? a.keys[e] : 0;
    const u32 s = claim_slot(st, key != 0, key, (u32)(e / max_blocks));
    if (e < total) a.eslot[e] = s;
  }
  bar.sync(st);
  PHASE_MARK(st, 4);

  // ---- count -----------------------------------------------------------------------------------------------------------
  const long long n_tiles = (total + INS_THREADS - 1) / INS_THREADS;
  for (long long t = blockIdx.x; t < n_tiles && bar.ok; t += gridDim.x) {
    const long long e = t * INS_THREADS + threadIdx.x;
    const u32 f = e < total ? creator_flag(st, a.eslot, e, max_blocks) : 0;
    u32 sum;
    block_scan_incl(f, warp_sums, &sum);
    if (threadIdx.x == 0) a.cta_sums[t] = sum;
  }
  bar.sync(st);
  PHASE_MARK(st, 5);

  // ---- plan (the same in every CTA) and assign -------------------------------------------------------------------------
  u32 total_new;
  {
    u32 part = 0;
    for (long long i = threadIdx.x; i < n_tiles; i += INS_THREADS) part += a.cta_sums[i];
    block_scan_incl(part, warp_sums, &total_new);
  }
  const u32 granted = total_new < count0 ? total_new : count0;
  if (blockIdx.x == 0 && threadIdx.x == 0 && bar.ok) {
    c->ins_total_new = total_new;
    c->ins_granted = granted;
    c->ins_base = head0;
    c->ring[0].head = (u32)(((u64)head0 + granted) % st.n[0]);
    c->ring[0].count = count0 - granted;
    c->live[0] += granted;
    c->n_pairs = granted;
    c->blocks_inserted += granted;
    c->blocks_denied += total_new - granted;
    if (granted < total_new) atomicOr(&c->status, S_NOSPACE);
  }
  for (long long t = blockIdx.x; t < n_tiles && bar.ok; t += gridDim.x) {
    u32 before;                                   // creators in earlier tiles
    {
      u32 part = 0;
      for (long long i = threadIdx.x; i < t; i += INS_THREADS) part += a.cta_sums[i];
      block_scan_incl(part, warp_sums, &before);
    }
    const long long e = t * INS_THREADS + threadIdx.x;
    const u32 f = e < total ? creator_flag(st, a.eslot, e, max_blocks) : 0;
    u32 sum;
    const u32 incl = block_scan_incl(f, warp_sums, &sum);
    if (!f) continue;
    const u32 rank = before + incl - 1;
    Slot* slot = st.table + a.eslot[e];
    if (rank >= granted) {                       // denied: the slot is empty again (nobody walks the table in this phase)
      slot->id = NO_ID;
      slot->key = KEY_EMPTY;
      continue;
    }
    const u32 id = (u32)st.ring_ids[0][(u32)(((u64)head0 + rank) % st.n[0])];
    const int j = (int)(e % max_blocks);
    st.m_key[id] = a.keys[e];
    st.m_parent[id] = j ? a.keys[e - 1] : st.root_key;
    st.m_last[id] = st.policy ? 0 : a.epoch;    // GDSF: the finish phase counts this call's accesses
    st.m_freq[id] = 0;
    st.m_ref[id] = 0;
    st.m_depth[id] = (u32)j;
    slot->id = id;
    {                                            // make the key findable: flag its slot in the home slot's hop word
      const u64 h = home_slot(a.keys[e], st.slots);
      const u32 d = displacement(a.eslot[e], h, st.slots);
      atomicOr(&st.table[h].hop, hop_bit(d));
      if (d >= HOP_EXACT) { atomicMax(&c->max_disp, d); atomicAdd(&c->far_keys, 1ull); }
    }
    int2 d = make_int2((int)id, 0);
    if (a.bt) {
      const int cb = a.bt[e];
      if (cb < 0 || (u32)cb >= a.cache_blocks) { raise(st, S_BOUNDS); d.x = -1; }
      d.y = cb;
    } else {
      d.x = -1;                                  // metadata-only insert: nothing to copy
    }
    a.desc[rank] = d;
    atomicAdd(&a.new_blocks[e / max_blocks], 1);
  }
  PHASE_MARK(st, 6);
  bar.sync(st);
  PHASE_MARK(st, 7);

  // ---- finish ----------------------------------------------------------------------------------------------------------
  for (long long e = gtid; e < total && bar.ok; e += gthreads) {
    const u32 s = a.eslot[e];
    int out = -1;
    if (s != NO_SLOT) {
      const u32 id = st.table[s].id;
      if (id < ID_PENDING) { out = (int)id; touch_block(st, id, a.epoch, inflation, 1); }
    }
    a.ids_out[e] = out;
  }
  PHASE_MARK(st, 8);
}

}  // namespace pts
