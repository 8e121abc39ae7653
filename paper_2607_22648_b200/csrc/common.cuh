// Shared device-side definitions of the prefix tensor store: table slot, per-block metadata views,
// control block, chained block hash.  Everything here is sm_100a device code or POD shared with the
// host side of the same library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace pts {

typedef unsigned long long u64;
typedef unsigned int u32;
constexpr unsigned FULL = 0xFFFFFFFFu;   // all lanes of a warp

// ---- hash table slot ------------------------------------------------------------------------------
// 16 bytes, loaded with one 128-bit access.  key 0 = empty (keys 0 and 1 are never produced by the hash).
// Keys are placed by linear probing (the first empty slot at or after the home slot), but a lookup does not walk the run:
// `hop` of a slot says where the keys that have THIS slot as their home sit -
//   bit d, d = 0..23          : slot home + d
//   bit 24 + g, g = 0..6      : somewhere in the 32 slots from home + 24 + 32 g
//   bit 31                    : 248 or more slots away (every slot from there to the largest distance ever used is compared)
// - so a lookup reads the home slot with its neighbours and then exactly the flagged slots, and a miss costs the same one
// round trip as a hit (at load factor 0.7 about one key in 250 sits 24 or more slots from home).  Nothing depends on runs
// being unbroken, so a deleted key simply leaves an empty slot: no deleted markers, no rebuilds.  Deleting clears an exact
// bit; a group bit or the far bit is cleared by the next lookup that follows it and finds no key of this home there.
// id: the block of the node; NO_ID in an empty slot; ID_PENDING | r while an insert that has claimed the slot in this
// call has not been granted its block yet (r = lowest request index that presented the key).
struct __align__(16) Slot {
  u64 key;
  u32 id;
  u32 hop;
};
constexpr u64 KEY_EMPTY = 0ull;
constexpr u32 ID_PENDING = 0x80000000u;     // block ids are below this
constexpr u32 HOP_EXACT = 24;               // displacements below this have a bit of their own
constexpr u32 HOP_GROUP = 32;               // slots per group bit
constexpr u32 HOP_GROUPS = 7;
constexpr u32 HOP_FAR_FROM = HOP_EXACT + HOP_GROUP * HOP_GROUPS;   // 248
constexpr u32 HOP_FAR = 0x80000000u;        // bit 31 of hop
__host__ __device__ __forceinline__ u32 hop_bit(u32 d) {
  return d < HOP_EXACT ? 1u << d : d < HOP_FAR_FROM ? 1u << (HOP_EXACT + (d - HOP_EXACT) / HOP_GROUP) : HOP_FAR;
}
constexpr u32 NO_ID = 0xFFFFFFFFu;
constexpr u32 NO_SLOT = 0xFFFFFFFFu;
constexpr u32 LINK_NIL = 0xFFFFFFFFu;  // end of a destination list (fetch)

// ---- status bits / flags (mirror include/ptstore.h) -------------------------------------------------
constexpr u32 S_NOSPACE = 1u, S_TABLE_FULL = 2u, S_BOUNDS = 4u, S_STATE = 8u, S_TIMEOUT = 16u, S_INFLIGHT = 32u;
constexpr u32 F_PIN = 1u, F_NO_TOUCH = 2u;

// ---- control block in device memory ----------------------------------------------------------------
constexpr int LOOKUP_STRIPES = 64;
struct Ring {
  u32 head;     // position of the next id to hand out
  u32 count;    // ids available
};
struct Ctrl {
  Ring ring[2];
  u32 status;
  u32 pad0;
  // per-call scalars produced by one kernel and consumed by the next
  u32 n_pairs;          // insert / promote: entries in the copy descriptor list
  u32 n_pairs_tier;     // demotion: entries in its own descriptor list (its copy may run on the library's side stream)
  u32 ins_total_new;    // insert: new unique nodes presented
  u32 ins_granted;      // insert / promote: of those, how many got a block
  u32 ins_base;         // insert / promote: ring head before this call
  u32 ev_take;          // promote: where the freed host ids go in the host ring
  u32 ev_host_dropped;  // evict: host-tier drops that made room for a demotion
  u32 live[2];
  u32 max_disp;         // largest distance from its home slot at which a key has ever been placed (0 while below HOP_EXACT)
  u32 pad1;
  // fetch: per-call scalars, double buffered by the call's sequence number so that no launch is needed to clear them:
  // call k uses entry k & 1 and zeroes entry (k + 1) & 1 for the call after it
  u32 f_pairs[2];       // distinct HBM-tier source blocks = entries of the descriptor list
  u32 f_pairs_host[2];  // distinct host-tier source blocks (a descriptor list of their own)
  u32 f_work[2];        // next work unit to hand out (dynamic dealing inside the copy kernel)
  u32 pad2[2];
  // arrival counters of the grid-wide barriers of cooperative kernels: launch k uses entry k % BAR_SLOTS and zeroes
  // the entry half a ring ahead, so a counter is always zero when its turn comes, whatever happened to earlier launches
  u32 bar[64];
#ifdef PTS_PHASE_TIMERS
  u64 phase_ns[16];     // diagnostic build only: globaltimer at phase boundaries of the last cooperative kernel
#endif
  // cumulative counters
  u64 query_blocks, probes_issued, slots_visited, blocks_matched;   // totals are these plus the stripes below
  u64 blocks_fetched[2];
  u64 blocks_inserted, blocks_denied;
  u64 blocks_dropped[2];
  u64 blocks_demoted;
  u64 far_keys;         // keys placed HOP_EXACT or more slots from home so far
  u64 blocks_promoted;
  u64 inflation;        // GDSF clock L: largest priority evicted so far
  u64 blocks_fetched_distinct;   // distinct source blocks read by fetch calls (<= blocks fetched)
  // lookup counters are striped so that thousands of warps do not queue on four addresses;
  // [stripe][0..3] = query blocks, probes issued, slots visited, blocks matched
  u64 lookup_stripes[LOOKUP_STRIPES][4];
};

// ---- everything a kernel needs to know about the store ---------------------------------------------
struct Store {
  Slot* table;          // current table
  u64 slots;
  // per-block metadata, indexed by block id (both tiers)
  u64* m_key;           // 0 = block not live
  u64* m_parent;        // key of the parent node (root key for depth 0)
  u64* m_last;          // LRU policy: stamp of the last touch; GDSF policy: priority H = L + F at the last touch
  u32* m_freq;          // GDSF policy: access count F
  u32* m_ref;
  u32* m_depth;
  u32* m_flight;        // host-tier blocks: tag of the asynchronous demotion that last wrote the block (0 = none)
  int* ring_ids[2];
  u32 n[2];             // blocks per tier
  Ctrl* ctrl;
  unsigned char* pool[2];
  u64 chunk_bytes, block_bytes;
  u32 layers;
  u32 block_tokens;
  u64 root_key;
  u32 policy;           // 0 = LRU, 1 = GDSF (equal size and cost per block)
};

// ---- chained block hash -----------------------------------------------------------------------------
// The paper gives each tensor a unique id that an object inherits from its longest common prefix
// (Section 4.1).  Here the id of a block is a 64-bit key that folds in the key of the parent block,
// so equal prefixes give equal key sequences and the trie becomes a flat table of keys.
constexpr u64 HC1 = 0x9E3779B97F4A7C15ull;   // floor(2^64 / golden ratio)
constexpr u64 HC2 = 0x6A09E667F3BCC909ull;   // frac(sqrt 2) * 2^64, low bit set
constexpr u64 HC3 = 0xBB67AE8584CAA73Bull;   // frac(sqrt 3) * 2^64
constexpr u64 HC5 = 0x3C6EF372FE94F82Bull;   // frac(sqrt 5) * 2^64

__host__ __device__ __forceinline__ u64 hmix(u64 x) {
  x ^= x >> 32; x *= HC3;
  x ^= x >> 29; x *= HC5;
  x ^= x >> 32;
  return x;
}
__host__ __device__ __forceinline__ u64 hfix(u64 k) { return k < 2 ? k + 2 : k; }
__host__ __device__ __forceinline__ u64 hroot(u64 salt) { return hfix(hmix(salt ^ HC2)); }
__host__ __device__ __forceinline__ u64 hchain(u64 parent, u64 content) { return hfix(hmix(parent * HC1 + content)); }
__device__ __forceinline__ u64 htoken(int tok, u32 pos) {
  return hmix((((u64)pos << 32) | (u64)(u32)tok) ^ HC1);
}

// content hash of one block by ONE thread; 16-byte loads when the block start allows it
__device__ __forceinline__ u64 content_block(const int* __restrict__ t, u32 B) {
  u64 s = 0;
  if (((B & 3u) == 0) && ((reinterpret_cast<uintptr_t>(t) & 15u) == 0)) {
    const int4* t4 = reinterpret_cast<const int4*>(t);
    for (u32 j = 0; j < B / 4; ++j) {
      int4 v = __ldg(t4 + j);
      s += htoken(v.x, 4 * j) + htoken(v.y, 4 * j + 1) + htoken(v.z, 4 * j + 2) + htoken(v.w, 4 * j + 3);
    }
  } else {
    for (u32 j = 0; j < B; ++j) s += htoken(__ldg(t + j), j);
  }
  return s;
}

// ---- table probing ----------------------------------------------------------------------------------
__device__ __forceinline__ u64 home_slot(u64 key, u64 slots) { return __umul64hi(key, slots); }

__device__ __forceinline__ Slot load_slot(const Slot* p) {
  uint4 v = *reinterpret_cast<const uint4*>(p);
  Slot s;
  s.key = ((u64)v.y << 32) | v.x;
  s.id = v.z;
  s.hop = v.w;
  return s;
}
__device__ __forceinline__ u64 wrap_slot(u64 t, u64 slots) { return t >= slots ? t - slots : t; }   // t < 2 * slots
__device__ __forceinline__ u32 displacement(u64 slot, u64 home, u64 slots) { return (u32)(slot >= home ? slot - home : slot + slots - home); }

// Lookup of `key` (see Slot).  One round trip loads the home slot - whose hop word names the slots that matter - and
// its three neighbours; keys placed further away cost a second round trip for exactly the flagged slots or groups.
// Split in two so that a caller can put independent work between the loads and their use.  *visited gets the slots
// compared; the slot index is returned through *slot_out when asked for.
constexpr int PROBE_WINDOW = 4;
struct ProbeWindow { uint4 v0, v1, v2, v3; };       // named members: an indexed array ended up in local memory
__device__ __forceinline__ void probe_issue(const Store& st, u64 key, ProbeWindow& w) {
  const u64 h = home_slot(key, st.slots);
  w.v0 = *reinterpret_cast<const uint4*>(st.table + h);
  w.v1 = *reinterpret_cast<const uint4*>(st.table + wrap_slot(h + 1, st.slots));
  w.v2 = *reinterpret_cast<const uint4*>(st.table + wrap_slot(h + 2, st.slots));
  w.v3 = *reinterpret_cast<const uint4*>(st.table + wrap_slot(h + 3, st.slots));
}
__device__ __forceinline__ u64 slot_key(const uint4& v) { return ((u64)v.y << 32) | v.x; }

// The near part of a lookup, from the loaded window: the flagged slots up to HOP_EXACT - 1 from home.  Returns the id or
// NO_ID; *far_bits gets the group / far bits that still have to be followed when the key was not found (0 = it is absent).
__device__ __forceinline__ u32 probe_near(const Store& st, u64 key, const ProbeWindow& w, u32* compared, u32* slot_out, u32* far_bits) {
  const u64 h = home_slot(key, st.slots);
  const u32 bits = w.v0.w;
  u32 n = 0;
  *far_bits = 0;
  if (bits & 1u) { ++n; if (slot_key(w.v0) == key) { *compared = n; *slot_out = (u32)h; return w.v0.z; } }
  if (bits & 2u) { ++n; if (slot_key(w.v1) == key) { *compared = n; *slot_out = (u32)wrap_slot(h + 1, st.slots); return w.v1.z; } }
  if (bits & 4u) { ++n; if (slot_key(w.v2) == key) { *compared = n; *slot_out = (u32)wrap_slot(h + 2, st.slots); return w.v2.z; } }
  if (bits & 8u) { ++n; if (slot_key(w.v3) == key) { *compared = n; *slot_out = (u32)wrap_slot(h + 3, st.slots); return w.v3.z; } }
  u32 rest = bits & ((1u << HOP_EXACT) - 1u) & ~((1u << PROBE_WINDOW) - 1u);
  while (rest) {                                   // the flagged slots beyond the window, up to four loads in flight
    const int d0 = __ffs(rest) - 1; rest &= rest - 1;
    const int d1 = rest ? __ffs(rest) - 1 : d0; rest &= rest - 1;
    const int d2 = rest ? __ffs(rest) - 1 : d0; rest &= rest - 1;
    const int d3 = rest ? __ffs(rest) - 1 : d0; rest &= rest - 1;
    const u32 a0 = (u32)wrap_slot(h + d0, st.slots), a1 = (u32)wrap_slot(h + d1, st.slots);
    const u32 a2 = (u32)wrap_slot(h + d2, st.slots), a3 = (u32)wrap_slot(h + d3, st.slots);
    const uint4 q0 = *reinterpret_cast<const uint4*>(st.table + a0);
    const uint4 q1 = *reinterpret_cast<const uint4*>(st.table + a1);      // a repeat of the first slot when fewer are flagged
    const uint4 q2 = *reinterpret_cast<const uint4*>(st.table + a2);
    const uint4 q3 = *reinterpret_cast<const uint4*>(st.table + a3);
    n += 1u + (d1 != d0) + (d2 != d0) + (d3 != d0);
    if ((((u64)q0.y << 32) | q0.x) == key) { *compared = n; *slot_out = a0; return q0.z; }
    if ((((u64)q1.y << 32) | q1.x) == key) { *compared = n; *slot_out = a1; return q1.z; }
    if ((((u64)q2.y << 32) | q2.x) == key) { *compared = n; *slot_out = a2; return q2.z; }
    if ((((u64)q3.y << 32) | q3.x) == key) { *compared = n; *slot_out = a3; return q3.z; }
  }
  *compared = n ? n : 1;
  *slot_out = NO_SLOT;
  *far_bits = bits & ~((1u << HOP_EXACT) - 1u);
  return NO_ID;
}

// The rare part: a group of HOP_GROUP slots per group bit, and for the far bit every slot from HOP_FAR_FROM to the largest
// distance ever used.  When a range holds no key of this home, the bit that sent the lookup there is cleared in the home's
// hop word, so that the next lookup of a key that hashes here is short again.  Only lookups and deletions run beside a
// lookup, never insertions, and neither can make "no key of this home is left there" false; during an insert's claim
// phase the keys claimed so far are in the table already and count.
//
// Two forms.  probe_far_warp: ALL 32 lanes of a warp call it together; the lanes that have bits to follow are served
// one after the other, each by the whole warp - one slot per lane, one round trip per 32 slots, no arrays in registers.
// probe_far_lane: any single thread, four loads in flight; out of line and by value so that it costs its callers
// nothing but a branch.
__device__ __forceinline__ void probe_far_warp(const Store& st, u64 key, u32 far_bits, u32* id, u32* slot, u32* compared) {
  const int lane = threadIdx.x & 31;
  const u64 h = home_slot(key, st.slots);
  for (unsigned pending = __ballot_sync(FULL, far_bits != 0); pending; pending &= pending - 1) {
    const int src = __ffs(pending) - 1;
    const u64 k0 = __shfl_sync(FULL, key, src), h0 = __shfl_sync(FULL, h, src);
    const u32 b0 = __shfl_sync(FULL, far_bits, src);
    u32 found_id = NO_ID, found_slot = NO_SLOT, cmp = 0;
    const u32 last = (b0 & HOP_FAR) ? *reinterpret_cast<volatile u32*>(&st.ctrl->max_disp) : 0;
    bool far_has_own = false;
    // ranges of 32 slots: the flagged groups, then (far bit) HOP_FAR_FROM ... last
    u32 groups = (b0 >> HOP_EXACT) & ((1u << HOP_GROUPS) - 1u);
    u32 d0 = HOP_FAR_FROM;
    while (found_id == NO_ID) {
      u32 base, heal;
      if (groups) { const u32 g = (u32)__ffs(groups) - 1; groups &= groups - 1; base = HOP_EXACT + g * HOP_GROUP; heal = 1u << (HOP_EXACT + g); }
      else if ((b0 & HOP_FAR) && d0 <= last) { base = d0; d0 += 32; heal = 0; }
      else break;
      const u32 d = base + lane;
      const bool in = heal ? true : d <= last;
      const u32 at = (u32)((h0 + d) % st.slots);
      uint4 v = make_uint4(0u, 0u, NO_ID, 0u);
      if (in) v = *reinterpret_cast<const uint4*>(st.table + at);
      const u64 kk = ((u64)v.y << 32) | v.x;
      const unsigned hit = __ballot_sync(FULL, in && kk == k0);
      const unsigned own = __ballot_sync(FULL, in && kk >= 2 && home_slot(kk, st.slots) == h0);
      cmp += heal ? 32 : (last - base + 1 < 32 ? last - base + 1 : 32);
      if (hit) {
        const int l = __ffs(hit) - 1;
        found_id = __shfl_sync(FULL, v.z, l);
        found_slot = __shfl_sync(FULL, at, l);
      } else if (heal) {
        if (!own && lane == 0) atomicAnd(&st.table[h0].hop, ~heal);
      } else if (own) {
        far_has_own = true;
      }
    }
    if (found_id == NO_ID && (b0 & HOP_FAR) && !far_has_own && lane == 0) atomicAnd(&st.table[h0].hop, ~HOP_FAR);
    if (lane == src) { *id = found_id; *slot = found_slot; *compared += cmp; }
  }
}
__device__ __noinline__ uint4 probe_far_lane(Slot* table, u64 slots, const u32* max_disp, u64 key, u64 h, u32 far_bits) {
  constexpr int B = 4;
  u32 compared = 0;
  u32 groups = (far_bits >> HOP_EXACT) & ((1u << HOP_GROUPS) - 1u);
  bool far_done = !(far_bits & HOP_FAR);
  while (groups || !far_done) {
    u32 d0, len, heal;
    if (groups) { const u32 g = (u32)__ffs(groups) - 1; groups &= groups - 1; d0 = HOP_EXACT + g * HOP_GROUP; len = HOP_GROUP; heal = 1u << (HOP_EXACT + g); }
    else {
      far_done = true;
      const u32 last = *reinterpret_cast<const volatile u32*>(max_disp);
      if (last < HOP_FAR_FROM) break;
      d0 = HOP_FAR_FROM; len = last - HOP_FAR_FROM + 1; heal = HOP_FAR;
    }
    bool any_of_this_home = false;
    u64 s = (h + d0) % slots;                          // one division here, none per slot
    for (u32 d = 0; d < len; d += B) {
      u64 k[B];
      const u64 s0 = s;
#pragma unroll
      for (int x = 0; x < B; ++x) {
        k[x] = d + x < len ? table[s].key : KEY_EMPTY;
        s = s + 1 == slots ? 0 : s + 1;
      }
#pragma unroll
      for (int x = 0; x < B; ++x) {
        if (d + x >= len) break;
        ++compared;
        if (k[x] == key) {
          const u32 at = (u32)((s0 + x) % slots);
          return make_uint4(table[at].id, at, compared, 0);
        }
        if (k[x] >= 2 && home_slot(k[x], slots) == h) any_of_this_home = true;
      }
    }
    if (!any_of_this_home) atomicAnd(&table[h].hop, ~heal);
  }
  return make_uint4(NO_ID, NO_SLOT, compared, 0);
}

// The whole lookup for one thread on its own ...
__device__ __forceinline__ u32 probe_finish(const Store& st, u64 key, const ProbeWindow& w, u32* visited, u32* slot_out = nullptr) {
  u32 slot, far_bits;
  u32 id = probe_near(st, key, w, visited, &slot, &far_bits);
  if (far_bits) {
    const uint4 r = probe_far_lane(st.table, st.slots, &st.ctrl->max_disp, key, home_slot(key, st.slots), far_bits);
    id = r.x; slot = r.y; *visited += r.z;
  }
  if (slot_out) *slot_out = slot;
  return id;
}
// ... and for the 32 lanes of a warp together (lanes with `active` false take part without a key of their own)
__device__ __forceinline__ u32 probe_finish_warp(const Store& st, bool active, u64 key, const ProbeWindow& w, u32* visited, u32* slot_out = nullptr) {
  u32 slot = NO_SLOT, far_bits = 0, id = NO_ID;
  *visited = 0;
  if (active) id = probe_near(st, key, w, visited, &slot, &far_bits);
  if (__any_sync(FULL, far_bits != 0)) probe_far_warp(st, key, far_bits, &id, &slot, visited);
  if (slot_out) *slot_out = slot;
  return id;
}

// slot of `key`, or NO_SLOT
__device__ __forceinline__ u32 find_slot(const Store& st, u64 key, u32* visited, u32* id_out) {
  ProbeWindow w;
  probe_issue(st, key, w);
  u32 slot;
  *id_out = probe_finish(st, key, w, visited, &slot);
  return slot;
}
__device__ __forceinline__ u32 find_slot_warp(const Store& st, bool active, u64 key, u32* visited, u32* id_out) {
  ProbeWindow w;
  probe_issue(st, active ? key : 0, w);          // lanes without a key read the first slots of the table and ignore them
  u32 slot;
  *id_out = probe_finish_warp(st, active, key, w, visited, &slot);
  return slot;
}

__device__ __forceinline__ int tier_of(const Store& st, u32 id) { return id < st.n[0] ? 0 : 1; }
__device__ __forceinline__ unsigned char* block_ptr(const Store& st, u32 id) {
  return id < st.n[0] ? st.pool[0] + (u64)id * st.block_bytes : st.pool[1] + (u64)(id - st.n[0]) * st.block_bytes;
}

__device__ __forceinline__ void raise(const Store& st, u32 bit) { atomicOr(&st.ctrl->status, bit); }

#ifdef PTS_PHASE_TIMERS
__device__ __forceinline__ void phase_mark(const Store& st, int i) {
  if (blockIdx.x == 0 && threadIdx.x == 0) { u64 t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); st.ctrl->phase_ns[i] = t; }
}
#define PHASE_MARK(st, i) phase_mark(st, i)
#else
#define PHASE_MARK(st, i)
#endif

// ---- grid-wide barrier for cooperative launches ---------------------------------------------------------------------
// All CTAs of a cooperative launch are resident at once, so they may wait for one another.  Every CTA calls sync() the
// same number of times; the k-th call returns once all CTAs have made their k-th call.  The wait is bounded: after
// GRID_POLL_LIMIT polls the CTA raises S_TIMEOUT and sync() returns false from then on without waiting (callers stop
// touching shared state and fall through to the end of the kernel).
constexpr int BAR_SLOTS = 64;
constexpr u32 GRID_POLL_LIMIT = 1u << 24;
struct GridBarrier {
  u32* counter;
  u32 arrived;      // arrivals expected by the end of the next sync(): gridDim.x * (calls so far + 1)
  bool ok;
  __device__ __forceinline__ void init(Ctrl* c, u32 launch_seq) {
    counter = &c->bar[launch_seq % BAR_SLOTS];
    arrived = 0;
    ok = true;
    if (blockIdx.x == 0 && threadIdx.x == 0) c->bar[(launch_seq + BAR_SLOTS / 2) % BAR_SLOTS] = 0;
  }
  __device__ __forceinline__ bool sync(const Store& st) {
    arrived += gridDim.x;
    if (gridDim.x == 1) { __syncthreads(); return ok; }
    __syncthreads();
    if (threadIdx.x == 0 && ok) {
      __threadfence();
      atomicAdd(counter, 1u);
      u32 polls = 0;
      while (true) {
        u32 seen;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
        if (seen >= arrived) break;
        if (++polls >= GRID_POLL_LIMIT) { ok = false; raise(st, S_TIMEOUT); break; }
        __nanosleep(32);
      }
      __threadfence();
    }
    ok = __syncthreads_and(ok ? 1 : 0) != 0;
    return ok;
  }
};

// `count` accesses to block `id` in the call with stamp `epoch` (paper Section 1: LRU; Section 4.1 "Access
// pattern-aware eviction policy": frequency-aware Greedy-Dual-Size-Frequency, H = L + F * cost / size with
// one size and one cost per block, so H = L + F; L = priority of the last victim, read once per kernel).
__device__ __forceinline__ void touch_block(const Store& st, u32 id, u64 epoch, u64 inflation, u32 count) {
  if (st.policy == 0) { st.m_last[id] = epoch; return; }
  const u32 f = atomicAdd(&st.m_freq[id], count) + count;
  atomicMax(&st.m_last[id], inflation + (u64)f);
}

// full blocks of request r, capped
__device__ __forceinline__ int full_blocks(const long long* __restrict__ offsets, int r, u32 B, int max_blocks) {
  long long len = offsets[r + 1] - offsets[r];
  long long nb = len < 0 ? 0 : len / (long long)B;
  return (int)(nb < (long long)max_blocks ? nb : (long long)max_blocks);
}

}  // namespace pts
