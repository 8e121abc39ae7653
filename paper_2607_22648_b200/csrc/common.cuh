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
// 16 bytes, loaded with one 128-bit access.  key 0 = never used, key 1 = deleted.
// id = NO_ID while a slot has been claimed by an insert that has not assigned its block yet.
struct __align__(16) Slot {
  u64 key;
  u32 id;
  u32 aux;      // insert only: lowest request index that presented this new key
};
constexpr u64 KEY_EMPTY = 0ull;
constexpr u64 KEY_TOMB = 1ull;
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
  u32 tombstones;
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
  u64 rebuilds;
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
  s.aux = v.w;
  return s;
}

// Linear probe for `key`.  Returns the slot index or NO_SLOT; *visited gets the slots examined.
// The walk is latency bound (each slot is a dependent L2 access) and a warp waits for its slowest lane, so
// PROBE_WINDOW consecutive slots are loaded at once and then examined in order: a miss at load factor 0.7
// needs ~6 slots on average with a long tail, which becomes two round trips instead of six or more.
constexpr int PROBE_WINDOW = 4;
__device__ __forceinline__ u32 find_slot(const Slot* __restrict__ table, u64 slots, u64 key, u32* visited, u32* id_out) {
  u64 s = home_slot(key, slots);
  u32 n = 0;
  for (u64 i = 0; i < slots; i += PROBE_WINDOW) {
    uint4 v[PROBE_WINDOW];
    u64 idx[PROBE_WINDOW];
#pragma unroll
    for (int w = 0; w < PROBE_WINDOW; ++w) {
      u64 t = s + w;
      idx[w] = t >= slots ? t - slots : t;
      v[w] = *reinterpret_cast<const uint4*>(table + idx[w]);
    }
#pragma unroll
    for (int w = 0; w < PROBE_WINDOW; ++w) {
      const u64 k = ((u64)v[w].y << 32) | v[w].x;
      ++n;
      if (k == key) { *visited = n; *id_out = v[w].z; return (u32)idx[w]; }
      if (k == KEY_EMPTY) { *visited = n; *id_out = NO_ID; return NO_SLOT; }
    }
    s += PROBE_WINDOW;
    if (s >= slots) s -= slots;
  }
  *visited = n;
  *id_out = NO_ID;
  return NO_SLOT;
}

// The same probe in two halves, so that a caller can put independent work between the loads of the first window and
// their use: probe_issue starts the loads, probe_finish examines them and walks on if the run is longer.
struct ProbeWindow { uint4 v[PROBE_WINDOW]; };
__device__ __forceinline__ void probe_issue(const Slot* __restrict__ table, u64 slots, u64 key, ProbeWindow& w) {
  const u64 s = home_slot(key, slots);
#pragma unroll
  for (int k = 0; k < PROBE_WINDOW; ++k) {
    u64 t = s + k;
    t = t >= slots ? t - slots : t;
    w.v[k] = *reinterpret_cast<const uint4*>(table + t);
  }
}
__device__ __forceinline__ u32 probe_finish(const Slot* __restrict__ table, u64 slots, u64 key, const ProbeWindow& w, u32* visited) {
  u32 n = 0;
#pragma unroll
  for (int k = 0; k < PROBE_WINDOW; ++k) {
    const u64 kk = ((u64)w.v[k].y << 32) | w.v[k].x;
    ++n;
    if (kk == key) { *visited = n; return w.v[k].z; }
    if (kk == KEY_EMPTY) { *visited = n; return NO_ID; }
  }
  u64 s = home_slot(key, slots) + PROBE_WINDOW;
  if (s >= slots) s -= slots;
  for (u64 i = PROBE_WINDOW; i < slots; i += PROBE_WINDOW) {
    uint4 v[PROBE_WINDOW];
#pragma unroll
    for (int k = 0; k < PROBE_WINDOW; ++k) {
      u64 t = s + k;
      t = t >= slots ? t - slots : t;
      v[k] = *reinterpret_cast<const uint4*>(table + t);
    }
#pragma unroll
    for (int k = 0; k < PROBE_WINDOW; ++k) {
      const u64 kk = ((u64)v[k].y << 32) | v[k].x;
      ++n;
      if (kk == key) { *visited = n; return v[k].z; }
      if (kk == KEY_EMPTY) { *visited = n; return NO_ID; }
    }
    s += PROBE_WINDOW;
    if (s >= slots) s -= slots;
  }
  *visited = n;
  return NO_ID;
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
