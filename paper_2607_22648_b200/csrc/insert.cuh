// Scatter-insert of new blocks (store operation: only the increment after the longest common prefix
// is saved and appended to the trie, paper Section 4 summary paragraph and Section 4.1).
//
// The batch must behave as if requests were inserted one after the other in index order.  Phases
// (one kernel each, all over the R*max_blocks elements e = (request r, block j)):
//   claim   : find the key of e in the table or claim an empty slot for it (atomicCAS on the key);
//             every element that lands on a slot claimed in this call lowers slot.aux to its request
//             index (atomicMin), so the lowest request presenting a new prefix becomes its creator.
//   count   : flag(e) = "e creates a node"; per-CTA sums.
//   plan    : scan of the CTA sums; grants = min(new nodes, free HBM blocks); ring head moves.
//   assign  : rank(e) among creators in (r, j) order; rank < grants gets ring[head + rank], writes the
//             slot value and the node's metadata and a copy descriptor; the others delete their claim.
//   finish  : every element reads its slot's block id (or -1) and refreshes the LRU stamp.
// Ranking creators in (r, j) order and granting the first `free` of them equals the sequential rule:
// a denied node's descendants always rank higher, so denials are prefix-closed per request.
#pragma once
#include "common.cuh"

namespace pts {

constexpr int INS_THREADS = 1024;

__global__ void __launch_bounds__(256) insert_claim_kernel(Store st, const u64* __restrict__ keys, int R, int max_blocks,
                                                           u32* __restrict__ eslot, int* __restrict__ new_blocks) {
  const long long total = (long long)R * max_blocks;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    const u32 r = (u32)(e / max_blocks);
    if (e % max_blocks == 0) new_blocks[r] = 0;
    const u64 key = keys[e];
    if (key == 0) { eslot[e] = NO_SLOT; continue; }
    u64 s = home_slot(key, st.slots);
    u32 got = NO_SLOT;
    for (u64 i = 0; i < st.slots; ++i) {
      u64 k = *reinterpret_cast<volatile u64*>(&st.table[s].key);
      if (k == KEY_EMPTY) {
        k = atomicCAS(&st.table[s].key, KEY_EMPTY, key);
        if (k == KEY_EMPTY) k = key;                     // claimed
      }
      if (k == key) { got = (u32)s; break; }
      s = (s + 1 == st.slots) ? 0 : s + 1;
    }
    eslot[e] = got;
    if (got == NO_SLOT) { raise(st, S_TABLE_FULL); continue; }
    if (*reinterpret_cast<volatile u32*>(&st.table[got].id) == NO_ID) atomicMin(&st.table[got].aux, r);
  }
}

__device__ __forceinline__ u32 creator_flag(const Store& st, const u32* __restrict__ eslot, long long e, int max_blocks) {
  const u32 s = eslot[e];
  if (s == NO_SLOT) return 0;
  const Slot v = load_slot(st.table + s);
  return (v.id == NO_ID && v.aux == (u32)(e / max_blocks)) ? 1u : 0u;
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
  return incl;
}

__global__ void __launch_bounds__(INS_THREADS) insert_count_kernel(Store st, const u32* __restrict__ eslot, long long total,
                                                                   int max_blocks, u32* __restrict__ cta_sums) {
  __shared__ u32 warp_sums[32];
  const long long e = (long long)blockIdx.x * INS_THREADS + threadIdx.x;
  const u32 f = e < total ? creator_flag(st, eslot, e, max_blocks) : 0;
  u32 sum;
  block_scan_incl(f, warp_sums, &sum);
  if (threadIdx.x == 0) cta_sums[blockIdx.x] = sum;
}

// single CTA: exclusive scan of cta_sums in place, then the allocation plan
__global__ void __launch_bounds__(INS_THREADS) insert_plan_kernel(Store st, u32* __restrict__ cta_sums, u32 n_ctas, u32 rebuild_threshold) {
  __shared__ u32 warp_sums[32];
  __shared__ u32 carry;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (u32 base = 0; base < n_ctas; base += INS_THREADS) {
    const u32 i = base + threadIdx.x;
    const u32 x = i < n_ctas ? cta_sums[i] : 0;
    u32 tile_total;
    const u32 incl = block_scan_incl(x, warp_sums, &tile_total);
    if (i < n_ctas) cta_sums[i] = carry + incl - x;
    __syncthreads();
    if (threadIdx.x == 0) carry += tile_total;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    Ctrl* c = st.ctrl;
    if (c->tombstones > rebuild_threshold) { c->tombstones = 0; c->rebuilds += 1; }   // this call began with a rebuild
    const u32 total_new = carry;
    const u32 granted = total_new < c->ring[0].count ? total_new : c->ring[0].count;
    c->ins_total_new = total_new;
    c->ins_granted = granted;
    c->ins_base = c->ring[0].head;
    c->ring[0].head = (u32)(((u64)c->ring[0].head + granted) % st.n[0]);
    c->ring[0].count -= granted;
    c->live[0] += granted;
    c->n_pairs = granted;
    c->blocks_inserted += granted;
    c->blocks_denied += total_new - granted;
    c->tombstones += total_new - granted;
    if (granted < total_new) atomicOr(&c->status, S_NOSPACE);
  }
}

__global__ void __launch_bounds__(INS_THREADS) insert_assign_kernel(Store st, const u64* __restrict__ keys,
                                                                    const u32* __restrict__ eslot, long long total, int max_blocks,
                                                                    const u32* __restrict__ cta_sums, const int* __restrict__ bt,
                                                                    u32 cache_blocks, u64 epoch, int2* __restrict__ desc,
                                                                    int* __restrict__ new_blocks) {
  __shared__ u32 warp_sums[32];
  const long long e = (long long)blockIdx.x * INS_THREADS + threadIdx.x;
  const u32 f = e < total ? creator_flag(st, eslot, e, max_blocks) : 0;
  u32 sum;
  const u32 incl = block_scan_incl(f, warp_sums, &sum);
  if (!f) return;
  const u32 rank = cta_sums[blockIdx.x] + incl - 1;
  const u32 granted = st.ctrl->ins_granted;
  Slot* slot = st.table + eslot[e];
  if (rank >= granted) {                       // denied: withdraw the claim
    slot->aux = NO_ID;
    slot->key = KEY_TOMB;
    return;
  }
  const u32 id = (u32)st.ring_ids[0][(u32)(((u64)st.ctrl->ins_base + rank) % st.n[0])];
  const int j = (int)(e % max_blocks);
  st.m_key[id] = keys[e];
  st.m_parent[id] = j ? keys[e - 1] : st.root_key;
  st.m_last[id] = st.policy ? 0 : epoch;      // GDSF: the finish kernel counts this call's accesses
  st.m_freq[id] = 0;
  st.m_ref[id] = 0;
  st.m_depth[id] = (u32)j;
  slot->aux = NO_ID;
  slot->id = id;
  int2 d = make_int2((int)id, 0);
  if (bt) {
    const int cb = bt[e];
    if (cb < 0 || (u32)cb >= cache_blocks) { raise(st, S_BOUNDS); d.x = -1; }
    d.y = cb;
  } else {
    d.x = -1;                                  // metadata-only insert: nothing to copy
  }
  desc[rank] = d;
  atomicAdd(&new_blocks[e / max_blocks], 1);
}

__global__ void __launch_bounds__(256) insert_finish_kernel(Store st, const u32* __restrict__ eslot, long long total, u64 epoch,
                                                            int* __restrict__ ids_out) {
  const u64 inflation = st.policy ? st.ctrl->inflation : 0;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    const u32 s = eslot[e];
    int out = -1;
    if (s != NO_SLOT) {
      const u32 id = st.table[s].id;
      if (id != NO_ID) { out = (int)id; touch_block(st, id, epoch, inflation, 1); }
    }
    ids_out[e] = out;
  }
}

}  // namespace pts
