// Promotion of host-tier blocks into HBM (the paper keeps the hot prefixes on the fastest memory tier,
// Section 4.1 "Replication of popular prefixes to improve access locality"; with a single store the analogue
// is moving a block that was just hit from the pinned-host pool to the HBM pool).
//
// Entries e = (request r, block j < matched[r]) are ranked in (r, j) order, so the front of a prefix moves
// first.  A block moves once (its first entry decides), only if nobody outside this list holds its id
// (refcount equals the number of entries of the list naming it, or 0 for an unpinned list), while the budget
// and the HBM free ring last.  Phases: mark (first entry and entry count per block) -> count -> plan ->
// assign (new id, metadata, table value, rings, copy descriptor) -> rewrite (every entry naming a moved
// block gets the new id) -> copy host -> HBM with the vector engine.
#pragma once
#include "common.cuh"
#include "insert.cuh"

namespace pts {

constexpr u32 PROMO_MOVED = 0x80000000u;     // first_e[id] = PROMO_MOVED | new id once a block has moved

__device__ __forceinline__ bool promo_entry(const Store& st, const int* __restrict__ ids, const int* __restrict__ matched,
                                            long long e, int max_blocks, u32* id_out) {
  const int r = (int)(e / max_blocks), j = (int)(e % max_blocks);
  int mr = matched[r];
  if (mr > max_blocks) mr = max_blocks;
  if (j >= mr) return false;
  const int id = ids[e];
  if (id < (int)st.n[0] || (u32)id >= st.n[0] + st.n[1] || st.m_key[id] == 0) return false;   // only live host-tier blocks
  *id_out = (u32)id;
  return true;
}

__global__ void __launch_bounds__(256) promote_mark_kernel(Store st, const int* __restrict__ ids, const int* __restrict__ matched,
                                                           long long total, int max_blocks, u32* __restrict__ first_e,
                                                           u32* __restrict__ cnt) {
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    u32 id;
    if (!promo_entry(st, ids, matched, e, max_blocks, &id)) continue;
    atomicMin(&first_e[id], (u32)e);
    atomicAdd(&cnt[id], 1u);
  }
}

__device__ __forceinline__ u32 promo_flag(const Store& st, const int* __restrict__ ids, const int* __restrict__ matched, long long e,
                                          long long total, int max_blocks, const u32* __restrict__ first_e, const u32* __restrict__ cnt,
                                          u32 pinned_list, u32* id_out) {
  if (e >= total) return 0;
  u32 id;
  if (!promo_entry(st, ids, matched, e, max_blocks, &id)) return 0;
  *id_out = id;
  if (first_e[id] != (u32)e) return 0;
  return st.m_ref[id] == (pinned_list ? cnt[id] : 0u) ? 1u : 0u;
}

__global__ void __launch_bounds__(INS_THREADS) promote_count_kernel(Store st, const int* __restrict__ ids, const int* __restrict__ matched,
                                                                    long long total, int max_blocks, const u32* __restrict__ first_e,
                                                                    const u32* __restrict__ cnt, u32 pinned_list, u32* __restrict__ cta_sums) {
  __shared__ u32 warp_sums[32];
  const long long e = (long long)blockIdx.x * INS_THREADS + threadIdx.x;
  u32 id;
  const u32 f = promo_flag(st, ids, matched, e, total, max_blocks, first_e, cnt, pinned_list, &id);
  u32 sum;
  block_scan_incl(f, warp_sums, &sum);
  if (threadIdx.x == 0) cta_sums[blockIdx.x] = sum;
}

__global__ void __launch_bounds__(INS_THREADS) promote_plan_kernel(Store st, u32* __restrict__ cta_sums, u32 n_ctas, u32 max_promote,
                                                                   int* __restrict__ n_promoted) {
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
    u32 granted = carry < max_promote ? carry : max_promote;
    if (granted > c->ring[0].count) granted = c->ring[0].count;
    c->ins_granted = granted;
    c->ins_base = c->ring[0].head;                                        // HBM ids come from here
    c->ev_take = (u32)(((u64)c->ring[1].head + c->ring[1].count) % (st.n[1] ? st.n[1] : 1));   // host ids go back here
    c->ring[0].head = (u32)(((u64)c->ring[0].head + granted) % st.n[0]);
    c->ring[0].count -= granted;
    c->ring[1].count += granted;
    c->live[0] += granted;
    c->live[1] -= granted;
    c->n_pairs = granted;
    c->blocks_promoted += granted;
    if (n_promoted) *n_promoted = (int)granted;
  }
}

__global__ void __launch_bounds__(INS_THREADS) promote_assign_kernel(Store st, const int* __restrict__ ids, const int* __restrict__ matched,
                                                                     long long total, int max_blocks, u32* __restrict__ first_e,
                                                                     const u32* __restrict__ cnt, u32 pinned_list,
                                                                     const u32* __restrict__ cta_sums, int2* __restrict__ desc) {
  __shared__ u32 warp_sums[32];
  const long long e = (long long)blockIdx.x * INS_THREADS + threadIdx.x;
  u32 old_id = 0;
  const u32 f = promo_flag(st, ids, matched, e, total, max_blocks, first_e, cnt, pinned_list, &old_id);
  u32 sum;
  const u32 incl = block_scan_incl(f, warp_sums, &sum);
  if (!f) return;
  const u32 rank = cta_sums[blockIdx.x] + incl - 1;
  const Ctrl* c = st.ctrl;
  if (rank >= c->ins_granted) return;
  const u32 new_id = (u32)st.ring_ids[0][(u32)(((u64)c->ins_base + rank) % st.n[0])];
  st.ring_ids[1][(u32)(((u64)c->ev_take + rank) % st.n[1])] = (int)old_id;
  u32 visited, sid;
  const u32 s = find_slot(st, st.m_key[old_id], &visited, &sid);
  if (s != NO_SLOT) st.table[s].id = new_id;
  st.m_key[new_id] = st.m_key[old_id];
  st.m_parent[new_id] = st.m_parent[old_id];
  st.m_last[new_id] = st.m_last[old_id];
  st.m_freq[new_id] = st.m_freq[old_id];
  st.m_ref[new_id] = st.m_ref[old_id];
  st.m_depth[new_id] = st.m_depth[old_id];
  st.m_key[old_id] = 0;
  st.m_ref[old_id] = 0;
  desc[rank] = make_int2((int)old_id, (int)new_id);
  first_e[old_id] = PROMO_MOVED | new_id;
}

__global__ void __launch_bounds__(256) promote_rewrite_kernel(Store st, int* __restrict__ ids, const int* __restrict__ matched, long long total,
                                                              int max_blocks, const u32* __restrict__ first_e) {
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    const int r = (int)(e / max_blocks), j = (int)(e % max_blocks);
    int mr = matched[r];
    if (mr > max_blocks) mr = max_blocks;
    if (j >= mr) continue;
    const int id = ids[e];
    if (id < (int)st.n[0] || (u32)id >= st.n[0] + st.n[1]) continue;
    const u32 v = first_e[id];
    if (v != 0xFFFFFFFFu && (v & PROMO_MOVED)) ids[e] = (int)(v & ~PROMO_MOVED);
  }
}

}  // namespace pts
