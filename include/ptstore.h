/*
 * ptstore.h — C ABI of the single-GPU prefix tensor store (sm_100a).
 *
 * The library keeps the K/V tensors of token prefixes as a trie of fixed-size token blocks
 * ("incremental, tensor-level prefix storage": an object stores only what follows its longest
 * common prefix with earlier objects — paper Section 4, first paragraph, and Section 4.1
 * "Co-optimized compact metadata and fast prefix queries").  The trie is encoded as an
 * open-addressing hash table of chained 64-bit block keys that lives in device memory.
 *
 * General conventions
 *   - Every array argument is a DEVICE-ACCESSIBLE pointer (device memory, or pinned host memory that
 *     is mapped into the device address space) unless the argument is marked "host".
 *   - The library allocates no device memory (it does allocate a few hundred bytes of host memory
 *     for the handle).  Pools and workspace are owned by the caller and must outlive the handle.
 *   - Every call that takes a stream only ENQUEUES work on that stream and returns; results are
 *     valid once the stream has reached that point.  Calls on one handle must be issued from one
 *     host thread at a time and onto one stream (or streams the caller has ordered); the library
 *     takes no lock.
 *   - ptstore_create makes cfg->device the calling thread's current CUDA device and leaves it so; every later call on
 *     the handle must be made with that device current (the library does not switch devices per call).
 *   - The LRU clock, the sequence numbers that tag a fetch's lists and the choice of barrier counter are host-side
 *     counters of the handle, passed to the kernels by value when a call is enqueued.  A call captured into a CUDA graph
 *     would replay stale values, so enqueue calls directly; do not replay them from a captured graph.
 *   - Return value: PTSTORE_OK (0) or a negative PTSTORE_E_* code for conditions the host can see
 *     (bad arguments, CUDA launch errors).  Conditions only the device can see (pool exhausted,
 *     table full, block-table entry out of range, refcount underflow) are OR-ed as PTSTORE_S_* bits
 *     into a device status word; the kernel skips the offending access and carries on.  Nothing
 *     traps, nothing prints.
 *   - Layout ("RDMA-aware consolidation", Section 4.1: an increment is one contiguous region and each
 *     tensor an (offset,size) segment of it):
 *       chunk  = one block of one layer's K (or V): [block_tokens][num_kv_heads][head_dim] elements,
 *                contiguous; chunk_bytes must be a multiple of 16.
 *       block  = [num_layers][2 (K,V)][chunk], contiguous: block_bytes = 2*num_layers*chunk_bytes.
 *       pool   = [n_blocks][block]; block ids 0..hbm_blocks-1 are the HBM tier, ids
 *                hbm_blocks..hbm_blocks+host_blocks-1 are the host tier (id - hbm_blocks indexes
 *                host_pool).
 *       paged cache (vLLM style), per layer: K block b at layer_base[l] + b*block_stride_bytes,
 *                V block b at layer_base[l] + kv_stride_bytes + b*block_stride_bytes.
 */
#ifndef PTSTORE_H
#define PTSTORE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ptstore ptstore_t;      /* opaque */
typedef void* ptstore_stream_t;        /* a cudaStream_t; NULL = the legacy default stream */

/* host-visible return codes */
#define PTSTORE_OK          0
#define PTSTORE_E_INVAL    (-1)   /* null / misaligned pointer, size out of range, bad struct_size */
#define PTSTORE_E_CUDA     (-2)   /* a CUDA runtime call or launch failed (see ptstore_last_cuda_error) */
#define PTSTORE_E_NOMEM    (-3)   /* host allocation of the handle failed, or workspace too small */
#define PTSTORE_E_LIMIT    (-4)   /* batch exceeds max_requests / max_batch_blocks given at create */

/* bits of the device status word (ptstore_status) */
#define PTSTORE_S_NOSPACE     0x1u   /* insert: HBM free ring ran dry, some blocks were denied */
#define PTSTORE_S_TABLE_FULL  0x2u   /* insert: no free slot found within table_slots probes */
#define PTSTORE_S_BOUNDS      0x4u   /* a block id or block-table entry was out of range; access skipped */
#define PTSTORE_S_STATE       0x8u   /* release would have driven a refcount below zero; skipped */
#define PTSTORE_S_TIMEOUT     0x10u  /* a bounded wait inside a kernel expired (a copy CTA stopped copying, or a grid-wide
                                        barrier gave up); the call's results are incomplete, the handle stays usable for
                                        copies, and nothing is left running */
#define PTSTORE_S_INFLIGHT    0x20u  /* fetch: a host-tier block named by the call was demoted by ptstore_evict_async /
                                        ptstore_reserve(PTSTORE_ASYNC_COPY) and its copy has not been joined yet; that
                                        entry was skipped */

/* flags of ptstore_lookup */
#define PTSTORE_PIN       0x1u   /* refcount++ on every matched (request, block) pair */
#define PTSTORE_NO_TOUCH  0x2u   /* do not refresh the LRU stamp of matched blocks */

/* flags of ptstore_promote */
#define PTSTORE_PINNED_LIST 0x1u  /* the id list passed in was produced by a lookup with PTSTORE_PIN */

/* flags of ptstore_config_t */
#define PTSTORE_COPY_BULK    0x0u  /* default copy engine for HBM<->HBM: bulk-async copies through a shared-memory ring */
#define PTSTORE_COPY_VECTOR  0x1u  /* use 16-byte vector loads/stores everywhere (the host tier always uses them) */
/* eviction order (Section 4.1 "Access pattern-aware eviction policy"): default is least recently used; with this
 * flag it is Greedy-Dual-Size-Frequency with one size and one cost per block: priority H = L + F, F = accesses of
 * the block (one per request that matched or stored it), L = the largest priority evicted so far.  Ties and the
 * leaves-first rule are as for LRU. */
#define PTSTORE_EVICT_GDSF   0x2u
/* tuning fields of flags (0 = library default):
 *   PTSTORE_LOOKUP_LANES(n)      lanes per request of lookup / hash: 4, 8, 16 or 32
 *   PTSTORE_COPY_CTAS_PER_SM(c)  CTAs per SM of the HBM<->HBM copy kernels
 *   PTSTORE_COPY_VARIANT(v)      geometry of the copy kernels.  With PTSTORE_COPY_BULK, the ring of shared-memory stages:
 *                                  0 sized from the chunk size (3 stages of min(chunk, 32 KiB), 1-4 CTAs per SM)
 *                                  1 8 x 8 KiB, 3 CTAs per SM      2 3 x 32 KiB          3 4 x 16 KiB, 3 CTAs per SM
 *                                  4 12 x 16 KiB                   5 6 x 16 KiB, two consecutive pieces per turn
 *                                  6 6 x 16 KiB with evict-first L2 hints on loads and stores     7 3 x 64 KiB
 *                                With PTSTORE_COPY_VECTOR, threads x 16-byte loads in flight per thread:
 *                                  0 256 x 4, 16 CTAs per SM       1 256 x 8, 8 CTAs per SM       2 512 x 4, 4 CTAs per SM
 *                                Other values select 0. */
#define PTSTORE_LOOKUP_LANES(n)   (((uint32_t)(n) & 0xFFu) << 8)
#define PTSTORE_COPY_VARIANT(v)   (((uint32_t)(v) & 0xFu) << 16)
#define PTSTORE_COPY_CTAS_PER_SM(c) (((uint32_t)(c) & 0xFFu) << 20)

/* flags of ptstore_reserve */
#define PTSTORE_ASYNC_COPY  0x1u  /* run the demotion copy on the library's side stream, as ptstore_evict_async does */

/* tiers of ptstore_evict */
#define PTSTORE_TIER_HBM   0
#define PTSTORE_TIER_HOST  1

typedef struct {
  uint32_t struct_size;          /* sizeof(ptstore_config_t), checked */
  uint32_t flags;                /* PTSTORE_COPY_* | PTSTORE_EVICT_GDSF | tuning fields; 0 = defaults */
  uint32_t num_layers, num_kv_heads, head_dim, elem_bytes;   /* bf16: elem_bytes = 2 */
  uint32_t block_tokens;         /* tokens per block, >= 1 */
  uint32_t max_requests;         /* largest R any call will pass */
  uint64_t max_batch_blocks;     /* largest R*max_blocks any call will pass */
  uint64_t salt;                 /* folded into the root key (model / namespace id) */
  void*    hbm_pool;             /* device memory, hbm_blocks*block_bytes, 16-byte aligned */
  void*    host_pool;            /* device-visible pointer of mapped pinned memory, or NULL */
  uint32_t hbm_blocks;           /* >= 1 */
  uint32_t host_blocks;          /* 0 = no host tier */
  uint64_t table_slots;          /* hash-table slots: any integer > hbm_blocks+host_blocks (values below 8 are raised to
                                    8); for short probe runs use about (hbm_blocks + host_blocks + largest insert
                                    batch) / 0.7 */
  void*    workspace;            /* device memory, 256-byte aligned */
  uint64_t workspace_bytes;      /* >= ptstore_workspace_bytes(cfg) */
  int32_t  device;               /* CUDA device ordinal that owns pools and workspace */
  int32_t  reserved;
} ptstore_config_t;

typedef struct {
  void* const* layer_base;       /* DEVICE array [num_layers] of device pointers, each 16-byte aligned */
  uint64_t kv_stride_bytes;      /* V plane offset inside a layer tensor; multiple of 16 */
  uint64_t block_stride_bytes;   /* distance between consecutive blocks; >= chunk_bytes, multiple of 16 */
  uint32_t num_blocks;           /* block-table entries must be in [0, num_blocks) */
  uint32_t reserved;
} ptstore_paged_cache_t;

typedef struct {                 /* all counters are cumulative since create */
  uint64_t epoch;                /* lookup + insert calls so far (the LRU clock) */
  uint64_t live_nodes[2];        /* trie nodes per tier right now */
  uint64_t free_blocks[2];       /* free-ring fill per tier right now */
  uint64_t max_displacement;     /* largest distance from its home slot at which the table has ever placed a key
                                    (counted from 24 slots up, else 0) */
  uint64_t query_blocks;         /* full blocks presented to lookup */
  uint64_t probes_issued;        /* keys actually searched by lookup */
  uint64_t slots_visited;        /* table slots read by those searches */
  uint64_t blocks_matched;       /* sum of matched lengths */
  uint64_t blocks_fetched[2];    /* per source tier */
  uint64_t blocks_inserted;
  uint64_t blocks_denied;
  uint64_t blocks_dropped[2];    /* deleted per tier */
  uint64_t blocks_demoted;       /* HBM -> host */
  uint64_t far_keys;             /* keys placed 24 or more slots from their home slot so far (a lookup of such a key
                                    takes a second round of loads) */
  uint64_t blocks_promoted;      /* host -> HBM */
  uint64_t gdsf_clock;           /* GDSF policy: largest priority evicted so far */
  uint64_t blocks_fetched_distinct; /* distinct source blocks read by fetch calls: a block named by several requests
                                       of one call is read once and written to each destination */
} ptstore_stats_t;

/*
 * Bytes of workspace ptstore_create needs for this configuration (table, per-block metadata,
 * free rings, per-batch scratch).  Only the size fields of cfg are read.  Returns 0 if cfg is invalid.
 * No paper counterpart: the paper couples its store to a pre-registered allocator (Section 5,
 * second paragraph); here the caller pre-allocates instead.
 */
uint64_t ptstore_workspace_bytes(const ptstore_config_t* cfg /*host*/);

/*
 * Create an empty store (Section 4: an empty trie; free rings hold every block id in ascending
 * order; LRU clock 0).  Enqueues the initialisation on `stream`.  *out receives a handle that
 * ptstore_destroy frees.  Errors: E_INVAL (geometry, alignment, sizes), E_NOMEM, E_CUDA.
 */
int ptstore_create(const ptstore_config_t* cfg /*host*/, ptstore_t** out /*host*/, ptstore_stream_t stream);

/* Free the handle.  Caller memory is not touched.  The caller syncs outstanding work first. */
int ptstore_destroy(ptstore_t* st);

/*
 * Chained block keys (the "unique tensor IDs" an object inherits from its longest common prefix and
 * then extends, Section 4.1): keys[r*max_blocks + i] for every full block i < min(full_blocks(r),
 * max_blocks) of request r; other entries are written as 0.  A trailing partial block is ignored.
 *   tokens  int32 [offsets[R]]   ragged token ids; request r is tokens[offsets[r] .. offsets[r+1])
 *   offsets int64 [R+1]          non-decreasing, offsets[0] >= 0
 * Auxiliary entry point for verification; lookup and insert hash internally.
 */
int ptstore_hash(ptstore_t* st, const int32_t* tokens, const int64_t* offsets, int32_t R, int32_t max_blocks,
                 uint64_t* keys_out /*[R*max_blocks]*/, ptstore_stream_t stream);

/*
 * Batched longest-common-prefix query (Section 1 "one-shot LCP query"; Section 4.1: a store or load
 * first finds the longest common prefix among all previously stored objects).
 *   matched_blocks[r] = number of leading full blocks of request r present in the store, capped at
 *                       max_blocks; matched tokens = matched_blocks[r] * block_tokens.
 *   block_ids[r*max_blocks + j] = pool block id holding block j for j < matched_blocks[r], else -1.
 * Advances the LRU clock by one; unless NO_TOUCH stamps every matched block; with PIN adds one
 * reference per matched (request, block) pair (reused blocks are marked by a reference counter,
 * Section 1).  Ids of pinned blocks stay valid until released; other ids only until the next
 * insert or evict.
 */
int ptstore_lookup(ptstore_t* st, const int32_t* tokens, const int64_t* offsets, int32_t R, int32_t max_blocks,
                   uint32_t flags, int32_t* matched_blocks /*[R]*/, int32_t* block_ids /*[R*max_blocks]*/,
                   ptstore_stream_t stream);

/*
 * ptstore_lookup followed by ptstore_fetch of what it matched, as one call (Section 4.1: a load first finds the longest
 * common prefix and then brings each of its tensors to the GPU pointers the application supplies; what matters to the
 * application is the latency of the pair).  Same results as the two calls: matched_blocks and block_ids are written
 * as by ptstore_lookup(flags), and every matched block j of request r is copied to cache block
 * block_tables[r*max_blocks+j] as by ptstore_fetch.  The lookup kernel builds the copy lists itself while it probes,
 * so the pair costs two kernel launches (three with a host tier).  A batch of at most 16 requests of more than 32 blocks
 * against a store without a host tier (default copy engine, no ptstore_time_next_copy pending) is one cooperative launch:
 * the copies of a request's first blocks run while the rest of its hash chain is still being looked up.  Either way a
 * pool block named by several entries of the call is read once and written to every destination.
 */
int ptstore_lookup_fetch(ptstore_t* st, const int32_t* tokens, const int64_t* offsets, int32_t R, int32_t max_blocks,
                         uint32_t flags, const ptstore_paged_cache_t* dst /*host struct*/,
                         const int32_t* block_tables /*[R*max_blocks]*/, int32_t* matched_blocks /*[R]*/,
                         int32_t* block_ids /*[R*max_blocks]*/, ptstore_stream_t stream);

/*
 * Load (Section 4.1: iterate over the ids of an object and bring each tensor to the GPU pointers
 * the application supplies).  For every r, j < matched_blocks[r], layer l, s in {K,V}: copy one chunk
 * from pool block block_ids[r*max_blocks+j] to block block_tables[r*max_blocks+j] of the paged cache.
 * Host-tier blocks are read in place through the mapped pointer.  No metadata changes.
 * A pool block named by several entries of the call is read once and written to every destination.
 * Entries with an id or table entry out of range are skipped and raise S_BOUNDS.
 */
int ptstore_fetch(ptstore_t* st, const int32_t* block_ids, const int32_t* matched_blocks, int32_t R,
                  int32_t max_blocks, const ptstore_paged_cache_t* dst /*host struct*/,
                  const int32_t* block_tables /*[R*max_blocks]*/, ptstore_stream_t stream);

/*
 * Store (Section 4: a store saves only the increment after the longest common prefix; Section 4.1:
 * the application supplies the GPU pointers of the new tensors).  Requests are taken as if one after
 * the other in index order: a block whose prefix is already stored is reused (and stamped), otherwise
 * a block id is popped from the front of the HBM free ring, the 2*num_layers chunks are copied from
 * src block block_tables[r*max_blocks+j] into it and a trie node is created.  When the ring runs dry
 * the remaining new blocks are denied (-1) and S_NOSPACE is raised; nothing is evicted implicitly.
 *   block_ids  out [R*max_blocks]: id now holding block j (existing or new), -1 if denied / beyond length
 *   new_blocks out [R]: nodes created on behalf of request r (the lowest request index that presents
 *                       a new prefix creates it)
 * Advances the LRU clock by one.
 */
int ptstore_insert(ptstore_t* st, const int32_t* tokens, const int64_t* offsets, int32_t R, int32_t max_blocks,
                   const ptstore_paged_cache_t* src /*host struct*/, const int32_t* block_tables,
                   int32_t* block_ids, int32_t* new_blocks, ptstore_stream_t stream);

/*
 * ptstore_insert for the batch the handle's most recent ptstore_lookup / ptstore_lookup_fetch call was given (Section 4:
 * a store begins by finding the longest common prefix, which the preceding load has just done for the same prompt).
 * Same results as ptstore_insert in every case.  If tokens, offsets, R and max_blocks are those of that lookup - the same
 * pointers and sizes, and the caller has not changed the arrays' contents since - and requests are few and long (a warp per
 * request: fewer than 1024 requests of more than 16 blocks), the chained block keys that lookup computed are reused and
 * hashing resumes behind them; the hash chain of a long prompt is a serial computation, so this takes tens of microseconds
 * off a small batch.  Otherwise the call is ptstore_insert.
 */
int ptstore_insert_after_lookup(ptstore_t* st, const int32_t* tokens, const int64_t* offsets, int32_t R, int32_t max_blocks,
                                const ptstore_paged_cache_t* src /*host struct*/, const int32_t* block_tables,
                                int32_t* block_ids, int32_t* new_blocks, ptstore_stream_t stream);

/* Calls of ptstore_insert_after_lookup so far that did reuse a lookup's keys (host counter, no sync). */
uint64_t ptstore_resumed_inserts(const ptstore_t* st);

/*
 * Drop one reference per (r, j < matched_blocks[r]) pair (the counterpart of PIN; Section 1: blocks
 * of finished requests become evictable).  A count that is already zero stays zero and raises S_STATE.
 */
int ptstore_release(ptstore_t* st, const int32_t* block_ids, const int32_t* matched_blocks, int32_t R,
                    int32_t max_blocks, ptstore_stream_t stream);

/*
 * Evict up to n_blocks least-recently-used unreferenced leaves of a tier (Section 1: LRU over blocks
 * of finished requests; Section 4.1 "Access pattern-aware eviction policy": owned tensors are flushed
 * to slower tiers).  Order: (LRU stamp ascending, deeper first, lower id first); a parent freed by the
 * removal of its last child in the same call may follow it.
 *   tier HOST, or tier HBM without a host pool: the node is deleted and its id appended to the back of
 *     that tier's free ring.
 *   tier HBM with a host pool: if the host ring holds fewer than n_blocks free ids, the shortfall is
 *     first dropped from the host tier; then up to min(n_blocks, host free) HBM blocks are copied to
 *     host blocks popped from the front of the host ring; the node keeps its place in the trie under
 *     its new id and the HBM id goes to the back of the HBM ring.
 *   n_evicted  out, device [2]: [0] = blocks taken out of `tier` (dropped or demoted), [1] = host-tier
 *              blocks dropped beforehand to make room for a demotion (0 in the other cases)
 *   victim_ids out, device [2*n_blocks] or NULL: former ids of the n_evicted[0] blocks in the order
 *              taken, followed by the n_evicted[1] room-making drops in the order taken
 */
int ptstore_evict(ptstore_t* st, int32_t tier, int32_t n_blocks, int32_t* n_evicted, int32_t* victim_ids,
                  ptstore_stream_t stream);

/*
 * ptstore_evict with the demotion copy (HBM -> host) on a stream of the library's own, so that it can share the
 * host link, which is full duplex, with a fetch of host-tier blocks running the other way (the paper overlaps its
 * transfers with computation, Section 4.1 "Fine-grain multi-level caching": data transfers happen asynchronously).
 * Everything else is as for ptstore_evict: the metadata changes and both outputs are ordered on `stream`.
 * The copy is ordered after them and before any later ptstore_insert, ptstore_promote, ptstore_evict[_async] and
 * ptstore_join on this handle.  It is NOT ordered with later ptstore_fetch calls: until the next of the calls just
 * named, fetch only block ids that were pinned (ptstore_lookup with PTSTORE_PIN) before this call — a pinned block
 * is never a victim, so such a fetch cannot touch a block in flight.  Without a host tier, or for tier HOST, this
 * is ptstore_evict.  The first call creates the stream and two events (no device memory).  A fetch that names a
 * host-tier block whose copy is still in flight skips that entry and raises PTSTORE_S_INFLIGHT.
 */
int ptstore_evict_async(ptstore_t* st, int32_t tier, int32_t n_blocks, int32_t* n_evicted, int32_t* victim_ids,
                        ptstore_stream_t stream);

/*
 * Make room before a store, decided on the device (Section 1: blocks of finished requests are evicted when space is
 * needed; this is ptstore_evict(PTSTORE_TIER_HBM, n) with n computed where the free count lives, so the host need not
 * wait for a lookup's result before it can queue the eviction):
 *     need = want_free - sum(max(minus[i], 0), i < n_minus) - free HBM blocks
 *     n    = need > 0 ? need + headroom : 0,   capped at max_victims.
 * Typical use: want_free = full blocks of the batch, minus = the matched_blocks array the preceding lookup wrote.
 * With headroom > 0 a call that has to evict takes that many blocks more, so that the calls after it find room and
 * return at once (an eviction costs tens of microseconds whatever its size, which matters for small batches).
 *   flags       0, or PTSTORE_ASYNC_COPY (the demotion copy runs as in ptstore_evict_async; same ordering rules)
 *   n_evicted   out, device [2], as for ptstore_evict
 *   victim_ids  out, device [2*max_victims] or NULL (then max_victims is ignored), as for ptstore_evict
 * n_minus may not exceed max_requests (PTSTORE_E_LIMIT).
 */
int ptstore_reserve(ptstore_t* st, int64_t want_free, int32_t headroom, const int32_t* minus, int32_t n_minus, uint32_t flags,
                    int32_t* n_evicted, int32_t* victim_ids, int32_t max_victims, ptstore_stream_t stream);

/* Make `stream` wait for a demotion copy left running by ptstore_evict_async (no-op if there is none). */
int ptstore_join(ptstore_t* st, ptstore_stream_t stream);

/*
 * Move host-tier blocks named by a batch into HBM (the paper keeps hot prefixes on the fastest tier, Section 4.1
 * "Replication of popular prefixes to improve access locality"; with one store the analogue is promoting a block
 * that was just hit).  Entries (r, j < matched_blocks[r]) are taken in (r, j) order, so the front of a prefix
 * moves first.  A block moves at most once per call, and only while (a) fewer than max_promote blocks have moved,
 * (b) the HBM free ring is not empty, and (c) nobody else holds its id: its reference count equals the number of
 * entries of this list that name it (flags = PTSTORE_PINNED_LIST) or zero (flags = 0).  The block gets the id at
 * the front of the HBM ring, its bytes are copied host -> HBM, its node keeps its place and stamps, and the host
 * id goes to the back of the host ring.
 *   block_ids   in/out [R*max_blocks]: entries naming a moved block are rewritten to its new id (use the
 *               rewritten list for the following fetch and release)
 *   n_promoted  out, device [1] or NULL: blocks moved
 * No host tier: returns PTSTORE_E_INVAL.  Call it between lookup and fetch.
 */
int ptstore_promote(ptstore_t* st, int32_t* block_ids, const int32_t* matched_blocks, int32_t R, int32_t max_blocks,
                    uint32_t flags, int32_t max_promote, int32_t* n_promoted, ptstore_stream_t stream);

/*
 * Synchronise `stream`, read the device status word into *status_out (host) and clear it.  The read and the clear
 * are two operations enqueued on `stream`: a bit raised by work running on ANOTHER stream between them is lost, so
 * keep everything on one stream (or ordered) around this call.
 */
int ptstore_status(ptstore_t* st, ptstore_stream_t stream, uint32_t* status_out /*host*/);

/* Synchronise `stream` and copy the counters to *out (host). */
int ptstore_stats(ptstore_t* st, ptstore_stream_t stream, ptstore_stats_t* out /*host*/);

/*
 * The same counters without blocking: a one-thread kernel on `stream` writes them to *out, which must be
 * device-accessible (device memory, or pinned host memory the device can write).  The caller waits for the stream,
 * or for an event recorded after this call, before reading.  Lets a scheduler learn the free-block count behind a
 * lookup while the fetch that follows is already running.
 */
int ptstore_stats_enqueue(ptstore_t* st, ptstore_stats_t* out /*device-accessible*/, ptstore_stream_t stream);

/*
 * Polls a copy kernel spends on one wait for a load, in its main loop, before its CTA gives up, raises
 * PTSTORE_S_TIMEOUT, waits (with the full built-in limit) for the loads it still has in flight and returns; 0 restores
 * the built-in limit.  No paper counterpart.  Meant for failure-detection tests: a limit of 1 is a single test that
 * never suspends, so a CTA whose first load has not landed yet gives up at once, without anything hanging or
 * faulting, and the give-up-and-drain path can be exercised on a healthy GPU.
 */
int ptstore_set_wait_limit(ptstore_t* st, uint32_t polls);

/*
 * Measurement aid (no paper counterpart): the next copy kernel the handle launches for HBM-resident data (the gather of
 * ptstore_fetch / ptstore_lookup_fetch, the scatter of ptstore_insert; not the small-grid host-link copies) gets
 * `before` recorded on its stream just ahead of it and `after` just behind it.  Both are cudaEvent_t created by the
 * caller with timing enabled; one shot.  cudaEventElapsedTime(before, after) is then the duration of that kernel alone,
 * which is what a bandwidth figure for the copy engine has to be divided by.
 */
int ptstore_time_next_copy(ptstore_t* st, void* before /*cudaEvent_t*/, void* after /*cudaEvent_t*/);

/*
 * Measurement aid (no paper counterpart; needs no handle): run the bulk copy engine's ring over two plain device buffers
 * in one traffic pattern, so the ceilings of the engine on this GPU can be measured next to a real fetch.
 *   mode  PTSTORE_PROBE_READ   loads only (global -> shared, data dropped)
 *         PTSTORE_PROBE_WRITE  stores only (shared -> global from a resident stage)
 *         PTSTORE_PROBE_COPY   one store per load
 *         PTSTORE_PROBE_MIX    writes_x100 / 100 stores per load on average (100..3200): the pattern of a fetch whose source
 *                              blocks are shared by several prompts
 *   src   `bytes` bytes; dst: `bytes` * ceil(writes_x100 / 100) bytes (`bytes` for the other modes); both 16-byte aligned
 *   bytes a multiple of 1024 * stage_bytes; with scatter != 0, bytes / stage_bytes / 64 must be a power of two
 *   stages, stage_bytes, ctas_per_sm   the ring: 2..32 stages of stage_bytes (multiple of 16, ring <= 200 KiB), 1..8 CTAs per SM
 *   scatter != 0   destinations laid out like a paged cache (64 planes, a pseudo-random block per 64 pieces) instead of linearly
 *   status device uint32, caller-cleared: PTSTORE_S_TIMEOUT is OR-ed in if a bounded wait expired
 * Bytes moved: `bytes` read (not for WRITE) + `bytes` x stores per load written.  Enqueues one kernel on `stream`.
 */
#define PTSTORE_PROBE_READ   0
#define PTSTORE_PROBE_WRITE  1
#define PTSTORE_PROBE_COPY   2
#define PTSTORE_PROBE_MIX    3
int ptstore_copy_probe(const void* src, void* dst, uint64_t bytes, int32_t mode, uint32_t writes_x100, int32_t stages,
                       uint32_t stage_bytes, int32_t ctas_per_sm, int32_t scatter, uint32_t* status, ptstore_stream_t stream);

/* Number of this library's kernels launched through the handle so far (host counter, no sync). */
uint64_t ptstore_launch_count(const ptstore_t* st);

/* cudaError_t value of the last failed CUDA call on this handle (0 if none). */
int ptstore_last_cuda_error(const ptstore_t* st);

/*
 * Gather without a handle, a workspace or any allocation (the paper has no counterpart: its store always
 * owns an allocator, Section 5).  For callers that must not call cudaMalloc — code running after a
 * serving engine has frozen its memory budget, or a plugin that receives pointers but no allocator — and
 * therefore cannot supply the workspace a handle needs.  Does exactly what ptstore_fetch does for HBM
 * block ids: for every r, j < matched_blocks[r], layer and K/V plane, one chunk is copied from pool
 * block block_ids[r*max_blocks+j] to cache block block_tables[r*max_blocks+j].
 *   hbm_pool     device memory, [hbm_blocks][num_layers][2][chunk_bytes], 16-byte aligned
 *   status_out   device uint32 or NULL: receives PTSTORE_S_BOUNDS if an id or table entry was skipped, else 0
 * Scratch (prefix sums, descriptor list) is a fixed device array inside the library, PTSTORE_STATIC_SCRATCH_BYTES
 * on every GPU that loads it, held until process exit.  Limits: R <= PTSTORE_STATIC_MAX_REQUESTS and
 * R*max_blocks <= PTSTORE_STATIC_MAX_PAIRS, else PTSTORE_E_LIMIT.  All calls on a GPU share that array: calls
 * that overlap on the GPU race, so keep them on one stream or order them.  The first call on each device
 * (made with that device current) looks up the array's address; issue it before any stream capture, and do not make
 * the first calls for one device from two host threads at once (the lookup is cached without a lock).
 * Calls no cudaMalloc / cudaFree / allocating routine.  Enqueues on `stream` and returns.
 */
#define PTSTORE_STATIC_MAX_REQUESTS   1024u
#define PTSTORE_STATIC_MAX_PAIRS      65536u
#define PTSTORE_STATIC_SCRATCH_BYTES  (4096u + 4352u + 8u * PTSTORE_STATIC_MAX_PAIRS)
int ptstore_fetch_static(const void* hbm_pool, uint32_t hbm_blocks, uint32_t num_layers, uint64_t chunk_bytes,
                         const int32_t* block_ids, const int32_t* matched_blocks, int32_t R, int32_t max_blocks,
                         const ptstore_paged_cache_t* dst /*host struct*/, const int32_t* block_tables,
                         uint32_t* status_out, ptstore_stream_t stream);

/* Static text for a PTSTORE_E_* code. */
const char* ptstore_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* PTSTORE_H */
