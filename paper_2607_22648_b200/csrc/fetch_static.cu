// ptstore_fetch_static: the gather of ptstore_fetch for callers that cannot allocate device memory.
//
// Who needs it: code that runs where cudaMalloc is off limits — inside a region whose memory budget is
// already fixed (a serving engine after its memory profiling pass, a plugin that is handed pointers but
// no allocator), or a process that must not disturb a caching allocator owned by someone else.  Such a
// caller cannot provide the workspace a store handle needs, yet it may still hold a pool pointer, the
// block ids of a prefix and a paged cache to fill.  This entry point needs no handle and no workspace:
// its scratch (request prefix sums, the copy descriptor list, a small control block) lives in a
// file-scope device array that every GPU loading this library holds until the process exits.
//
// Consequences the caller must know:
//   - the array has a fixed size: at most PTSTORE_STATIC_MAX_REQUESTS requests and
//     PTSTORE_STATIC_MAX_PAIRS (request, block) entries per call; larger calls are refused;
//   - every call on a GPU shares the one array.  Calls that overlap on the GPU (two streams, two
//     threads) race on it; serialise them;
//   - the first call on each device looks up the array's device address (cudaGetSymbolAddress) with that
//     device current; make that first call before any stream capture begins, and not from two host threads
//     at once (the address is cached without a lock);
//   - nothing is allocated or freed here: no cudaMalloc, no cudaFree, no allocating library call.
#include "../../include/ptstore.h"

// This file is its own translation unit; the shared kernel headers are compiled here under another
// namespace name so that their kernels do not collide with the copies in the main translation unit.
#define pts pts_noalloc
#include "common.cuh"
#include "copy.cuh"

using namespace pts;

namespace {

constexpr u64 SCR_CTRL = 0;                                                    // Ctrl block
constexpr u64 SCR_PREFIX = 4096;                                               // u32 [MAX_REQUESTS + 1]
constexpr u64 SCR_DESC = SCR_PREFIX + ((PTSTORE_STATIC_MAX_REQUESTS + 1) * 4 + 255) / 256 * 256;   // int2 [MAX_PAIRS]
constexpr u64 SCR_BYTES = SCR_DESC + (u64)PTSTORE_STATIC_MAX_PAIRS * 8;
static_assert(sizeof(Ctrl) <= SCR_PREFIX, "control block must fit in front of the prefix array");

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress, not an address
// a kernel could use.
static __device__ __align__(256) unsigned char g_static_scratch[SCR_BYTES];

constexpr int MAX_DEVICES = 64;
unsigned char* g_scratch_addr[MAX_DEVICES];    // device address of the array, per device ordinal (0 = not looked up yet)

// status word of the call: cleared here, read back at the end
__global__ void static_begin_kernel(Ctrl* c) {
  c->status = 0;
  c->n_pairs = 0;
}
__global__ void static_end_kernel(const Ctrl* c, u32* status_out) {
  if (status_out) *status_out = c->status;
}

}  // namespace

extern "C" int ptstore_fetch_static(const void* hbm_pool, uint32_t hbm_blocks, uint32_t num_layers, uint64_t chunk_bytes,
                                    const int32_t* block_ids, const int32_t* matched_blocks, int32_t R, int32_t max_blocks,
                                    const ptstore_paged_cache_t* dst, const int32_t* block_tables, uint32_t* status_out,
                                    ptstore_stream_t stream) {
  if (R < 0 || max_blocks < 1) return PTSTORE_E_INVAL;
  if ((u32)R > PTSTORE_STATIC_MAX_REQUESTS || (u64)R * (u64)max_blocks > PTSTORE_STATIC_MAX_PAIRS) return PTSTORE_E_LIMIT;
  if (!hbm_pool || (reinterpret_cast<uintptr_t>(hbm_pool) & 15u) || hbm_blocks == 0 || hbm_blocks >= 0x7FFFFFFFu || num_layers == 0 ||
      chunk_bytes == 0 || chunk_bytes % 16)
    return PTSTORE_E_INVAL;
  if (!dst || !dst->layer_base || dst->num_blocks == 0 || dst->kv_stride_bytes % 16 || dst->block_stride_bytes % 16 ||
      dst->block_stride_bytes < chunk_bytes)
    return PTSTORE_E_INVAL;
  if (R > 0 && (!block_ids || !matched_blocks || !block_tables)) return PTSTORE_E_INVAL;

  // set-up, once per device, with that device current
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) { (void)cudaGetLastError(); return PTSTORE_E_CUDA; }
  if (!g_scratch_addr[dev]) {
    unsigned char* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch) != cudaSuccess || !p) {
      (void)cudaGetLastError();
      return PTSTORE_E_CUDA;
    }
    g_scratch_addr[dev] = p;
  }
  unsigned char* scratch = g_scratch_addr[dev];
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  Store st = {};
  st.n[0] = hbm_blocks;
  st.n[1] = 0;
  st.ctrl = reinterpret_cast<Ctrl*>(scratch + SCR_CTRL);
  st.pool[0] = static_cast<unsigned char*>(const_cast<void*>(hbm_pool));
  st.pool[1] = nullptr;
  st.chunk_bytes = chunk_bytes;
  st.block_bytes = 2ull * num_layers * chunk_bytes;
  st.layers = num_layers;
  u32* prefix = reinterpret_cast<u32*>(scratch + SCR_PREFIX);
  int2* desc = reinterpret_cast<int2*>(scratch + SCR_DESC);
  Paged pc;
  pc.layer_base = reinterpret_cast<unsigned char* const*>(dst->layer_base);
  pc.kv_stride = dst->kv_stride_bytes;
  pc.block_stride = dst->block_stride_bytes;
  pc.num_blocks = dst->num_blocks;

  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) { (void)cudaGetLastError(); return PTSTORE_E_CUDA; }

  (void)cudaGetLastError();                                   // an error left pending by the caller's earlier calls is not ours to report
  static_begin_kernel<<<1, 1, 0, s>>>(st.ctrl);              // the array keeps the last call's contents: clear what must start at zero
  if (cudaGetLastError() != cudaSuccess) return PTSTORE_E_CUDA;
  if (R > 0) {
    scan_matched_kernel<<<1, 1024, 0, s>>>(st, matched_blocks, R, max_blocks, prefix);
    if (cudaGetLastError() != cudaSuccess) return PTSTORE_E_CUDA;
    long long total = (long long)R * max_blocks;
    int grid = (int)((total + 255) / 256);
    if (grid > sms * 8) grid = sms * 8;
    build_pairs_kernel<<<grid, 256, 0, s>>>(st, block_ids, matched_blocks, block_tables, R, max_blocks, dst->num_blocks, prefix, desc);
    if (cudaGetLastError() != cudaSuccess) return PTSTORE_E_CUDA;
    copy_vector_kernel<COPY_FETCH, 256, 4><<<sms * 16, 256, 0, s>>>(st, pc, desc, &st.ctrl->n_pairs);
    if (cudaGetLastError() != cudaSuccess) return PTSTORE_E_CUDA;
  }
  static_end_kernel<<<1, 1, 0, s>>>(st.ctrl, status_out);
  if (cudaGetLastError() != cudaSuccess) return PTSTORE_E_CUDA;
  return PTSTORE_OK;
}
