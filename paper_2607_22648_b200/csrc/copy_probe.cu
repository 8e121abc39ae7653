// ptstore_copy_probe: the bulk copy engine's ring (one issuing thread per CTA, bulk-async copies global -> shared ->
// global through mbarrier-tracked stages, as in copy.cuh) run over plain buffers in four traffic patterns, so that the
// ceilings of THIS engine on the machine at hand can be measured next to a real fetch: loads only, stores only, one
// store per load (a copy), and the read-once-write-many mix of a fetch whose source blocks are shared by several
// prompts.  A measurement aid; the store itself never calls it.
#include "../../include/ptstore.h"

#define pts pts_probe
#include "common.cuh"
#include "copy.cuh"

using namespace pts;

namespace {

struct ProbeTune {
  int mode;            // PTSTORE_PROBE_*
  int stages;
  u32 stage_bytes;
  u32 writes_x100;     // PTSTORE_PROBE_MIX: stores per load, times 100
  int scatter;         // destination pieces laid out like a paged cache: 64 planes, a pseudo-random block per source block
  u32 unit;            // consecutive pieces a CTA takes before striding on
};

__device__ __forceinline__ u32 probe_writes(const ProbeTune& t, u64 p) {
  if (t.mode == PTSTORE_PROBE_READ) return 0;
  if (t.mode != PTSTORE_PROBE_MIX) return 1;
  const u32 whole = t.writes_x100 / 100, frac = t.writes_x100 % 100;
  return whole + (((p * 37) % 100) < frac ? 1u : 0u);
}

__global__ void __launch_bounds__(32) copy_probe_kernel(const unsigned char* __restrict__ src, unsigned char* __restrict__ dst, u64 pieces,
                                                        u64 mult, ProbeTune t, u32* __restrict__ status) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) u64 bars[BULK_MAX_STAGES];
  if (threadIdx.x != 0) return;
  const int S = t.stages;
  const u32 SB = t.stage_bytes;
  const u64 U = t.unit;
  const u64 units = pieces / U;
  if (blockIdx.x >= units) return;
  const u64 mine = ((units - blockIdx.x + gridDim.x - 1) / gridDim.x) * U;
  for (int s = 0; s < S; ++s) mbar_init(&bars[s], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  fence_async_smem();
  auto piece = [&](u64 i) { return (blockIdx.x + (i / U) * gridDim.x) * U + (i % U); };
  auto dst_of = [&](u64 p, u32 k) {
    u64 q = p;
    if (t.scatter) { const u64 nb = pieces / 64; q = (p % 64) * nb + ((p / 64) * mult) % nb; }
    return dst + ((u64)k * pieces + q) * SB;
  };
  u64 issued = 0;
  int ls = 0;
  auto issue = [&]() {
    if (t.mode != PTSTORE_PROBE_WRITE) {
      mbar_expect_tx(&bars[ls], SB);
      bulk_g2s(smem + (size_t)ls * SB, src + piece(issued) * SB, SB, &bars[ls]);
    } else {
      mbar_expect_tx(&bars[ls], 0);                  // nothing to load: the phase completes at once
    }
    ++issued;
    ls = ls + 1 == S ? 0 : ls + 1;
  };
  for (int k = 0; k < S - 1 && issued < mine; ++k) issue();
  int s = 0;
  u32 parity = 0;
  u64 i = 0;
  bool ok = true;
  for (; i < mine; ++i) {
    if (!mbar_wait_bounded(&bars[s], parity, BULK_POLL_LIMIT)) { ok = false; break; }
    const u64 p = piece(i);
    const u32 w = probe_writes(t, p);
    for (u32 k = 0; k < w; ++k) bulk_s2g(dst_of(p, k), smem + (size_t)s * SB, SB);
    bulk_commit();
    if (issued < mine) { bulk_wait_read<1>(); issue(); }
    if (++s == S) { s = 0; parity ^= 1u; }
  }
  if (!ok) {
    atomicOr(status, S_TIMEOUT);
    for (u64 k = i; k < issued; ++k) {               // drain loads in flight (bounded)
      mbar_wait_bounded(&bars[s], parity, BULK_POLL_LIMIT);
      if (++s == S) { s = 0; parity ^= 1u; }
    }
  }
  bulk_wait_all();
}

}  // namespace

extern "C" int ptstore_copy_probe(const void* src, void* dst, uint64_t bytes, int32_t mode, uint32_t writes_x100, int32_t stages,
                                  uint32_t stage_bytes, int32_t ctas_per_sm, int32_t scatter, uint32_t* status, ptstore_stream_t stream) {
  if (!src || !dst || !status || (reinterpret_cast<uintptr_t>(src) & 15u) || (reinterpret_cast<uintptr_t>(dst) & 15u)) return PTSTORE_E_INVAL;
  if (mode < PTSTORE_PROBE_READ || mode > PTSTORE_PROBE_MIX) return PTSTORE_E_INVAL;
  if (stages < 2 || stages > BULK_MAX_STAGES || stage_bytes < 16 || stage_bytes % 16 || (u64)stages * stage_bytes > 200u * 1024u) return PTSTORE_E_INVAL;
  if (ctas_per_sm < 1 || ctas_per_sm > 8) return PTSTORE_E_INVAL;
  if (mode == PTSTORE_PROBE_MIX && (writes_x100 < 100 || writes_x100 > 3200)) return PTSTORE_E_INVAL;
  const u64 unit = 16;
  const u64 pieces = bytes / stage_bytes;
  if (pieces == 0 || bytes % stage_bytes || pieces % (64 * unit)) return PTSTORE_E_INVAL;
  if (scatter && ((pieces / 64) & (pieces / 64 - 1))) return PTSTORE_E_INVAL;      // the block permutation needs a power of two
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
    (void)cudaGetLastError();
    return PTSTORE_E_CUDA;
  }
  const int smem = stages * (int)stage_bytes;
  if (cudaFuncSetAttribute(copy_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
    (void)cudaGetLastError();
    return PTSTORE_E_CUDA;
  }
  ProbeTune t = {mode, stages, stage_bytes, writes_x100, scatter ? 1 : 0, (u32)unit};
  u64 mult = 2654435761ull % (pieces / 64);
  mult |= 1ull;                                        // odd: a bijection when pieces / 64 is a power of two
  copy_probe_kernel<<<sms * ctas_per_sm, 32, smem, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const unsigned char*>(src), static_cast<unsigned char*>(dst), pieces, mult, t, status);
  return cudaGetLastError() == cudaSuccess ? PTSTORE_OK : PTSTORE_E_CUDA;
}
