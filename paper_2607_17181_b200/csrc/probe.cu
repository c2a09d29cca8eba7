// Copy-mechanism probe: the same bytes moved by 128-bit loads/stores, 256-bit loads/stores
// and TMA bulk copies (cp.async.bulk through a shared-memory ring), between any two
// device-visible ranges (HBM or device-mapped pinned host memory).  It exists so the choice
// of mechanism in the copy kernels rests on numbers anyone can reproduce:
// `bench.py --workload probe`.
#include <algorithm>

#include "internal.h"

namespace tal {

constexpr int kProbeChunk = 16384;   // bytes per TMA transfer = one Qwen3-235B KV chunk
constexpr int kProbeStages = 4;

template <int VB>
__global__ void __launch_bounds__(512) probe_ldst_kernel(const char *__restrict__ src, char *__restrict__ dst,
                                                        int64_t bytes) {
  // a warp moves 4 KiB per step, 128 bytes per lane in flight, like the copy kernels
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t u = warp; u < bytes / 4096; u += nwarps) {
    const char *s = src + u * 4096;
    char *d = dst + u * 4096;
    if (VB == 32) {
      Vec32 v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) v[k] = ld_cs_32(s + (lane + k * 32) * 32);
#pragma unroll
      for (int k = 0; k < 4; ++k) st_cs_32(d + (lane + k * 32) * 32, v[k]);
    } else {
      int4 v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = __ldcs((const int4 *)s + lane + k * 32);
#pragma unroll
      for (int k = 0; k < 8; ++k) __stcs((int4 *)d + lane + k * 32, v[k]);
    }
  }
}

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Bounded wait on an mbarrier phase: gives up after a fixed number of polls and reports it.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  for (int it = 0; it < (1 << 22); ++it) {
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}

// One thread per CTA drives a ring of kProbeStages chunks: bulk load global -> shared (completion
// on an mbarrier), bulk store shared -> global (bulk async-group).  No cluster, no multicast.
__global__ void probe_tma_kernel(const char *__restrict__ src, char *__restrict__ dst, int64_t nchunks,
                                 volatile unsigned int *status) {
  extern __shared__ __align__(128) char ring[];
  __shared__ __align__(8) unsigned long long bars[kProbeStages];
  if (threadIdx.x != 0) return;
  for (int s = 0; s < kProbeStages; ++s) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bars[s])));
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  const int64_t first = blockIdx.x, stride = gridDim.x;
  const int64_t mine = nchunks > first ? (nchunks - first + stride - 1) / stride : 0;
  auto load = [&](int64_t it) {
    const int s = (int)(it % kProbeStages);
    const uint32_t bar = smem_addr(&bars[s]), sm = smem_addr(ring + (size_t)s * kProbeChunk);
    const char *g = src + (first + it * stride) * (int64_t)kProbeChunk;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kProbeChunk) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(sm),
                 "l"(g), "r"(kProbeChunk), "r"(bar)
                 : "memory");
  };
  const int64_t ahead = mine < kProbeStages - 1 ? mine : kProbeStages - 1;
  int64_t issued = 0;
  for (; issued < ahead; ++issued) load(issued);
  for (int64_t it = 0; it < mine; ++it) {
    const int s = (int)(it % kProbeStages);
    if (!mbar_wait_bounded(smem_addr(&bars[s]), (uint32_t)((it / kProbeStages) & 1))) {
      // gave up waiting for a load: report it, give the other loads in flight one more bounded
      // wait each (they target this CTA's shared memory), then drain the stores and leave
      *status = 2u;
      for (int64_t j = it + 1; j < issued; ++j)
        (void)mbar_wait_bounded(smem_addr(&bars[j % kProbeStages]), (uint32_t)((j / kProbeStages) & 1));
      break;
    }
    char *g = dst + (first + it * stride) * (int64_t)kProbeChunk;
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(g),
                 "r"(smem_addr(ring + (size_t)s * kProbeChunk)), "r"(kProbeChunk)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    if (issued < mine) {
      asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // the previous store has read its stage
      load(issued);
      ++issued;
    }
  }
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

}  // namespace tal

extern "C" talaria_status_t talaria_probe_copy(talaria_ctx *ctx, int32_t mechanism, const void *src, void *dst,
                                               int64_t bytes, int32_t ctas, void *stream) {
  using namespace tal;
  if (!ctx || !src || !dst || bytes < 0 || ctas <= 0 || mechanism < 0 || mechanism > 2) return TALARIA_ERR_INVALID_ARG;
  if (bytes % kProbeChunk != 0 || ((uintptr_t)src | (uintptr_t)dst) % 32 != 0) return TALARIA_ERR_INVALID_ARG;
  if (bytes == 0) return TALARIA_OK;
  std::lock_guard<std::mutex> lk(ctx->mu);
  DeviceGuard g(ctx->device);
  if (!g.ok) return TALARIA_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  if (mechanism == 0) {
    probe_ldst_kernel<16><<<ctas, 512, 0, st>>>((const char *)src, (char *)dst, bytes);
  } else if (mechanism == 1) {
    probe_ldst_kernel<32><<<ctas, 512, 0, st>>>((const char *)src, (char *)dst, bytes);
  } else {
    const int smem = kProbeStages * kProbeChunk;
    TAL_CUDA(ctx, cudaFuncSetAttribute(probe_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    probe_tma_kernel<<<ctas, 32, smem, st>>>((const char *)src, (char *)dst, bytes / kProbeChunk, ctx->status_dev);
  }
  TAL_CUDA(ctx, cudaGetLastError());
  ctx->counters.kernel_launches++;
  return TALARIA_OK;
}
