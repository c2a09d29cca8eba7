// Context, error handling, descriptor ring, pinned-memory registration.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>

#include <cuda.h>   // types of the driver's pointer query only; the entry point is looked up at run time

#include "internal.h"

namespace tal {

talaria_status_t cuda_fail(talaria_ctx *ctx, cudaError_t e) {
  if (ctx) ctx->last_cuda_error = (int32_t)e;
  (void)cudaGetLastError();  // clear the sticky-free error so later calls start clean
  return TALARIA_ERR_CUDA;
}

talaria_status_t acquire_slot(talaria_ctx *ctx, size_t bytes, DescSlot **out) {
  DescSlot &s = ctx->ring[ctx->ring_next];
  ctx->ring_next = (ctx->ring_next + 1) % kRing;
  if (s.used) {
    TAL_CUDA(ctx, cudaEventSynchronize(s.ev));
    s.used = false;
  }
  if (s.cap < bytes) {
    // Growing frees device memory, which makes the whole device wait.  Do it once for
    // the whole ring so the stall cannot recur slot by slot while other streams
    // are busy.
    const size_t cap = std::max<size_t>(bytes + bytes / 2, kSlotBytes);
    for (DescSlot &r : ctx->ring) {
      if (r.cap >= cap) continue;
      if (r.used) {
        TAL_CUDA(ctx, cudaEventSynchronize(r.ev));
        r.used = false;
      }
      if (r.h) cudaFreeHost(r.h);
      if (r.d) cudaFree(r.d);
      r.h = r.d = nullptr;
      r.cap = 0;
      TAL_CUDA(ctx, cudaHostAlloc((void **)&r.h, cap, cudaHostAllocDefault));
      TAL_CUDA(ctx, cudaMalloc((void **)&r.d, cap));
      r.cap = cap;
    }
  }
  *out = &s;
  return TALARIA_OK;
}

talaria_status_t upload_slot(talaria_ctx *ctx, DescSlot *slot, size_t bytes, cudaStream_t stream) {
  if (bytes == 0) return TALARIA_OK;
  TAL_CUDA(ctx, cudaMemcpyAsync(slot->d, slot->h, bytes, cudaMemcpyHostToDevice, stream));
  ctx->counters.memcpy_calls++;
  return TALARIA_OK;
}

talaria_status_t release_slot(talaria_ctx *ctx, DescSlot *slot, cudaStream_t stream) {
  TAL_CUDA(ctx, cudaEventRecord(slot->ev, stream));
  slot->used = true;
  return TALARIA_OK;
}

talaria_status_t grow(talaria_ctx *ctx, DevBuf *b, size_t bytes) {
  if (b->cap >= bytes) return TALARIA_OK;
  size_t cap = std::max<size_t>(bytes + bytes / 4, 1 << 20);
  if (b->p) {
    // cudaFree waits for the device, so nothing still reads the old buffer
    TAL_CUDA(ctx, cudaFree(b->p));
    b->p = nullptr;
    b->cap = 0;
  }
  cudaError_t e = cudaMalloc((void **)&b->p, cap);
  if (e == cudaErrorMemoryAllocation) {
    (void)cudaGetLastError();
    return TALARIA_ERR_NO_MEMORY;
  }
  TAL_CUDA(ctx, e);
  b->cap = cap;
  return TALARIA_OK;
}

talaria_status_t mapped_pointer(talaria_ctx *ctx, const void *host, void **dev_alias) {
  cudaPointerAttributes a{};
  cudaError_t e = cudaPointerGetAttributes(&a, host);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return TALARIA_ERR_HOST_NOT_PINNED;
  }
  if (a.type != cudaMemoryTypeHost || a.devicePointer == nullptr) return TALARIA_ERR_HOST_NOT_PINNED;
  (void)ctx;
  *dev_alias = a.devicePointer;
  return TALARIA_OK;
}

talaria_status_t require_device_pointer(talaria_ctx *ctx, const void *p) {
  cudaPointerAttributes a{};
  cudaError_t e = cudaPointerGetAttributes(&a, p);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return TALARIA_ERR_INVALID_ARG;
  }
  if (a.type == cudaMemoryTypeDevice || a.type == cudaMemoryTypeManaged) {
    if (a.type == cudaMemoryTypeDevice && a.device != ctx->device) return TALARIA_ERR_INVALID_ARG;
    return TALARIA_OK;
  }
  return TALARIA_ERR_INVALID_ARG;
}

bool RangeCache::covers(uintptr_t p, uintptr_t bytes) const {
  // last range that starts at or before p
  auto it = std::upper_bound(v.begin(), v.end(), p, [](uintptr_t x, const AddrRange &r) { return x < r.lo; });
  if (it == v.begin()) return false;
  --it;
  return p >= it->lo && p + bytes <= it->hi && p + bytes >= p;
}

bool RangeCache::find(uintptr_t p, AddrRange *out) const {
  auto it = std::upper_bound(v.begin(), v.end(), p, [](uintptr_t x, const AddrRange &r) { return x < r.lo; });
  if (it == v.begin()) return false;
  --it;
  if (p < it->lo || p >= it->hi) return false;
  *out = *it;
  return true;
}

void RangeCache::insert(AddrRange r) {
  // whatever overlaps the new range described memory that has been freed since
  v.erase(std::remove_if(v.begin(), v.end(), [&](const AddrRange &o) { return o.lo < r.hi && r.lo < o.hi; }), v.end());
  v.insert(std::upper_bound(v.begin(), v.end(), r.lo, [](uintptr_t x, const AddrRange &o) { return x < o.lo; }), r);
  if (v.size() > 4096) v.erase(v.begin(), v.begin() + 2048);   // bounded; dropped entries are simply asked again
}

// The allocation (or registration) that holds p, as the driver knows it.  The driver entry
// point is resolved through the runtime, so the library does not link against libcuda.
static bool query_allocation(const void *p, AddrRange *out) {
  typedef CUresult (*pointer_attr_fn)(void *, CUpointer_attribute, CUdeviceptr);
  static pointer_attr_fn fn = []() -> pointer_attr_fn {
    void *f = nullptr;
    cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuPointerGetAttribute", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess) {
      (void)cudaGetLastError();
      return nullptr;
    }
    return (pointer_attr_fn)f;
  }();
  if (!fn) return false;
  CUdeviceptr start = 0;
  size_t size = 0;
  if (fn(&start, CU_POINTER_ATTRIBUTE_RANGE_START_ADDR, (CUdeviceptr)(uintptr_t)p) != CUDA_SUCCESS) return false;
  if (fn(&size, CU_POINTER_ATTRIBUTE_RANGE_SIZE, (CUdeviceptr)(uintptr_t)p) != CUDA_SUCCESS) return false;
  if (size == 0 || (uintptr_t)p < (uintptr_t)start || (uintptr_t)p >= (uintptr_t)start + size) return false;
  *out = AddrRange{(uintptr_t)start, (uintptr_t)start + size};
  return true;
}

talaria_status_t mapped_range(talaria_ctx *ctx, const void *host, int64_t bytes, void **dev_alias) {
  if (bytes < 0) return TALARIA_ERR_INVALID_ARG;
  const uintptr_t p = (uintptr_t)host, n = (uintptr_t)bytes;
  // ranges registered through this context: their size is known exactly
  for (const auto &r : ctx->registered) {
    const uintptr_t lo = (uintptr_t)r.first, hi = lo + r.second;
    if (p >= lo && p < hi) {
      TAL_TRY(mapped_pointer(ctx, host, dev_alias));
      return (!ctx->cfg.validate || p + n <= hi) ? TALARIA_OK : TALARIA_ERR_EXTENT;
    }
  }
  TAL_TRY(mapped_pointer(ctx, host, dev_alias));
  if (!ctx->cfg.validate || bytes <= 1) return TALARIA_OK;
  if (p + n < p) return TALARIA_ERR_EXTENT;
  if (ctx->host_ranges.covers(p, n)) return TALARIA_OK;
  AddrRange a{};
  if (query_allocation(host, &a)) {
    ctx->host_ranges.insert(a);
    return p + n <= a.hi ? TALARIA_OK : TALARIA_ERR_EXTENT;
  }
  // no range from the driver: at least the last byte must be pinned and mapped right behind the first
  void *last = nullptr;
  if (mapped_pointer(ctx, (const char *)host + (bytes - 1), &last) != TALARIA_OK) return TALARIA_ERR_EXTENT;
  return ((uintptr_t)last - (uintptr_t)*dev_alias == n - 1) ? TALARIA_OK : TALARIA_ERR_EXTENT;
}

talaria_status_t mapped_range(talaria_ctx *ctx, HostRangeMemo *memo, const void *host, int64_t bytes, void **dev_alias) {
  const uintptr_t p = (uintptr_t)host;
  if (bytes >= 0 && memo->alias_lo && p >= memo->lo && p + (uintptr_t)bytes >= p && p + (uintptr_t)bytes <= memo->hi) {
    *dev_alias = (void *)(memo->alias_lo + (p - memo->lo));
    return TALARIA_OK;
  }
  TAL_TRY(mapped_range(ctx, host, bytes, dev_alias));
  // remember the registration or allocation that answered (the driver has just confirmed it)
  AddrRange a{};
  bool known = false;
  for (const auto &r : ctx->registered)
    if (p >= (uintptr_t)r.first && p < (uintptr_t)r.first + r.second) {
      a = AddrRange{(uintptr_t)r.first, (uintptr_t)r.first + r.second};
      known = true;
      break;
    }
  if (!known) known = ctx->host_ranges.find(p, &a);
  if (known) {
    memo->lo = a.lo;
    memo->hi = a.hi;
    memo->alias_lo = (const char *)*dev_alias - (p - a.lo);
  }
  return TALARIA_OK;
}

talaria_status_t require_device_range(talaria_ctx *ctx, const void *ptr, int64_t bytes) {
  if (bytes < 0) return TALARIA_ERR_INVALID_ARG;
  const uintptr_t p = (uintptr_t)ptr, n = (uintptr_t)bytes;
  if (ctx->cfg.validate && p + n >= p && ctx->dev_ranges.covers(p, n ? n : 1)) return TALARIA_OK;
  TAL_TRY(require_device_pointer(ctx, ptr));
  if (!ctx->cfg.validate || bytes <= 1) return TALARIA_OK;
  if (p + n < p) return TALARIA_ERR_EXTENT;
  AddrRange a{};
  if (query_allocation(ptr, &a)) {
    ctx->dev_ranges.insert(a);
    return p + n <= a.hi ? TALARIA_OK : TALARIA_ERR_EXTENT;
  }
  return require_device_pointer(ctx, (const char *)ptr + (bytes - 1)) == TALARIA_OK ? TALARIA_OK : TALARIA_ERR_EXTENT;
}

}  // namespace tal

using namespace tal;

static void destroy_impl(talaria_ctx *ctx) {
  for (auto &ln : ctx->lane) {
    for (int j = 0; j < 2; ++j) {
      if (ln.s[j]) {
        cudaStreamSynchronize(ln.s[j]);
        cudaStreamDestroy(ln.s[j]);
      }
      if (ln.done[j]) cudaEventDestroy(ln.done[j]);
    }
    if (ln.fork) cudaEventDestroy(ln.fork);
    if (ln.buf) cudaFree(ln.buf);
  }
  if (ctx->reload_stream) {
    cudaStreamSynchronize(ctx->reload_stream);
    cudaStreamDestroy(ctx->reload_stream);
  }
  for (cudaEvent_t e : ctx->tm)
    if (e) cudaEventDestroy(e);
  if (ctx->match_done) cudaEventDestroy(ctx->match_done);
  if (ctx->stage_free) cudaEventDestroy(ctx->stage_free);
  if (ctx->reload_fork) cudaEventDestroy(ctx->reload_fork);
  if (ctx->reload_done) cudaEventDestroy(ctx->reload_done);
  for (auto &s : ctx->ring) {
    if (s.used) cudaEventSynchronize(s.ev);
    if (s.ev) cudaEventDestroy(s.ev);
    if (s.h) cudaFreeHost(s.h);
    if (s.d) cudaFree(s.d);
  }
  if (ctx->prefix_busy) cudaEventSynchronize(ctx->prefix_done);
  if (ctx->prefix_done) cudaEventDestroy(ctx->prefix_done);
  if (ctx->prefix_counters) cudaFree(ctx->prefix_counters);
  if (ctx->status_host) cudaFreeHost(ctx->status_host);
  if (ctx->prefix_scratch.p) cudaFree(ctx->prefix_scratch.p);
  if (ctx->host_tok.p) cudaFree(ctx->host_tok.p);
  if (ctx->match_pin) cudaFreeHost(ctx->match_pin);
  for (auto &r : ctx->registered) cudaHostUnregister(r.first);
  (void)cudaGetLastError();
  delete ctx;
}

extern "C" talaria_status_t talaria_create(talaria_ctx **out, int32_t device, const talaria_config_t *cfg) {
  if (!out) return TALARIA_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
    (void)cudaGetLastError();
    return TALARIA_ERR_CUDA;
  }
  talaria_ctx *ctx = new (std::nothrow) talaria_ctx();
  if (!ctx) return TALARIA_ERR_NO_MEMORY;
  ctx->device = device;
  if (cfg) ctx->cfg = *cfg;
  if (!cfg) ctx->cfg.validate = 1;
  if (ctx->cfg.bounce_bytes <= 0) ctx->cfg.bounce_bytes = 128ll << 20;
  if (ctx->cfg.bounce_bytes < (1 << 20)) ctx->cfg.bounce_bytes = 1 << 20;
  if (ctx->cfg.host_match_bytes <= 0) ctx->cfg.host_match_bytes = 16ll << 20;
  if (ctx->cfg.host_match_bytes < (1 << 20)) ctx->cfg.host_match_bytes = 1 << 20;
  if (const char *v = getenv("TALARIA_VARIANT")) {
    int x = atoi(v);
    if (x >= TALARIA_VARIANT_AUTO && x <= TALARIA_VARIANT_RUNS) ctx->cfg.variant = x;
  }
  if (ctx->cfg.variant < TALARIA_VARIANT_AUTO || ctx->cfg.variant > TALARIA_VARIANT_RUNS) {
    delete ctx;
    return TALARIA_ERR_INVALID_ARG;
  }
  DeviceGuard g(device);
  talaria_status_t st = [&]() -> talaria_status_t {
    if (!g.ok) return TALARIA_ERR_CUDA;
    cudaDeviceProp prop{};
    TAL_CUDA(ctx, cudaGetDeviceProperties(&prop, device));
    ctx->sm_count = prop.multiProcessorCount;
    for (auto &s : ctx->ring) {
      TAL_CUDA(ctx, cudaEventCreateWithFlags(&s.ev, cudaEventDisableTiming));
      TAL_CUDA(ctx, cudaHostAlloc((void **)&s.h, kSlotBytes, cudaHostAllocDefault));
      TAL_CUDA(ctx, cudaMalloc((void **)&s.d, kSlotBytes));
      s.cap = kSlotBytes;
    }
    TAL_CUDA(ctx, cudaHostAlloc((void **)&ctx->status_host, 64, cudaHostAllocMapped));
    *ctx->status_host = 0;
    TAL_CUDA(ctx, cudaHostGetDevicePointer((void **)&ctx->status_dev, ctx->status_host, 0));
    TAL_CUDA(ctx, cudaMalloc((void **)&ctx->prefix_counters, 64 * sizeof(unsigned int)));
    TAL_CUDA(ctx, cudaMemset(ctx->prefix_counters, 0, 64 * sizeof(unsigned int)));
    TAL_CUDA(ctx, cudaEventCreateWithFlags(&ctx->prefix_done, cudaEventDisableTiming));
    TAL_TRY(grow(ctx, &ctx->host_tok, (size_t)ctx->cfg.host_match_bytes));
    TAL_CUDA(ctx, cudaHostAlloc((void **)&ctx->match_pin, ctx->host_tok.cap, cudaHostAllocMapped));
    TAL_CUDA(ctx, cudaHostGetDevicePointer((void **)&ctx->match_pin_dev, ctx->match_pin, 0));
    TAL_CUDA(ctx, cudaEventCreateWithFlags(&ctx->match_done, cudaEventDisableTiming));
    TAL_CUDA(ctx, cudaEventCreateWithFlags(&ctx->stage_free, cudaEventDisableTiming));
    // Internal streams run at the highest priority: their kernels are short packing
    // steps that gate copy-engine transfers, so they should not queue behind a long
    // kernel of the caller's (for example a staging copy on another stream).
    int prio_least = 0, prio_greatest = 0;
    TAL_CUDA(ctx, cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest));
    // highest priority as well: the reload kernel is a handful of CTAs that must find SM slots while
    // the D2D gather, launched just before it with a grid far larger than the GPU, is still running
    TAL_CUDA(ctx, cudaStreamCreateWithPriority(&ctx->reload_stream, cudaStreamNonBlocking, prio_greatest));
    for (cudaEvent_t &e : ctx->tm) TAL_CUDA(ctx, cudaEventCreate(&e));
    TAL_CUDA(ctx, cudaEventCreateWithFlags(&ctx->reload_fork, cudaEventDisableTiming));
    TAL_CUDA(ctx, cudaEventCreateWithFlags(&ctx->reload_done, cudaEventDisableTiming));
    for (auto &ln : ctx->lane) {
      for (int j = 0; j < 2; ++j) {
        TAL_CUDA(ctx, cudaStreamCreateWithPriority(&ln.s[j], cudaStreamNonBlocking, prio_greatest));
        TAL_CUDA(ctx, cudaEventCreateWithFlags(&ln.done[j], cudaEventDisableTiming));
      }
      TAL_CUDA(ctx, cudaEventCreateWithFlags(&ln.fork, cudaEventDisableTiming));
      ln.half = ((size_t)ctx->cfg.bounce_bytes / 2) & ~(size_t)255;
      cudaError_t e = cudaMalloc((void **)&ln.buf, ln.half * 2);
      if (e == cudaErrorMemoryAllocation) {
        (void)cudaGetLastError();
        return TALARIA_ERR_NO_MEMORY;
      }
      TAL_CUDA(ctx, e);
    }
    return TALARIA_OK;
  }();
  if (st != TALARIA_OK) {
    destroy_impl(ctx);
    return st;
  }
  *out = ctx;
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_destroy(talaria_ctx *ctx) {
  if (!ctx) return TALARIA_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  destroy_impl(ctx);
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_host_register(talaria_ctx *ctx, void *host, size_t bytes) {
  if (!ctx || !host || bytes == 0) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(ctx->mu);
  DeviceGuard g(ctx->device);
  TAL_CUDA(ctx, cudaHostRegister(host, bytes, cudaHostRegisterMapped | cudaHostRegisterPortable));
  ctx->registered.emplace_back((char *)host, bytes);
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_host_unregister(talaria_ctx *ctx, void *host) {
  if (!ctx || !host) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(ctx->mu);
  DeviceGuard g(ctx->device);
  for (size_t k = 0; k < ctx->registered.size(); ++k) {
    if (ctx->registered[k].first == (char *)host) {
      TAL_CUDA(ctx, cudaHostUnregister(host));
      ctx->registered.erase(ctx->registered.begin() + k);
      ctx->host_ranges.v.clear();          // what the driver said about this memory no longer holds
      return TALARIA_OK;
    }
  }
  return TALARIA_ERR_INVALID_ARG;
}

extern "C" talaria_status_t talaria_sync(talaria_ctx *ctx, void *stream) {
  if (!ctx) return TALARIA_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  TAL_CUDA(ctx, cudaStreamSynchronize((cudaStream_t)stream));
  // a copy kernel met a table entry outside the pool (possible only with validation off):
  // it skipped that chunk instead of touching foreign memory; report it once
  std::lock_guard<std::mutex> lk(ctx->mu);
  if (*(volatile unsigned int *)ctx->status_host) {
    *(volatile unsigned int *)ctx->status_host = 0;
    return TALARIA_ERR_BAD_BLOCK_ID;
  }
  return TALARIA_OK;
}

extern "C" const char *talaria_strerror(talaria_status_t s) {
  switch (s) {
    case TALARIA_OK: return "ok";
    case TALARIA_ERR_INVALID_ARG: return "invalid argument";
    case TALARIA_ERR_BAD_BLOCK_ID: return "block id out of range";
    case TALARIA_ERR_DUP_BLOCK: return "duplicate block id in a restore table";
    case TALARIA_ERR_HOST_NOT_PINNED: return "host buffer is not pinned / device-mapped";
    case TALARIA_ERR_EXTENT: return "buffer smaller than the layout requires";
    case TALARIA_ERR_OVERLAP: return "stage plan ranges overlap";
    case TALARIA_ERR_CUDA: return "CUDA call failed (see talaria_last_cuda_error)";
    case TALARIA_ERR_NO_MEMORY: return "out of memory";
    default: return "unknown status";
  }
}

extern "C" int32_t talaria_last_cuda_error(talaria_ctx *ctx) { return ctx ? ctx->last_cuda_error : 0; }

extern "C" talaria_status_t talaria_get_counters(talaria_ctx *ctx, talaria_counters_t *out) {
  if (!ctx || !out) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(ctx->mu);
  *out = ctx->counters;
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_set_timing(talaria_ctx *ctx, int32_t enabled) {
  if (!ctx) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(ctx->mu);
  ctx->timing = enabled != 0;
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_get_timing(talaria_ctx *ctx, talaria_timing_t *out) {
  if (!ctx || !out) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(ctx->mu);
  DeviceGuard g(ctx->device);
  if (ctx->tm_op == 0) return TALARIA_ERR_INVALID_ARG;
  talaria_timing_t t{};
  t.op = ctx->tm_op;
  TAL_CUDA(ctx, cudaEventSynchronize(ctx->tm[1]));
  TAL_CUDA(ctx, cudaEventElapsedTime(&t.total_ms, ctx->tm[0], ctx->tm[1]));
  if (ctx->tm_d2d) {
    TAL_CUDA(ctx, cudaEventSynchronize(ctx->tm[3]));
    TAL_CUDA(ctx, cudaEventElapsedTime(&t.d2d_ms, ctx->tm[2], ctx->tm[3]));
  }
  if (ctx->tm_h2d) {
    TAL_CUDA(ctx, cudaEventSynchronize(ctx->tm[5]));
    TAL_CUDA(ctx, cudaEventElapsedTime(&t.h2d_ms, ctx->tm[4], ctx->tm[5]));
  }
  if (t.op == 1) t.d2h_ms = t.total_ms;
  if (t.op == 2) t.h2d_ms = t.total_ms;
  *out = t;
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_reset_counters(talaria_ctx *ctx) {
  if (!ctx) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(ctx->mu);
  int32_t v = ctx->counters.last_variant;
  ctx->counters = talaria_counters_t{};
  ctx->counters.last_variant = v;
  return TALARIA_OK;
}

extern "C" int64_t talaria_prefix_agree(int32_t n_ranks, const int64_t *committed_blocks,
                                        const uint64_t *hashes, int64_t stride) {
  if (n_ranks <= 0 || !committed_blocks) return 0;
  int64_t agreed = committed_blocks[0];
  for (int32_t r = 1; r < n_ranks; ++r) agreed = std::min(agreed, committed_blocks[r]);
  if (agreed <= 0 || !hashes) return 0;
  // every rank is compared with rank 0; the first column where any differs ends the prefix
  for (int32_t r = 1; r < n_ranks; ++r) {
    const uint64_t *a = hashes, *b = hashes + (int64_t)r * stride;
    int64_t k = 0;
    while (k < agreed && a[k] == b[k]) ++k;
    agreed = k;
  }
  return agreed;
}
