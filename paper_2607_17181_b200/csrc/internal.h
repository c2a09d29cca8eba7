// Internal declarations shared by the CUDA sources of libtalaria (not installed).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <mutex>
#include <utility>
#include <vector>

#include "talaria.h"

namespace tal {

constexpr int kRing = 8;              // descriptor slots in flight
constexpr size_t kSlotBytes = 2u << 20;  // initial size of each slot (pinned + device)
constexpr int kLanes = 2;             // 0: offload (device->host), 1: restore (host->device)
constexpr int64_t kReloadPiece = 32ll << 20;   // largest single host->device copy of a weight reload

struct DescSlot {
  char *h = nullptr;                  // pinned staging
  char *d = nullptr;                  // device copy
  size_t cap = 0;
  cudaEvent_t ev = nullptr;           // recorded after the last consumer was enqueued
  bool used = false;
};

struct BounceLane {
  cudaStream_t s[2] = {nullptr, nullptr};
  cudaEvent_t done[2] = {nullptr, nullptr};
  cudaEvent_t fork = nullptr;
  char *buf = nullptr;                // two halves of `half` bytes
  size_t half = 0;
};

struct DevBuf {                       // growable device scratch
  char *p = nullptr;
  size_t cap = 0;
};

// Allocations the driver has already described to us, sorted by start and disjoint.  A hit
// saves the driver query; a miss or a range that looks too short is always asked again, so a
// stale entry (memory freed and allocated anew by the caller) can never cause a rejection.
struct AddrRange {
  uintptr_t lo, hi;
};
struct RangeCache {
  std::vector<AddrRange> v;
  bool covers(uintptr_t p, uintptr_t bytes) const;
  bool find(uintptr_t p, AddrRange *out) const;      // the cached range that holds p
  void insert(AddrRange r);
};

}  // namespace tal

struct talaria_ctx {
  int device = 0;
  int sm_count = 0;
  talaria_config_t cfg{};
  std::mutex mu;
  tal::DescSlot ring[tal::kRing];
  int ring_next = 0;
  tal::BounceLane lane[tal::kLanes];
  // Host-sourced reloads of a staged switch run on a stream of their own, cut into bounded
  // pieces, so a KV restore issued meanwhile gets its turns on the host link (Sec. 3.4 charges
  // the restore, not the weight reload, to the admission budget).
  cudaStream_t reload_stream = nullptr;
  cudaEvent_t reload_fork = nullptr, reload_done = nullptr;
  tal::DevBuf prefix_scratch;         // digests + per-tile mismatch positions
  unsigned int *prefix_counters = nullptr;  // per-pair tile counters of the fused prefix kernel (zero at rest)
  cudaEvent_t prefix_done = nullptr;  // end of the last prefix call (its scratch is shared)
  bool prefix_busy = false;
  cudaStream_t prefix_stream = nullptr;  // stream of that call (same stream: already ordered)
  tal::DevBuf host_tok;               // device side of talaria_prefix_match_host's staging (fixed size)
  char *match_pin = nullptr;          // pinned side, same size and layout
  cudaEvent_t match_done = nullptr;   // resident match: its kernels have written the result records
  cudaEvent_t stage_free = nullptr;   // ... and the prompts have been spread out of the device staging
  bool stage_busy = false;            // a spread may still be reading the device staging
  cudaStream_t stage_stream = nullptr;  // ... on this stream
  char *match_pin_dev = nullptr;      // ... as the device sees it (results are written through this mapping)
  std::vector<std::pair<char *, size_t>> registered;
  tal::RangeCache host_ranges;        // pinned host allocations seen so far
  tal::RangeCache dev_ranges;         // device allocations seen so far
  std::vector<uint64_t> dup_bits;     // restore-table duplicate check
  unsigned int *status_host = nullptr;  // pinned, device-mapped: kernels set it when they skip a bad entry
  unsigned int *status_dev = nullptr;   // the same word as the device sees it
  int32_t last_cuda_error = 0;
  talaria_counters_t counters{};
  // optional per-call timing: [0],[1] whole call on the caller's stream; [2],[3] the D2D gather
  // kernel of a stage; [4],[5] its host reloads on the reload stream
  bool timing = false;
  cudaEvent_t tm[6] = {};
  int32_t tm_op = 0;                  // 0 = nothing timed yet
  bool tm_d2d = false, tm_h2d = false;
};

namespace tal {

// Records the CUDA error in the context and maps it to TALARIA_ERR_CUDA.
talaria_status_t cuda_fail(talaria_ctx *ctx, cudaError_t e);

#define TAL_CUDA(ctx, call)                                   \
  do {                                                        \
    cudaError_t e__ = (call);                                 \
    if (e__ != cudaSuccess) return tal::cuda_fail((ctx), e__);\
  } while (0)

#define TAL_TRY(expr)                                         \
  do {                                                        \
    talaria_status_t s__ = (expr);                            \
    if (s__ != TALARIA_OK) return s__;                        \
  } while (0)

// Brackets one timed call on the caller's stream (no-op while timing is off).
struct CallTimer {
  talaria_ctx *ctx;
  cudaStream_t stream;
  CallTimer(talaria_ctx *c, cudaStream_t s, int32_t op) : ctx(c), stream(s) {
    if (!ctx->timing) return;
    ctx->tm_op = op;
    ctx->tm_d2d = ctx->tm_h2d = false;
    cudaEventRecord(ctx->tm[0], stream);
  }
  ~CallTimer() {
    if (ctx->timing) cudaEventRecord(ctx->tm[1], stream);
  }
};

// RAII: make the context's device current for the duration of a call.
struct DeviceGuard {
  int prev = -1;
  bool ok = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && cudaSetDevice(dev) == cudaSuccess) ok = true;
  }
  ~DeviceGuard() {
    if (ok && prev >= 0) cudaSetDevice(prev);
  }
};

// Descriptor ring: a pinned + device buffer pair of at least `bytes`, free to
// overwrite (its previous consumers have finished).
talaria_status_t acquire_slot(talaria_ctx *ctx, size_t bytes, DescSlot **out);
// Uploads the first `bytes` of the slot on `stream`.
talaria_status_t upload_slot(talaria_ctx *ctx, DescSlot *slot, size_t bytes, cudaStream_t stream);
// Marks the slot busy until everything enqueued on `stream` so far is done.
talaria_status_t release_slot(talaria_ctx *ctx, DescSlot *slot, cudaStream_t stream);

talaria_status_t grow(talaria_ctx *ctx, DevBuf *b, size_t bytes);

// Device-visible alias of a pinned host range, or HOST_NOT_PINNED.
talaria_status_t mapped_pointer(talaria_ctx *ctx, const void *host, void **dev_alias);
// OK if `p` is device memory of this context's device.
talaria_status_t require_device_pointer(talaria_ctx *ctx, const void *p);
// The same two checks for a whole range: every byte of [p, p + bytes) must belong to the
// one pinned (device) allocation that holds p.  HOST_NOT_PINNED / INVALID_ARG when the first
// byte is wrong, EXTENT when the range runs off its allocation or registration.  With
// validation off only the first byte is looked at.
talaria_status_t mapped_range(talaria_ctx *ctx, const void *host, int64_t bytes, void **dev_alias);
// The same for many ranges checked within ONE call: the pinned allocation that held the last
// range is remembered together with its device alias, and later ranges inside it are answered
// without asking the driver again (a plan with thousands of host-sourced chunks of one pinned
// buffer would otherwise pay a driver query each).  A memo must not outlive the call.
struct HostRangeMemo {
  uintptr_t lo = 0, hi = 0;
  const char *alias_lo = nullptr;
};
talaria_status_t mapped_range(talaria_ctx *ctx, HostRangeMemo *memo, const void *host, int64_t bytes, void **dev_alias);
talaria_status_t require_device_range(talaria_ctx *ctx, const void *p, int64_t bytes);

#ifdef __CUDACC__
// 256-bit streaming accesses (sm_100): fewer instructions per byte than 128-bit ones.
struct alignas(32) Vec32 {
  unsigned r[8];
};
__device__ __forceinline__ Vec32 ld_cs_32(const void *p) {
  Vec32 v;
  asm volatile("ld.global.cs.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(v.r[0]), "=r"(v.r[1]), "=r"(v.r[2]), "=r"(v.r[3]), "=r"(v.r[4]), "=r"(v.r[5]),
                 "=r"(v.r[6]), "=r"(v.r[7])
               : "l"(p));
  return v;
}
__device__ __forceinline__ void st_cs_32(void *p, const Vec32 &v) {
  asm volatile("st.global.cs.v8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};" ::"r"(v.r[0]), "r"(v.r[1]), "r"(v.r[2]),
               "r"(v.r[3]), "r"(v.r[4]), "r"(v.r[5]), "r"(v.r[6]), "r"(v.r[7]), "l"(p)
               : "memory");
}
#endif

}  // namespace tal
