// Staged switching (Sec. 4.4): clean staged chunks move device-to-device into
// their stable-address slots, dirty or missing chunks are reloaded from the
// pinned host copy (App. D: such chunks come from the host copy, never from a staged
// source that may have been overwritten).
//
// The D2D leg is one kernel over the whole plan: the plan is cut into 64 KiB tiles
// and every CTA takes one short contiguous span of tiles (512 KiB), moving each
// tile with four 256-bit loads per thread in flight (128 bytes per thread).  The grid is NOT persistent
// on purpose: staging runs next to KV offload / restore on other streams, and
// short CTAs let the hardware scheduler interleave those kernels instead of
// making them wait for a resident grid to drain.  The host precomputes the plan
// entry each span starts in, so no CTA searches.  The H2D leg runs on an internal
// stream next to the kernel: a handful of host-sourced runs go through the copy
// engine; many of them (thousands of scattered dirty chunks) are read by a second,
// small launch of the same kernel straight from the device-mapped pinned host copy,
// so the host thread is not held for the length of the transfer by thousands of
// copy calls and a restore issued meanwhile shares the link instead of queueing.
#include <algorithm>
#include <cstring>

#include "internal.h"

namespace tal {

struct StageEntry {
  const char *src;  // null: the chunk has no staged copy (always host-sourced)
  const char *src_host;  // device-visible alias of the pinned authoritative copy, or null
  char *dst;
  int64_t bytes;
  int64_t tile0;    // first tile of this entry
  int32_t chunk_id; // bit index into the dirty bitmap, or -1
  int32_t pad;
};

constexpr int kStageThreads = 512;
constexpr int kStageTile = kStageThreads * 128;      // 64 KiB: 128 bytes in flight per thread
constexpr int kSpanTiles = 8;                        // tiles per CTA (512 KiB)

struct StageParams {
  const StageEntry *entries;   // DEVICE [n + 1]; entries[n].tile0 = total tiles
  const int32_t *span_entry;   // DEVICE [spans]: entry that holds the span's first tile
  int64_t n;
  int64_t tiles;
  const uint8_t *dirty;        // DEVICE bitmap or null: which entries are host-sourced this time
  int32_t host_leg;            // 0: copy the clean staged entries; 1: copy the host-sourced ones from src_host
};

// An entry comes from the host when it was never staged or its dirty bit is set; each leg
// leaves the other leg's entries alone.
__device__ __forceinline__ bool stage_skip(const StageParams &p, const StageEntry &e) {
  const bool from_host = !e.src || (p.dirty && e.chunk_id >= 0 && ((p.dirty[e.chunk_id >> 3] >> (e.chunk_id & 7)) & 1));
  return p.host_leg ? !from_host : from_host;
}

// One tile (at most 64 KiB) by the whole CTA: four 256-bit loads per thread in flight when the
// addresses allow, 128-bit or byte accesses otherwise.
__device__ __forceinline__ void copy_tile(const char *src, char *dst, const int64_t len) {
  const int tid = threadIdx.x;
  const uintptr_t low = (uintptr_t)src | (uintptr_t)dst;
  if ((low & 31) == 0 && len == kStageTile) {
    Vec32 v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) v[k] = ld_cs_32(src + ((size_t)tid + k * kStageThreads) * 32);
#pragma unroll
    for (int k = 0; k < 4; ++k) st_cs_32(dst + ((size_t)tid + k * kStageThreads) * 32, v[k]);
  } else if ((low & 15) == 0) {
    const int4 *s4 = (const int4 *)src;
    int4 *d4 = (int4 *)dst;
    if (len == kStageTile) {
      int4 v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = __ldcs(s4 + tid + k * kStageThreads);
#pragma unroll
      for (int k = 0; k < 8; ++k) __stcs(d4 + tid + k * kStageThreads, v[k]);
    } else {
      const int n16 = (int)(len >> 4);
      for (int k = tid; k < n16; k += kStageThreads) __stcs(d4 + k, __ldcs(s4 + k));
      for (int k = (n16 << 4) + tid; k < len; k += kStageThreads) dst[k] = src[k];
    }
  } else {
    for (int k = tid; k < len; k += kStageThreads) dst[k] = src[k];
  }
}

__global__ void __launch_bounds__(kStageThreads) stage_copy_kernel(const __grid_constant__ StageParams p) {
  if (p.host_leg) {
    // Host leg: a small grid walks the ENTRIES (most are skipped with one descriptor read) and a CTA
    // moves a whole host-sourced entry from the mapped pinned copy, tile by tile.
    for (int64_t e = blockIdx.x; e < p.n; e += gridDim.x) {
      const StageEntry cur = p.entries[e];
      if (stage_skip(p, cur)) continue;
      for (int64_t off = 0; off < cur.bytes; off += kStageTile)
        copy_tile(cur.src_host + off, cur.dst + off, min((int64_t)kStageTile, cur.bytes - off));
    }
    return;
  }
  // D2D leg: one CTA per span of tiles
  const int64_t t_begin = (int64_t)blockIdx.x * kSpanTiles;
  const int64_t t_end = min(p.tiles, t_begin + kSpanTiles);
  int64_t e = p.span_entry[blockIdx.x];
  StageEntry cur = p.entries[e];
  int64_t next_tile0 = p.entries[e + 1].tile0;
  bool skip = stage_skip(p, cur);
  for (int64_t t = t_begin; t < t_end; ++t) {
    while (t >= next_tile0) {            // entries with zero tiles are skipped too
      ++e;
      cur = p.entries[e];
      next_tile0 = p.entries[e + 1].tile0;
      skip = stage_skip(p, cur);
    }
    if (skip) continue;
    const int64_t off = (t - cur.tile0) * kStageTile;
    copy_tile(cur.src + off, cur.dst + off, min((int64_t)kStageTile, cur.bytes - off));
  }
}

// Host-sourced runs beyond this count go through the kernel's host leg instead of one
// copy-engine call each; its grid is small because a few CTAs already saturate the host link.
constexpr size_t kReloadKernelMinRuns = 32;
// Measured with 21 GB of scattered 2 MiB reloads (36 % of the chunks dirty): 8 CTAs read 51.4 GB/s
// from pinned memory, as many as 32 do, and a 25,000-token restore issued meanwhile keeps 35 GB/s
// of the link (18 GB/s next to a 16- or 32-CTA reload; 39 GB/s next to 4 CTAs, which however
// no longer hide a 1 % reload under the 18 ms D2D gather).
static int64_t reload_ctas(const talaria_ctx *ctx) { return ctx->cfg.reload_ctas > 0 ? ctx->cfg.reload_ctas : 8; }

struct Range {
  uintptr_t lo, hi;
};

static void sort_ranges(std::vector<Range> &a) {
  // plans are normally written in address order: skip the sort when they already are
  bool sorted = true;
  for (size_t k = 1; k < a.size() && sorted; ++k) sorted = a[k - 1].lo <= a[k].lo;
  if (!sorted) std::sort(a.begin(), a.end(), [](const Range &x, const Range &y) { return x.lo < y.lo; });
}

static bool any_overlap_sorted(std::vector<Range> &a) {
  sort_ranges(a);
  for (size_t k = 1; k < a.size(); ++k)
    if (a[k].lo < a[k - 1].hi) return true;
  return false;
}

// a sorted & disjoint; does any range of b intersect a range of a?
static bool cross_overlap(const std::vector<Range> &a, std::vector<Range> &b) {
  sort_ranges(b);
  size_t i = 0;
  for (const Range &r : b) {
    while (i < a.size() && a[i].hi <= r.lo) ++i;
    // a is sorted and disjoint and b arrives in order of lo, so the first a[i] whose end lies
    // beyond r.lo is the only range of a that can intersect r
    size_t j = i;
    if (j < a.size() && a[j].lo < r.hi && r.lo < a[j].hi) return true;
  }
  return false;
}

// Which entries come from host, byte / chunk counts, and (optionally) the overlap rules.
// Needs no GPU: it is also the body of talaria_check_stage_plan.
static talaria_status_t classify_plan(const talaria_copy_t *plan, int64_t n, const uint8_t *dirty, bool validate,
                                      std::vector<uint8_t> *from_host_out, int64_t *n_clean_out,
                                      talaria_stage_stats_t *st_out) {
  talaria_stage_stats_t st{0, 0, 0, 0};
  std::vector<uint8_t> from_host((size_t)n, 0);
  int64_t n_clean = 0;
  for (int64_t k = 0; k < n; ++k) {
    const talaria_copy_t &c = plan[k];
    if (c.bytes < 0 || !c.dst_dev) return TALARIA_ERR_INVALID_ARG;
    const bool missing = (c.src_dev == nullptr);
    const bool is_dirty = !missing && dirty && c.chunk_id >= 0 && ((dirty[c.chunk_id >> 3] >> (c.chunk_id & 7)) & 1);
    if (missing || is_dirty) {
      if (!c.src_host) return TALARIA_ERR_INVALID_ARG;
      from_host[(size_t)k] = 1;
      st.h2d_bytes += c.bytes;
      if (missing) st.missing_chunks++; else st.dirty_chunks++;
    } else {
      st.d2d_bytes += c.bytes;
      ++n_clean;
    }
  }
  if (validate) {
    std::vector<Range> dsts, srcs;
    dsts.reserve((size_t)n);
    srcs.reserve((size_t)n_clean);
    for (int64_t k = 0; k < n; ++k) {
      if (plan[k].bytes == 0) continue;
      dsts.push_back({(uintptr_t)plan[k].dst_dev, (uintptr_t)plan[k].dst_dev + (uintptr_t)plan[k].bytes});
      if (!from_host[(size_t)k])
        srcs.push_back({(uintptr_t)plan[k].src_dev, (uintptr_t)plan[k].src_dev + (uintptr_t)plan[k].bytes});
    }
    if (any_overlap_sorted(dsts)) return TALARIA_ERR_OVERLAP;
    if (cross_overlap(dsts, srcs)) return TALARIA_ERR_OVERLAP;
  }
  if (from_host_out) from_host_out->swap(from_host);
  if (n_clean_out) *n_clean_out = n_clean;
  if (st_out) *st_out = st;
  return TALARIA_OK;
}

// One merged host-sourced run, as copy-engine copies of bounded size on the reload stream: a
// restore running on the context's other streams gets the link between two pieces.
static talaria_status_t enqueue_reload(talaria_ctx *ctx, const char *h, char *d, int64_t bytes) {
  for (int64_t at = 0; at < bytes; at += kReloadPiece) {
    const size_t n = (size_t)std::min(kReloadPiece, bytes - at);
    TAL_CUDA(ctx, cudaMemcpyAsync(d + at, h + at, n, cudaMemcpyHostToDevice, ctx->reload_stream));
    ctx->counters.memcpy_calls++;
  }
  return TALARIA_OK;
}

// Every destination, and every staged source that will be read, must lie inside one device
// allocation for its whole length.  from_host (nullable): entries whose staged source is not read.
static talaria_status_t check_device_ranges(talaria_ctx *ctx, const talaria_copy_t *plan, int64_t n,
                                            const uint8_t *from_host) {
  if (!ctx->cfg.validate) return TALARIA_OK;
  for (int64_t k = 0; k < n; ++k) {
    if (plan[k].bytes == 0) continue;
    TAL_TRY(require_device_range(ctx, plan[k].dst_dev, plan[k].bytes));
    if (plan[k].src_dev && !(from_host && from_host[k])) TAL_TRY(require_device_range(ctx, plan[k].src_dev, plan[k].bytes));
  }
  return TALARIA_OK;
}

// One leg of a one-shot switch: a compact descriptor (entries, then one int32 per span) is
// built in a slot, uploaded on `stream` and consumed by one launch on `stream`.
struct LegItem {
  const char *src, *src_host;
  char *dst;
  int64_t bytes;
};

static talaria_status_t launch_leg(talaria_ctx *ctx, const std::vector<LegItem> &items, bool host_leg,
                                   cudaStream_t stream) {
  int64_t tiles = 0;
  for (const LegItem &it : items) tiles += (it.bytes + kStageTile - 1) / kStageTile;
  if (tiles == 0) return TALARIA_OK;
  const int64_t spans = (tiles + kSpanTiles - 1) / kSpanTiles;
  if (spans > 0x7fffffffll) return TALARIA_ERR_INVALID_ARG;
  const int64_t m = (int64_t)items.size();
  const size_t ent_bytes = ((size_t)(m + 1) * sizeof(StageEntry) + 15) & ~(size_t)15;
  const size_t desc_bytes = ent_bytes + (size_t)spans * sizeof(int32_t);
  DescSlot *slot;
  TAL_TRY(acquire_slot(ctx, desc_bytes, &slot));
  StageEntry *e = (StageEntry *)slot->h;
  int32_t *span_entry = (int32_t *)(slot->h + ent_bytes);
  int64_t t0 = 0, next_span = 0;
  for (int64_t k = 0; k < m; ++k) {
    const int64_t nt = (items[(size_t)k].bytes + kStageTile - 1) / kStageTile;
    e[k] = StageEntry{items[(size_t)k].src, items[(size_t)k].src_host, items[(size_t)k].dst, items[(size_t)k].bytes, t0, -1, 0};
    // spans whose first tile falls inside this entry
    while (next_span < spans && next_span * kSpanTiles < t0 + nt) span_entry[next_span++] = (int32_t)k;
    t0 += nt;
  }
  e[m] = StageEntry{nullptr, nullptr, nullptr, 0, tiles, -1, 0};
  TAL_TRY(upload_slot(ctx, slot, desc_bytes, stream));
  StageParams p{(const StageEntry *)slot->d, (const int32_t *)(slot->d + ent_bytes), m, tiles, nullptr, host_leg ? 1 : 0};
  const unsigned grid = host_leg ? (unsigned)std::min<int64_t>(m, reload_ctas(ctx)) : (unsigned)spans;
  stage_copy_kernel<<<grid, kStageThreads, 0, stream>>>(p);
  TAL_CUDA(ctx, cudaGetLastError());
  ctx->counters.kernel_launches++;
  return release_slot(ctx, slot, stream);
}

static talaria_status_t stage_impl(talaria_ctx *ctx, const talaria_copy_t *plan, int64_t n,
                                   const uint8_t *dirty, talaria_stage_stats_t *stats, cudaStream_t stream) {
  if (n < 0 || (n > 0 && !plan)) return TALARIA_ERR_INVALID_ARG;
  talaria_stage_stats_t st{0, 0, 0, 0};
  if (n == 0) {
    if (stats) *stats = st;
    return TALARIA_OK;
  }
  std::vector<uint8_t> from_host;
  int64_t n_clean = 0;
  TAL_TRY(classify_plan(plan, n, dirty, ctx->cfg.validate != 0, &from_host, &n_clean, &st));

  // ---- H2D leg, part 1: merge neighbouring host-sourced chunks and check every host
  // source before anything is enqueued, so a rejected plan leaves no partial copy behind.
  std::vector<LegItem> runs;
  HostRangeMemo host_memo;
  for (int64_t k = 0; k < n;) {
    if (!from_host[(size_t)k] || plan[k].bytes == 0) { ++k; continue; }
    LegItem r{nullptr, (const char *)plan[k].src_host, (char *)plan[k].dst_dev, plan[k].bytes};
    int64_t j = k + 1;
    while (j < n && from_host[(size_t)j] && (const char *)plan[j].src_host == r.src_host + r.bytes &&
           (char *)plan[j].dst_dev == r.dst + r.bytes) {
      r.bytes += plan[j].bytes;
      ++j;
    }
    void *alias;
    TAL_TRY(mapped_range(ctx, &host_memo, r.src_host, r.bytes, &alias));
    r.src = (const char *)alias;               // kept beside the host address: the kernel leg reads through it
    runs.push_back(r);
    k = j;
  }
  TAL_TRY(check_device_ranges(ctx, plan, n, from_host.data()));
  // The internal stream forks from the caller's stream BEFORE the D2D kernel is launched, so
  // the host-sourced leg depends only on earlier work and runs next to the kernel.
  const bool forked = !runs.empty();
  if (forked) {
    TAL_CUDA(ctx, cudaEventRecord(ctx->reload_fork, stream));
    TAL_CUDA(ctx, cudaStreamWaitEvent(ctx->reload_stream, ctx->reload_fork, 0));
  }
  // ---- D2D leg ---------------------------------------------------------------
  if (n_clean > 0 && st.d2d_bytes > 0) {
    std::vector<LegItem> clean;
    clean.reserve((size_t)n_clean);
    for (int64_t k = 0; k < n; ++k)
      if (!from_host[(size_t)k]) clean.push_back(LegItem{(const char *)plan[k].src_dev, nullptr, (char *)plan[k].dst_dev, plan[k].bytes});
    if (ctx->timing) cudaEventRecord(ctx->tm[2], stream);
    TAL_TRY(launch_leg(ctx, clean, false, stream));
    if (ctx->timing) { cudaEventRecord(ctx->tm[3], stream); ctx->tm_d2d = true; }
  }
  // ---- H2D leg, part 2: enqueued second, so the kernel is already running meanwhile
  if (forked) {
    if (ctx->timing) cudaEventRecord(ctx->tm[4], ctx->reload_stream);
    if (runs.size() > kReloadKernelMinRuns) {
      std::vector<LegItem> items;
      items.reserve(runs.size());
      for (const LegItem &r : runs) items.push_back(LegItem{nullptr, r.src, r.dst, r.bytes});
      TAL_TRY(launch_leg(ctx, items, true, ctx->reload_stream));
    } else {
      for (const LegItem &r : runs) TAL_TRY(enqueue_reload(ctx, r.src_host, r.dst, r.bytes));
    }
    if (ctx->timing) { cudaEventRecord(ctx->tm[5], ctx->reload_stream); ctx->tm_h2d = true; }
    TAL_CUDA(ctx, cudaEventRecord(ctx->reload_done, ctx->reload_stream));
    TAL_CUDA(ctx, cudaStreamWaitEvent(stream, ctx->reload_done, 0));
  }
  ctx->counters.payload_bytes += st.d2d_bytes + st.h2d_bytes;
  if (stats) *stats = st;
  return TALARIA_OK;
}

}  // namespace tal

// A prepared switch plan: validated once, descriptors resident in device memory.  Running it
// costs one small bitmap upload, one launch and the copy-engine copies of the chunks that are
// dirty or missing this time; nothing is re-planned on the host.
struct talaria_stage_plan {
  std::vector<talaria_copy_t> plan;
  std::vector<uint8_t> host_pinned;   // per entry: its host copy was found pinned when the plan was made
  std::vector<const char *> host_alias;  // ... and its device-visible alias
  char *d_desc = nullptr;        // entries, then one int32 per span
  size_t ent_bytes = 0;
  int64_t tiles = 0, spans = 0, max_chunk = -1;
  static constexpr int kBitmapRing = 4;
  uint8_t *d_dirty = nullptr;    // device copy of the bitmap of the current run
  uint8_t *h_dirty = nullptr;    // pinned staging for it: kBitmapRing buffers used in turn
  size_t bitmap_bytes = 0;
  cudaEvent_t uploaded[kBitmapRing] = {};
  bool busy[kBitmapRing] = {};
  int next = 0;
};

namespace tal {

static void plan_free(talaria_stage_plan *sp) {
  if (!sp) return;
  for (int r = 0; r < talaria_stage_plan::kBitmapRing; ++r) {
    if (sp->busy[r]) cudaEventSynchronize(sp->uploaded[r]);
    if (sp->uploaded[r]) cudaEventDestroy(sp->uploaded[r]);
  }
  if (sp->d_desc) cudaFree(sp->d_desc);
  if (sp->d_dirty) cudaFree(sp->d_dirty);
  if (sp->h_dirty) cudaFreeHost(sp->h_dirty);
  (void)cudaGetLastError();
  delete sp;
}

static talaria_status_t plan_create(talaria_ctx *ctx, const talaria_copy_t *plan, int64_t n, talaria_stage_plan **out) {
  if (!out || n < 0 || (n > 0 && !plan)) return TALARIA_ERR_INVALID_ARG;
  *out = nullptr;
  // validate as if every staged source could be read (whatever the bitmap of a later run says)
  TAL_TRY(classify_plan(plan, n, nullptr, true, nullptr, nullptr, nullptr));
  talaria_stage_plan *sp = new (std::nothrow) talaria_stage_plan();
  if (!sp) return TALARIA_ERR_NO_MEMORY;
  talaria_status_t st = [&]() -> talaria_status_t {
    sp->plan.assign(plan, plan + n);
    sp->host_pinned.assign((size_t)n, 0);
    sp->host_alias.assign((size_t)n, nullptr);
    HostRangeMemo host_memo;
    for (int64_t k = 0; k < n; ++k) {
      sp->tiles += (plan[k].bytes + kStageTile - 1) / kStageTile;
      if (plan[k].chunk_id > sp->max_chunk) sp->max_chunk = plan[k].chunk_id;
      void *alias = nullptr;
      if (plan[k].src_host && mapped_range(ctx, &host_memo, plan[k].src_host, plan[k].bytes, &alias) == TALARIA_OK) {
        sp->host_pinned[(size_t)k] = 1;
        sp->host_alias[(size_t)k] = (const char *)alias;
      }
    }
    TAL_TRY(check_device_ranges(ctx, plan, n, nullptr));
    sp->spans = (sp->tiles + kSpanTiles - 1) / kSpanTiles;
    if (sp->spans > 0x7fffffffll) return TALARIA_ERR_INVALID_ARG;
    sp->ent_bytes = ((size_t)(n + 1) * sizeof(StageEntry) + 15) & ~(size_t)15;
    const size_t desc_bytes = sp->ent_bytes + (size_t)std::max<int64_t>(sp->spans, 1) * sizeof(int32_t);
    std::vector<char> host(desc_bytes);
    StageEntry *e = (StageEntry *)host.data();
    int32_t *span_entry = (int32_t *)(host.data() + sp->ent_bytes);
    int64_t t0 = 0, next_span = 0;
    for (int64_t k = 0; k < n; ++k) {
      const int64_t nt = (plan[k].bytes + kStageTile - 1) / kStageTile;
      e[k] = StageEntry{(const char *)plan[k].src_dev, sp->host_alias[(size_t)k], (char *)plan[k].dst_dev, plan[k].bytes, t0,
                        plan[k].chunk_id, 0};
      while (next_span < sp->spans && next_span * kSpanTiles < t0 + nt) span_entry[next_span++] = (int32_t)k;
      t0 += nt;
    }
    e[n] = StageEntry{nullptr, nullptr, nullptr, 0, sp->tiles, -1, 0};
    TAL_CUDA(ctx, cudaMalloc((void **)&sp->d_desc, desc_bytes));
    TAL_CUDA(ctx, cudaMemcpy(sp->d_desc, host.data(), desc_bytes, cudaMemcpyHostToDevice));
    sp->bitmap_bytes = (size_t)((sp->max_chunk + 8) / 8);
    if (sp->bitmap_bytes) {
      TAL_CUDA(ctx, cudaMalloc((void **)&sp->d_dirty, sp->bitmap_bytes));
      TAL_CUDA(ctx, cudaHostAlloc((void **)&sp->h_dirty, sp->bitmap_bytes * talaria_stage_plan::kBitmapRing,
                                  cudaHostAllocDefault));
    }
    for (int r = 0; r < talaria_stage_plan::kBitmapRing; ++r)
      TAL_CUDA(ctx, cudaEventCreateWithFlags(&sp->uploaded[r], cudaEventDisableTiming));
    return TALARIA_OK;
  }();
  if (st != TALARIA_OK) {
    plan_free(sp);
    return st;
  }
  *out = sp;
  return TALARIA_OK;
}

static talaria_status_t plan_run(talaria_ctx *ctx, talaria_stage_plan *sp, const uint8_t *dirty,
                                 talaria_stage_stats_t *stats, cudaStream_t stream) {
  if (!sp) return TALARIA_ERR_INVALID_ARG;
  const int64_t n = (int64_t)sp->plan.size();
  talaria_stage_stats_t st{0, 0, 0, 0};
  struct HostRun { const char *h; char *d; int64_t bytes; };
  std::vector<HostRun> runs;
  for (int64_t k = 0; k < n; ++k) {
    const talaria_copy_t &c = sp->plan[k];
    const bool missing = (c.src_dev == nullptr);
    const bool is_dirty = !missing && dirty && c.chunk_id >= 0 && ((dirty[c.chunk_id >> 3] >> (c.chunk_id & 7)) & 1);
    if (!(missing || is_dirty)) {
      st.d2d_bytes += c.bytes;
      continue;
    }
    if (!c.src_host) return TALARIA_ERR_INVALID_ARG;
    st.h2d_bytes += c.bytes;
    if (missing) st.missing_chunks++; else st.dirty_chunks++;
    if (c.bytes == 0) continue;
    if (!runs.empty() && runs.back().h + runs.back().bytes == (const char *)c.src_host &&
        runs.back().d + runs.back().bytes == (char *)c.dst_dev) {
      runs.back().bytes += c.bytes;
    } else {
      if (!sp->host_pinned[(size_t)k]) return TALARIA_ERR_HOST_NOT_PINNED;
      runs.push_back(HostRun{(const char *)c.src_host, (char *)c.dst_dev, c.bytes});
    }
  }
  const uint8_t *d_bitmap = nullptr;
  if (dirty && sp->bitmap_bytes) {
    const int r = sp->next;
    sp->next = (sp->next + 1) % talaria_stage_plan::kBitmapRing;
    if (sp->busy[r]) TAL_CUDA(ctx, cudaEventSynchronize(sp->uploaded[r]));   // this pinned buffer is free again
    uint8_t *h = sp->h_dirty + (size_t)r * sp->bitmap_bytes;
    memcpy(h, dirty, sp->bitmap_bytes);
    TAL_CUDA(ctx, cudaMemcpyAsync(sp->d_dirty, h, sp->bitmap_bytes, cudaMemcpyHostToDevice, stream));
    TAL_CUDA(ctx, cudaEventRecord(sp->uploaded[r], stream));            // h may be rewritten after this
    sp->busy[r] = true;
    ctx->counters.memcpy_calls++;
    d_bitmap = sp->d_dirty;
  }
  if (!runs.empty()) {
    TAL_CUDA(ctx, cudaEventRecord(ctx->reload_fork, stream));
    TAL_CUDA(ctx, cudaStreamWaitEvent(ctx->reload_stream, ctx->reload_fork, 0));
  }
  if (sp->tiles > 0 && st.d2d_bytes > 0) {
    StageParams p{(const StageEntry *)sp->d_desc, (const int32_t *)(sp->d_desc + sp->ent_bytes), n, sp->tiles, d_bitmap, 0};
    if (ctx->timing) cudaEventRecord(ctx->tm[2], stream);
    stage_copy_kernel<<<(unsigned)sp->spans, kStageThreads, 0, stream>>>(p);
    TAL_CUDA(ctx, cudaGetLastError());
    if (ctx->timing) { cudaEventRecord(ctx->tm[3], stream); ctx->tm_d2d = true; }
    ctx->counters.kernel_launches++;
  }
  // (the device bitmap is rewritten by the next run's upload, which the caller orders after
  // this kernel: runs of one prepared plan share a stream or are chained with events)
  if (!runs.empty()) {
    if (ctx->timing) cudaEventRecord(ctx->tm[4], ctx->reload_stream);
    if (runs.size() > kReloadKernelMinRuns) {
      // the resident descriptors already name every entry's pinned copy: the same kernel, told to
      // take the host-sourced entries, on a grid small enough to leave the SMs to everyone else
      StageParams p{(const StageEntry *)sp->d_desc, (const int32_t *)(sp->d_desc + sp->ent_bytes), n, sp->tiles, d_bitmap, 1};
      stage_copy_kernel<<<(unsigned)std::min<int64_t>(n, reload_ctas(ctx)), kStageThreads, 0, ctx->reload_stream>>>(p);
      TAL_CUDA(ctx, cudaGetLastError());
      ctx->counters.kernel_launches++;
    } else {
      for (const HostRun &r : runs) TAL_TRY(enqueue_reload(ctx, r.h, r.d, r.bytes));
    }
    if (ctx->timing) { cudaEventRecord(ctx->tm[5], ctx->reload_stream); ctx->tm_h2d = true; }
    TAL_CUDA(ctx, cudaEventRecord(ctx->reload_done, ctx->reload_stream));
    TAL_CUDA(ctx, cudaStreamWaitEvent(stream, ctx->reload_done, 0));
  }
  ctx->counters.payload_bytes += st.d2d_bytes + st.h2d_bytes;
  if (stats) *stats = st;
  return TALARIA_OK;
}

// Pre-staging (Sec. 4.4): authoritative host bytes -> the chunk's place in the staging
// region, for every chunk whose rows are not blocked by a KV allocation.  Copy-engine
// H2D, merged over neighbouring chunks, on the caller's stream.
static talaria_status_t prestage_impl(talaria_ctx *ctx, const talaria_copy_t *plan, int64_t n,
                                      const uint8_t *blocked, uint8_t *staged, uint8_t *dirty,
                                      talaria_stage_stats_t *stats, cudaStream_t stream) {
  if (n < 0 || (n > 0 && !plan)) return TALARIA_ERR_INVALID_ARG;
  talaria_stage_stats_t st{0, 0, 0, 0};
  struct HostRun { const char *h; char *d; int64_t bytes; };
  std::vector<HostRun> runs;
  auto bit = [](const uint8_t *bm, int64_t i) { return (bm[i >> 3] >> (i & 7)) & 1; };
  for (int64_t k = 0; k < n; ++k) {
    const talaria_copy_t &c = plan[k];
    if (c.bytes < 0 || c.chunk_id < 0 || !c.src_dev || !c.src_host) return TALARIA_ERR_INVALID_ARG;
  }
  if (ctx->cfg.validate) {           // staging ranges that are written must not overlap each other
    std::vector<Range> dsts;
    for (int64_t k = 0; k < n; ++k)
      if (plan[k].bytes > 0 && !(blocked && bit(blocked, plan[k].chunk_id)))
        dsts.push_back({(uintptr_t)plan[k].src_dev, (uintptr_t)plan[k].src_dev + (uintptr_t)plan[k].bytes});
    if (any_overlap_sorted(dsts)) return TALARIA_ERR_OVERLAP;
  }
  for (int64_t k = 0; k < n; ++k) {
    const talaria_copy_t &c = plan[k];
    if (blocked && bit(blocked, c.chunk_id)) continue;
    if (c.bytes == 0) continue;
    const char *h = (const char *)c.src_host;
    char *d = (char *)c.src_dev;
    if (!runs.empty() && runs.back().h + runs.back().bytes == h && runs.back().d + runs.back().bytes == d) {
      runs.back().bytes += c.bytes;
    } else {
      runs.push_back(HostRun{h, d, c.bytes});
    }
  }
  HostRangeMemo host_memo;
  for (const HostRun &r : runs) {          // every range is checked before anything is enqueued
    void *alias;
    TAL_TRY(mapped_range(ctx, &host_memo, r.h, r.bytes, &alias));
    TAL_TRY(require_device_range(ctx, r.d, r.bytes));
  }
  for (const HostRun &r : runs) {
    TAL_CUDA(ctx, cudaMemcpyAsync(r.d, r.h, (size_t)r.bytes, cudaMemcpyHostToDevice, stream));
    ctx->counters.memcpy_calls++;
  }
  // bookkeeping only after every copy was accepted
  for (int64_t k = 0; k < n; ++k) {
    const talaria_copy_t &c = plan[k];
    if (blocked && bit(blocked, c.chunk_id)) { st.missing_chunks++; continue; }
    st.h2d_bytes += c.bytes;
    if (staged) staged[c.chunk_id >> 3] |= (uint8_t)(1u << (c.chunk_id & 7));
    if (dirty && bit(dirty, c.chunk_id)) {
      dirty[c.chunk_id >> 3] &= (uint8_t)~(1u << (c.chunk_id & 7));
      st.dirty_chunks++;
    }
  }
  ctx->counters.payload_bytes += st.h2d_bytes;
  if (stats) *stats = st;
  return TALARIA_OK;
}

}  // namespace tal

extern "C" talaria_status_t talaria_prestage(talaria_ctx *ctx, const talaria_copy_t *plan, int64_t n,
                                             const uint8_t *blocked_bitmap, uint8_t *staged_bitmap,
                                             uint8_t *dirty_bitmap, talaria_stage_stats_t *stats,
                                             void *stream) {
  if (!ctx) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(ctx->mu);
  tal::DeviceGuard g(ctx->device);
  if (!g.ok) return TALARIA_ERR_CUDA;
  return tal::prestage_impl(ctx, plan, n, blocked_bitmap, staged_bitmap, dirty_bitmap, stats, (cudaStream_t)stream);
}

extern "C" talaria_status_t talaria_stage_plan_create(talaria_ctx *ctx, const talaria_copy_t *plan, int64_t n,
                                                      talaria_stage_plan **out) {
  if (!ctx) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(ctx->mu);
  tal::DeviceGuard g(ctx->device);
  if (!g.ok) return TALARIA_ERR_CUDA;
  return tal::plan_create(ctx, plan, n, out);
}

extern "C" talaria_status_t talaria_stage_plan_run(talaria_ctx *ctx, talaria_stage_plan *prepared,
                                                   const uint8_t *dirty_bitmap, talaria_stage_stats_t *stats,
                                                   void *stream) {
  if (!ctx) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(ctx->mu);
  tal::DeviceGuard g(ctx->device);
  if (!g.ok) return TALARIA_ERR_CUDA;
  tal::CallTimer timer__(ctx, (cudaStream_t)stream, 3);
  return tal::plan_run(ctx, prepared, dirty_bitmap, stats, (cudaStream_t)stream);
}

extern "C" talaria_status_t talaria_stage_plan_destroy(talaria_ctx *ctx, talaria_stage_plan *prepared) {
  if (!ctx || !prepared) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(ctx->mu);
  tal::DeviceGuard g(ctx->device);
  tal::plan_free(prepared);
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_check_stage_plan(const talaria_copy_t *plan, int64_t n,
                                                     const uint8_t *dirty_bitmap, talaria_stage_stats_t *stats) {
  if (n < 0 || (n > 0 && !plan)) return TALARIA_ERR_INVALID_ARG;
  return tal::classify_plan(plan, n, dirty_bitmap, true, nullptr, nullptr, stats);
}

extern "C" int64_t talaria_mark_dirty(const talaria_copy_t *plan, int64_t n, const void *alloc_base,
                                      int64_t alloc_bytes, const uint8_t *staged_bitmap,
                                      uint8_t *dirty_bitmap) {
  if (!plan || n <= 0 || !dirty_bitmap || alloc_bytes <= 0) return 0;
  const uintptr_t a0 = (uintptr_t)alloc_base, a1 = a0 + (uintptr_t)alloc_bytes;
  int64_t changed = 0;
  for (int64_t k = 0; k < n; ++k) {
    const talaria_copy_t &c = plan[k];
    if (c.bytes <= 0 || c.chunk_id < 0 || !c.src_dev) continue;
    const int64_t id = c.chunk_id;
    if (staged_bitmap && !((staged_bitmap[id >> 3] >> (id & 7)) & 1)) continue;
    const uintptr_t s0 = (uintptr_t)c.src_dev, s1 = s0 + (uintptr_t)c.bytes;
    if (s0 < a1 && a0 < s1 && !((dirty_bitmap[id >> 3] >> (id & 7)) & 1)) {
      dirty_bitmap[id >> 3] |= (uint8_t)(1u << (id & 7));
      ++changed;
    }
  }
  return changed;
}

extern "C" talaria_status_t talaria_stage(talaria_ctx *ctx, const talaria_copy_t *plan, int64_t n,
                                          const uint8_t *dirty_bitmap, talaria_stage_stats_t *stats,
                                          void *stream) {
  if (!ctx) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(ctx->mu);
  tal::DeviceGuard g(ctx->device);
  if (!g.ok) return TALARIA_ERR_CUDA;
  tal::CallTimer timer__(ctx, (cudaStream_t)stream, 3);
  return tal::stage_impl(ctx, plan, n, dirty_bitmap, stats, (cudaStream_t)stream);
}
