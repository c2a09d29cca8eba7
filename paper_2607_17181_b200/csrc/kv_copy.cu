// Block-table copies between the paged KV pool and an image of logical blocks:
// KV offload (pool -> pinned host), KV restore (pinned host -> new pool blocks)
// and the in-HBM gather / scatter (Sec. 4.3; App. C layer-first / page-first).
//
// One kernel serves every case.  The image is enumerated in ITS OWN memory order
// (fastest-varying dimension first), so the image side of the copy is a single
// sequential stream -- full 128-byte lines on the host link -- while the pool side
// jumps from chunk to chunk as the block table says.  Each warp moves 4 KiB per
// step, every lane keeping 128 bytes in flight (four 256-bit or eight 128-bit accesses).
#include <algorithm>
#include <cstring>

#include "internal.h"

namespace tal {

struct ImgOrder {
  // linear chunk index w = (d2*e1 + d1)*e0 + d0, dimension 0 innermost in the image
  int64_t e0, e1;
  int32_t pos_l, pos_p, pos_i;  // which digit (0,1,2) holds layer / plane / block (host use)
  int32_t lp_coef[3];           // plane index l*P + p = sum_k d_k * lp_coef[k]
  int32_t i_coef[3];            // logical block i   = sum_k d_k * i_coef[k]
};

struct KvCopyParams {
  const void *const *plane_base;  // DEVICE [L*P]
  const int32_t *table;           // DEVICE [n], already offset to first_block
  char *img;                      // image base as seen from the device
  const int64_t *page_off;        // DEVICE [n] or null: extra image offset per logical block
  int64_t sd[3];                  // image stride of digit 0, 1, 2 (bytes)
  int64_t chunk_bytes;
  int64_t w0, w1;                 // chunks [w0, w1) of the image order
  int64_t num_blocks;             // pool capacity: a table entry outside [0, num_blocks) is skipped
  volatile unsigned int *status;  // device-visible pinned word, set to 1 when an entry was skipped
  ImgOrder ord;
};

constexpr int kPart = 4096;       // bytes one warp moves per step (vector path)

__device__ __forceinline__ void decode_chunk(const KvCopyParams &p, int64_t w, int64_t &lp, int64_t &i,
                                             int64_t &img_off) {
  const int64_t t = w / p.ord.e0;
  const int64_t d0 = w - t * p.ord.e0;
  const int64_t d2 = t / p.ord.e1;
  const int64_t d1 = t - d2 * p.ord.e1;
  lp = d0 * p.ord.lp_coef[0] + d1 * p.ord.lp_coef[1] + d2 * p.ord.lp_coef[2];
  i = d0 * p.ord.i_coef[0] + d1 * p.ord.i_coef[1] + d2 * p.ord.i_coef[2];
  img_off = d0 * p.sd[0] + d1 * p.sd[1] + d2 * p.sd[2];
  if (p.page_off) img_off += p.page_off[i];
}

// TO_IMAGE: pool -> image (offload / gather); else image -> pool (restore / scatter).
// VB: bytes per access (16 or 32); every lane keeps 128 bytes in flight per step.
template <bool TO_IMAGE, int VB>
__device__ __forceinline__ void kv_copy_vec_body(const KvCopyParams &p) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const int64_t parts = (p.chunk_bytes + kPart - 1) / kPart;
  const int64_t units = (p.w1 - p.w0) * parts;
  for (int64_t u = warp; u < units; u += nwarps) {
    int64_t c = u / parts;
    int64_t part = u - c * parts;
    int64_t lp, i, img_off;
    decode_chunk(p, p.w0 + c, lp, i, img_off);
    int64_t blk = p.table[i];
    if ((unsigned long long)blk >= (unsigned long long)p.num_blocks) {
      // never touch memory outside the pool, even when host-side validation was switched off
      if (lane == 0) *p.status = 1u;
      continue;
    }
    char *pool = (char *)p.plane_base[lp] + blk * p.chunk_bytes + part * kPart;
    char *img = p.img + img_off + part * kPart;
    const char *src = TO_IMAGE ? pool : img;
    char *dst = TO_IMAGE ? img : pool;
    int64_t left = p.chunk_bytes - part * kPart;
    if (left >= kPart) {
      if (VB == 32) {
        Vec32 v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) v[k] = ld_cs_32(src + (lane + k * 32) * 32);
#pragma unroll
        for (int k = 0; k < 4; ++k) st_cs_32(dst + (lane + k * 32) * 32, v[k]);
      } else {
        int4 v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = __ldcs((const int4 *)src + lane + k * 32);
#pragma unroll
        for (int k = 0; k < 8; ++k) __stcs((int4 *)dst + lane + k * 32, v[k]);
      }
    } else {
      int n16 = (int)(left >> 4);
      for (int k = lane; k < n16; k += 32) __stcs((int4 *)dst + k, __ldcs((const int4 *)src + k));
    }
  }
}

template <bool TO_IMAGE, int VB>
__global__ void __launch_bounds__(512) kv_copy_vec_kernel(const __grid_constant__ KvCopyParams p) {
  kv_copy_vec_body<TO_IMAGE, VB>(p);
}

// Transfers of a few blocks carry their whole descriptor in the kernel parameters: plane
// addresses, table slice and (for page slabs or fused sessions) per-block offsets.  Nothing is
// uploaded and no descriptor slot is taken, which is most of the fixed cost of a small copy.
constexpr int kInlinePlanes = 256;
constexpr int kInlineBlocks = 256;
struct KvCopyInline {
  KvCopyParams p;                       // plane_base / table / page_off are filled in by the kernel
  const void *planes[kInlinePlanes];
  int64_t page_off[kInlineBlocks];
  int32_t table[kInlineBlocks];
  int32_t has_page_off;
};

template <bool TO_IMAGE, int VB>
__global__ void __launch_bounds__(512) kv_copy_vec_inline_kernel(const __grid_constant__ KvCopyInline q) {
  KvCopyParams p = q.p;
  p.plane_base = q.planes;
  p.table = q.table;
  p.page_off = q.has_page_off ? q.page_off : nullptr;
  kv_copy_vec_body<TO_IMAGE, VB>(p);
}

// Any chunk size / alignment: plain byte copies (odd shapes only).
template <bool TO_IMAGE>
__global__ void __launch_bounds__(256) kv_copy_byte_kernel(const __grid_constant__ KvCopyParams p) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t c = warp; c < p.w1 - p.w0; c += nwarps) {
    int64_t lp, i, img_off;
    decode_chunk(p, p.w0 + c, lp, i, img_off);
    int64_t blk = p.table[i];
    if ((unsigned long long)blk >= (unsigned long long)p.num_blocks) {
      if (lane == 0) *p.status = 1u;
      continue;
    }
    char *pool = (char *)p.plane_base[lp] + blk * p.chunk_bytes;
    char *img = p.img + img_off;
    const char *src = TO_IMAGE ? pool : img;
    char *dst = TO_IMAGE ? img : pool;
    for (int64_t k = lane; k < p.chunk_bytes; k += 32) dst[k] = src[k];
  }
}

// ---------------------------------------------------------------------------

struct Dim {
  int64_t extent, stride;
  int which;  // 0 layer, 1 plane, 2 block
};

struct Plan {
  int64_t L, P, n, C, chunks;
  ImgOrder ord;
  int64_t run_chunks;  // chunks that are contiguous in the image, aligned in w
  int vec;             // widest usable access: 32, 16, or 0 (byte path)
};

// Shape and stride checks, image order, contiguous run length, widest usable access.
// need_planes = false skips everything that needs the plane addresses (host-only check).
static talaria_status_t make_plan(const talaria_kv_layout_t *kv, int64_t n, const void *img,
                                  const talaria_host_layout_t *hl, Plan *out, bool need_planes = true) {
  if (kv->num_layers <= 0 || kv->num_kv_heads <= 0 || kv->block_tokens <= 0 || kv->head_dim <= 0 ||
      kv->elt_bytes <= 0 || kv->num_planes <= 0 || kv->num_blocks <= 0 || (need_planes && !kv->plane_base))
    return TALARIA_ERR_INVALID_ARG;
  Plan pl{};
  pl.L = kv->num_layers;
  pl.P = kv->num_planes;
  pl.n = n;
  pl.C = (int64_t)kv->num_kv_heads * kv->block_tokens * kv->head_dim * kv->elt_bytes;
  pl.chunks = pl.L * pl.P * n;
  if (hl->stride_layer < 0 || hl->stride_plane < 0 || hl->stride_block < 0 || hl->capacity_bytes < 0)
    return TALARIA_ERR_INVALID_ARG;
  Dim d[3] = {{pl.L, hl->stride_layer, 0}, {pl.P, hl->stride_plane, 1}, {n, hl->stride_block, 2}};
  // innermost first; dimensions of extent 1 have no meaningful stride: keep them innermost
  std::stable_sort(d, d + 3, [](const Dim &a, const Dim &b) {
    bool a1 = a.extent == 1, b1 = b.extent == 1;
    if (a1 != b1) return a1;
    if (a1 && b1) return false;
    return a.stride < b.stride;
  });
  // the three dimensions must nest without overlap
  int64_t span = pl.C;
  for (int k = 0; k < 3; ++k) {
    if (d[k].extent == 1) continue;
    if (d[k].stride < span) return TALARIA_ERR_INVALID_ARG;
    span = d[k].stride * (d[k].extent - 1) + span;
  }
  if (span > hl->capacity_bytes) return TALARIA_ERR_EXTENT;
  pl.ord.e0 = d[0].extent;
  pl.ord.e1 = d[1].extent;
  for (int k = 0; k < 3; ++k) {
    pl.ord.lp_coef[k] = 0;
    pl.ord.i_coef[k] = 0;
    if (d[k].which == 0) { pl.ord.pos_l = k; pl.ord.lp_coef[k] = (int32_t)pl.P; }
    if (d[k].which == 1) { pl.ord.pos_p = k; pl.ord.lp_coef[k] = 1; }
    if (d[k].which == 2) { pl.ord.pos_i = k; pl.ord.i_coef[k] = 1; }
  }
  int64_t run = 1, bytes = pl.C;
  for (int k = 0; k < 3; ++k) {
    if (d[k].extent != 1 && d[k].stride != bytes) break;
    run *= d[k].extent;
    bytes *= d[k].extent;
  }
  pl.run_chunks = run;
  uintptr_t bits = (uintptr_t)pl.C | (uintptr_t)img;    // low bits of everything an address is built from
  for (int k = 0; k < 3; ++k)
    if (d[k].extent != 1) bits |= (uintptr_t)d[k].stride;
  for (int64_t k = 0; need_planes && k < pl.L * pl.P; ++k) {
    if (!kv->plane_base[k]) return TALARIA_ERR_INVALID_ARG;
    bits |= (uintptr_t)kv->plane_base[k];
  }
  pl.vec = (bits % 32 == 0) ? 32 : (bits % 16 == 0) ? 16 : 0;
  *out = pl;
  return TALARIA_OK;
}

static int64_t image_offset(const Plan &pl, const talaria_host_layout_t *hl, int64_t w) {
  int64_t d[3];
  int64_t t = w / pl.ord.e0;
  d[0] = w - t * pl.ord.e0;
  d[2] = t / pl.ord.e1;
  d[1] = t - d[2] * pl.ord.e1;
  return d[pl.ord.pos_l] * hl->stride_layer + d[pl.ord.pos_p] * hl->stride_plane +
         d[pl.ord.pos_i] * hl->stride_block;
}

static talaria_status_t check_table(const int32_t *bt, int64_t n, int64_t num_blocks, bool reject_dups,
                                    std::vector<uint64_t> *bits) {
  for (int64_t i = 0; i < n; ++i)
    if (bt[i] < 0 || (int64_t)bt[i] >= num_blocks) return TALARIA_ERR_BAD_BLOCK_ID;
  if (reject_dups) {
    bits->assign((size_t)((num_blocks + 63) / 64), 0);
    for (int64_t i = 0; i < n; ++i) {
      const uint64_t bit = 1ull << (bt[i] & 63);
      uint64_t &w = (*bits)[(size_t)bt[i] >> 6];
      if (w & bit) return TALARIA_ERR_DUP_BLOCK;
      w |= bit;
    }
  }
  return TALARIA_OK;
}

static talaria_status_t validate_table(talaria_ctx *ctx, const talaria_kv_layout_t *kv, const int32_t *bt,
                                       int64_t n, bool reject_dups) {
  if (!ctx->cfg.validate) return TALARIA_OK;
  return check_table(bt, n, kv->num_blocks, reject_dups, &ctx->dup_bits);
}

// Every plane must hold num_blocks chunks inside one device allocation.
static talaria_status_t check_planes(talaria_ctx *ctx, const talaria_kv_layout_t *kv, const Plan &pl) {
  for (int64_t k = 0; k < pl.L * pl.P; ++k)
    TAL_TRY(require_device_range(ctx, kv->plane_base[k], kv->num_blocks * pl.C));
  return TALARIA_OK;
}

// vec: access width the addresses allow (0 = byte path); img_bits: low bits of the image base in use.
template <bool TO_IMAGE>
static talaria_status_t launch_copy(talaria_ctx *ctx, const KvCopyParams &p, int vec, int64_t grid_cap,
                                    cudaStream_t stream) {
  if (p.w1 <= p.w0) return TALARIA_OK;
  if ((uintptr_t)p.img % 32 != 0 && vec == 32) vec = 16;
  if ((uintptr_t)p.img % 16 != 0) vec = 0;
  if (vec) {
    const int threads = 512;
    int64_t parts = (p.chunk_bytes + kPart - 1) / kPart;
    int64_t warps = (p.w1 - p.w0) * parts;
    int64_t need = (warps + threads / 32 - 1) / (threads / 32);
    int grid = (int)std::max<int64_t>(1, std::min<int64_t>(need, grid_cap));
    if (vec == 32) kv_copy_vec_kernel<TO_IMAGE, 32><<<grid, threads, 0, stream>>>(p);
    else           kv_copy_vec_kernel<TO_IMAGE, 16><<<grid, threads, 0, stream>>>(p);
  } else {
    const int threads = 256;
    int64_t need = ((p.w1 - p.w0) + threads / 32 - 1) / (threads / 32);
    int grid = (int)std::max<int64_t>(1, std::min<int64_t>(need, std::min<int64_t>(grid_cap, 1 << 20)));
    kv_copy_byte_kernel<TO_IMAGE><<<grid, threads, 0, stream>>>(p);
  }
  TAL_CUDA(ctx, cudaGetLastError());
  ctx->counters.kernel_launches++;
  return TALARIA_OK;
}

// The same launch with the descriptor in the kernel parameters.  planes: L*P device addresses (host
// array); table: n ids; page_off: n offsets or null.  Needs vec != 0 and the inline limits.
static talaria_status_t launch_inline(talaria_ctx *ctx, bool to_image, const KvCopyParams &p, int vec,
                                      int64_t grid_cap, const void *const *planes, int64_t n_planes,
                                      const int32_t *table, const int64_t *page_off, int64_t n,
                                      cudaStream_t stream) {
  if (p.w1 <= p.w0) return TALARIA_OK;
  KvCopyInline q{};
  q.p = p;
  memcpy(q.planes, planes, (size_t)n_planes * sizeof(void *));
  memcpy(q.table, table, (size_t)n * sizeof(int32_t));
  if (page_off) memcpy(q.page_off, page_off, (size_t)n * sizeof(int64_t));
  q.has_page_off = page_off ? 1 : 0;
  if ((uintptr_t)p.img % 32 != 0 && vec == 32) vec = 16;
  const int threads = 512;
  const int64_t parts = (p.chunk_bytes + kPart - 1) / kPart;
  const int64_t warps = (p.w1 - p.w0) * parts;
  const int64_t need = (warps + threads / 32 - 1) / (threads / 32);
  const int grid = (int)std::max<int64_t>(1, std::min<int64_t>(need, grid_cap));
  if (to_image) {
    if (vec == 32) kv_copy_vec_inline_kernel<true, 32><<<grid, threads, 0, stream>>>(q);
    else           kv_copy_vec_inline_kernel<true, 16><<<grid, threads, 0, stream>>>(q);
  } else {
    if (vec == 32) kv_copy_vec_inline_kernel<false, 32><<<grid, threads, 0, stream>>>(q);
    else           kv_copy_vec_inline_kernel<false, 16><<<grid, threads, 0, stream>>>(q);
  }
  TAL_CUDA(ctx, cudaGetLastError());
  ctx->counters.kernel_launches++;
  return TALARIA_OK;
}

static bool fits_inline(int64_t n_planes, int64_t n, int vec, const void *img) {
  return n_planes <= kInlinePlanes && n <= kInlineBlocks && vec != 0 && (uintptr_t)img % 16 == 0;
}

static talaria_status_t launch_dir(talaria_ctx *ctx, bool to_image, const KvCopyParams &p, int vec,
                                   int64_t grid_cap, cudaStream_t stream) {
  return to_image ? launch_copy<true>(ctx, p, vec, grid_cap, stream)
                  : launch_copy<false>(ctx, p, vec, grid_cap, stream);
}

static void set_image_strides(KvCopyParams &p, const ImgOrder &o, int64_t sL, int64_t sP, int64_t sI) {
  p.sd[o.pos_l] = sL;
  p.sd[o.pos_p] = sP;
  p.sd[o.pos_i] = sI;
}

// Zero-copy kernels are bound by the host link: 8 CTAs already saturate it, 32 leave headroom
// and keep 100+ SMs free for whatever else is running.
static int64_t zc_grid(const talaria_ctx *ctx) { return ctx->cfg.zc_ctas > 0 ? ctx->cfg.zc_ctas : 32; }
// Pack / unpack kernels of the bounce variant only have to stay ahead of a 56 GB/s copy engine;
// a small grid does that with a 20x margin and barely disturbs concurrent kernels.
static int64_t pack_grid(const talaria_ctx *ctx) { return ctx->cfg.pack_ctas > 0 ? ctx->cfg.pack_ctas : 64; }
// In-HBM gather / scatter: one short CTA per 16 warps of work, scheduled by the hardware.
static int64_t full_grid() { return 0x7fffffff; }

// Number of runs of adjacent ids in a table (bt[i+1] == bt[i]+1 continues a run).
static int64_t count_id_runs(const int32_t *bt, int64_t n) {
  int64_t runs = n > 0 ? 1 : 0;
  for (int64_t i = 1; i < n; ++i)
    if (bt[i] != bt[i - 1] + 1) ++runs;
  return runs;
}

// How a host-side transfer crosses the link.  Measured at the Qwen3-235B shape: below 8 MB of
// payload the zero-copy kernel and the bounce pipeline are within noise of each other (80 us for
// one 3.1 MB block) and the kernel needs no bounce buffer; from 8 MB up the copy engine behind
// the pack kernel is 6-7 % faster (55.3-56.1 vs 51.4-52.7 GB/s at 4.81 GB); one copy per run of
// adjacent ids only pays for tables of few, long runs (13x slower on random tables).
static int choose_variant(const talaria_ctx *ctx, const Plan &pl, const talaria_host_layout_t *hl,
                          const int32_t *bt, int64_t n, bool to_image) {
  const BounceLane &ln = ctx->lane[to_image ? 0 : 1];
  const int64_t payload = pl.chunks * pl.C;
  const int64_t dma_min = ctx->cfg.dma_min_bytes > 0 ? ctx->cfg.dma_min_bytes : (8ll << 20);
  const int64_t seg_bytes = pl.run_chunks * pl.C;
  const bool bounce_ok = (int64_t)ln.half >= pl.C;
  int variant = ctx->cfg.variant;
  if (variant == TALARIA_VARIANT_AUTO) {
    variant = TALARIA_VARIANT_ZEROCOPY;
    if (bounce_ok && payload >= dma_min && seg_bytes >= (256 << 10)) variant = TALARIA_VARIANT_BOUNCE;
    // a table of few long runs of adjacent ids needs no kernel at all
    if (payload >= dma_min && (hl->stride_block == pl.C || n == 1)) {
      const int64_t copies = pl.L * pl.P * count_id_runs(bt, n);
      if (copies <= 1024 && payload / copies >= (1 << 20)) variant = TALARIA_VARIANT_RUNS;
    }
  }
  if (variant == TALARIA_VARIANT_BOUNCE && !bounce_ok) variant = TALARIA_VARIANT_ZEROCOPY;
  return variant;
}

// to_image: offload / gather; img_on_device: the image is device memory (gather / scatter).
static talaria_status_t kv_transfer(talaria_ctx *ctx, const talaria_kv_layout_t *kv, const int32_t *table,
                                    int64_t first, int64_t n, void *img, const talaria_host_layout_t *hl,
                                    cudaStream_t stream, bool to_image, bool img_on_device) {
  if (!kv || !hl || first < 0 || n < 0) return TALARIA_ERR_INVALID_ARG;
  if (n == 0) return TALARIA_OK;
  if (!table || !img) return TALARIA_ERR_INVALID_ARG;
  Plan pl;
  TAL_TRY(make_plan(kv, n, img, hl, &pl));
  const int32_t *bt = table + first;
  TAL_TRY(validate_table(ctx, kv, bt, n, /*reject_dups=*/!to_image));

  TAL_TRY(check_planes(ctx, kv, pl));
  void *img_dev = img;
  if (img_on_device) {
    TAL_TRY(require_device_range(ctx, img, hl->capacity_bytes));
  } else {
    TAL_TRY(mapped_range(ctx, img, hl->capacity_bytes, &img_dev));
    if (((uintptr_t)img_dev) % 16 != 0) pl.vec = 0;
  }

  KvCopyParams p{};
  p.num_blocks = kv->num_blocks;
  p.status = ctx->status_dev;
  p.chunk_bytes = pl.C;
  p.ord = pl.ord;
  const int64_t payload = pl.chunks * pl.C;
  ctx->counters.payload_bytes += payload;

  int variant = TALARIA_VARIANT_ZEROCOPY;     // gather / scatter: the copy kernel on a full grid
  if (!img_on_device) {
    variant = choose_variant(ctx, pl, hl, bt, n, to_image);
    ctx->counters.last_variant = variant;
  }

  if (variant == TALARIA_VARIANT_ZEROCOPY) {
    p.img = (char *)img_dev;
    set_image_strides(p, pl.ord, hl->stride_layer, hl->stride_plane, hl->stride_block);
    p.w0 = 0; p.w1 = pl.chunks;
    const int64_t grid_cap = img_on_device ? full_grid() : zc_grid(ctx);
    if (fits_inline(pl.L * pl.P, n, pl.vec, p.img))
      return launch_inline(ctx, to_image, p, pl.vec, grid_cap, kv->plane_base, pl.L * pl.P, bt, nullptr, n, stream);
  }

  // descriptor: plane pointers, then the table slice
  const size_t ptr_bytes = (size_t)(pl.L * pl.P) * sizeof(void *);
  const size_t desc_bytes = ptr_bytes + (size_t)n * sizeof(int32_t);
  DescSlot *slot = nullptr;
  if (variant != TALARIA_VARIANT_RUNS) {
    TAL_TRY(acquire_slot(ctx, desc_bytes, &slot));
    memcpy(slot->h, kv->plane_base, ptr_bytes);
    memcpy(slot->h + ptr_bytes, bt, (size_t)n * sizeof(int32_t));
    TAL_TRY(upload_slot(ctx, slot, desc_bytes, stream));
    p.plane_base = (const void *const *)slot->d;
    p.table = (const int32_t *)(slot->d + ptr_bytes);
  }

  if (variant == TALARIA_VARIANT_ZEROCOPY) {
    TAL_TRY(launch_dir(ctx, to_image, p, pl.vec, img_on_device ? full_grid() : zc_grid(ctx), stream));
    return release_slot(ctx, slot, stream);
  }
  BounceLane &ln = ctx->lane[to_image ? 0 : 1];

  if (variant == TALARIA_VARIANT_RUNS) {
    // one copy-engine copy per (layer, plane, run of adjacent ids); needs no descriptor
    const bool blocks_contig = (hl->stride_block == pl.C) || n == 1;
    for (int64_t l = 0; l < pl.L; ++l)
      for (int64_t q = 0; q < pl.P; ++q) {
        char *plane = (char *)kv->plane_base[l * pl.P + q];
        int64_t i = 0;
        while (i < n) {
          int64_t j = i + 1;
          if (blocks_contig)
            while (j < n && bt[j] == bt[j - 1] + 1) ++j;
          char *h = (char *)img + l * hl->stride_layer + q * hl->stride_plane + i * hl->stride_block;
          char *d = plane + (int64_t)bt[i] * pl.C;
          size_t bytes = (size_t)((j - i) * pl.C);
          if (to_image) TAL_CUDA(ctx, cudaMemcpyAsync(h, d, bytes, cudaMemcpyDeviceToHost, stream));
          else          TAL_CUDA(ctx, cudaMemcpyAsync(d, h, bytes, cudaMemcpyHostToDevice, stream));
          ctx->counters.memcpy_calls++;
          i = j;
        }
      }
    return TALARIA_OK;
  }

  // ---- bounce: kernel <-> device bounce half <-> large copy-engine copies ----
  // The bounce half holds a piece of the image in image order, densely packed.
  int64_t piece = (int64_t)ln.half / pl.C;                     // chunks per piece
  if (pl.run_chunks < piece) piece = (piece / pl.run_chunks) * pl.run_chunks;
  // dense image strides of the bounce copy: offset(w) = w*C
  p.sd[0] = pl.C;
  p.sd[1] = p.sd[0] * pl.ord.e0;
  p.sd[2] = p.sd[1] * pl.ord.e1;

  TAL_CUDA(ctx, cudaEventRecord(ln.fork, stream));
  for (int j = 0; j < 2; ++j) TAL_CUDA(ctx, cudaStreamWaitEvent(ln.s[j], ln.fork, 0));
  int k = 0;
  for (int64_t w0 = 0; w0 < pl.chunks; w0 += piece, ++k) {
    const int64_t w1 = std::min(pl.chunks, w0 + piece);
    const int j = k & 1;
    char *half = ln.buf + (size_t)j * ln.half;
    p.img = half - w0 * pl.C;   // so that offset(w) lands at (w - w0)*C inside the half
    p.w0 = w0; p.w1 = w1;
    if (to_image) TAL_TRY(launch_dir(ctx, true, p, pl.vec, pack_grid(ctx), ln.s[j]));
    for (int64_t ws = w0; ws < w1;) {
      int64_t we = std::min(w1, (ws / pl.run_chunks + 1) * pl.run_chunks);
      char *h = (char *)img + image_offset(pl, hl, ws);
      char *d = half + (ws - w0) * pl.C;
      size_t bytes = (size_t)((we - ws) * pl.C);
      if (to_image) TAL_CUDA(ctx, cudaMemcpyAsync(h, d, bytes, cudaMemcpyDeviceToHost, ln.s[j]));
      else          TAL_CUDA(ctx, cudaMemcpyAsync(d, h, bytes, cudaMemcpyHostToDevice, ln.s[j]));
      ctx->counters.memcpy_calls++;
      ws = we;
    }
    if (!to_image) TAL_TRY(launch_dir(ctx, false, p, pl.vec, pack_grid(ctx), ln.s[j]));
  }
  for (int j = 0; j < 2; ++j) {
    TAL_CUDA(ctx, cudaEventRecord(ln.done[j], ln.s[j]));
    TAL_CUDA(ctx, cudaStreamWaitEvent(stream, ln.done[j], 0));
  }
  return release_slot(ctx, slot, stream);
}


// ---------------------------------------------------------------------------
// Page-first registry slabs (App. C): logical block i is one slab of L*P*C bytes,
// fragments ordered [layer][plane], at byte offset page_off[i] of a pinned host pool.
// Zero-copy: the copy kernel with one extra offset per block.  Bounce: the dense
// page-first bounce half is filled / drained by one copy-engine copy per run of
// adjacent slabs.
static talaria_status_t kv_transfer_pages(talaria_ctx *ctx, const talaria_kv_layout_t *kv, const int32_t *table,
                                          int64_t first, int64_t n, void *host_pool, int64_t pool_bytes,
                                          const int64_t *page_off, cudaStream_t stream, bool to_image) {
  if (!kv || first < 0 || n < 0 || pool_bytes < 0) return TALARIA_ERR_INVALID_ARG;
  if (n == 0) return TALARIA_OK;
  if (!table || !host_pool || !page_off) return TALARIA_ERR_INVALID_ARG;
  // a one-block page-first image gives the plan its shape checks and alignment
  talaria_host_layout_t one{};
  Plan pl;
  {
    const int64_t C0 = (int64_t)kv->num_kv_heads * kv->block_tokens * kv->head_dim * kv->elt_bytes;
    one.stride_plane = C0;
    one.stride_layer = (int64_t)kv->num_planes * C0;
    one.stride_block = (int64_t)kv->num_layers * kv->num_planes * C0;
    one.capacity_bytes = one.stride_block;
    TAL_TRY(make_plan(kv, 1, host_pool, &one, &pl));
  }
  const int64_t C = pl.C, L = pl.L, P = pl.P, slab = L * P * C;
  const int32_t *bt = table + first;
  TAL_TRY(validate_table(ctx, kv, bt, n, /*reject_dups=*/!to_image));
  uintptr_t bits = 0;
  for (int64_t i = 0; i < n; ++i) {
    if (page_off[i] < 0 || page_off[i] + slab > pool_bytes) return TALARIA_ERR_EXTENT;
    bits |= (uintptr_t)page_off[i];
  }
  if (ctx->cfg.validate && to_image) {       // two blocks written into the same slab bytes: order-dependent
    std::vector<int64_t> sorted(page_off, page_off + n);
    std::sort(sorted.begin(), sorted.end());
    for (int64_t i = 1; i < n; ++i)
      if (sorted[i] < sorted[i - 1] + slab) return TALARIA_ERR_OVERLAP;
  }
  int vec = pl.vec;
  if (bits % 32 != 0 && vec == 32) vec = 16;
  if (bits % 16 != 0) vec = 0;
  TAL_TRY(check_planes(ctx, kv, pl));
  void *pool_dev;
  TAL_TRY(mapped_range(ctx, host_pool, pool_bytes, &pool_dev));

  const size_t ptr_bytes = (size_t)(L * P) * sizeof(void *);
  const size_t off_bytes = (size_t)n * sizeof(int64_t);
  const size_t desc_bytes = ptr_bytes + off_bytes + (size_t)n * sizeof(int32_t);
  const int64_t payload = n * slab;
  ctx->counters.payload_bytes += payload;

  KvCopyParams p{};
  p.num_blocks = kv->num_blocks;
  p.status = ctx->status_dev;
  p.chunk_bytes = C;
  // digits: plane, layer, block -- the order of bytes inside consecutive slabs
  p.ord.e0 = P; p.ord.e1 = L;
  p.ord.lp_coef[0] = 1; p.ord.lp_coef[1] = (int32_t)P; p.ord.lp_coef[2] = 0;
  p.ord.i_coef[0] = 0; p.ord.i_coef[1] = 0; p.ord.i_coef[2] = 1;
  p.sd[0] = C; p.sd[1] = P * C;

  BounceLane &ln = ctx->lane[to_image ? 0 : 1];
  const int64_t dma_min = ctx->cfg.dma_min_bytes > 0 ? ctx->cfg.dma_min_bytes : (8ll << 20);
  int variant = ctx->cfg.variant;
  const bool bounce_ok = vec != 0 && (int64_t)ln.half >= slab;
  if (variant == TALARIA_VARIANT_AUTO || variant == TALARIA_VARIANT_RUNS) {
    // Measured: for scattered 3 MB slabs the zero-copy kernel (52.7 / 51.5 GB/s) beats one
    // copy-engine copy per slab (51.9 / 51.2); the copy engine only wins once adjacent slabs
    // merge into transfers of 16 MiB and more.
    int64_t runs = 1;
    for (int64_t i = 1; i < n; ++i)
      if (page_off[i] != page_off[i - 1] + slab) ++runs;
    variant = (bounce_ok && payload >= dma_min && payload / runs >= (16ll << 20)) ? TALARIA_VARIANT_BOUNCE
                                                                                   : TALARIA_VARIANT_ZEROCOPY;
  }
  if (variant == TALARIA_VARIANT_BOUNCE && !bounce_ok) variant = TALARIA_VARIANT_ZEROCOPY;
  ctx->counters.last_variant = variant;

  if (variant == TALARIA_VARIANT_ZEROCOPY && fits_inline(L * P, n, vec, pool_dev)) {
    p.img = (char *)pool_dev;
    p.sd[2] = 0;                              // the block's place comes from its page offset
    p.w0 = 0; p.w1 = n * L * P;
    return launch_inline(ctx, to_image, p, vec, zc_grid(ctx), kv->plane_base, L * P, bt, page_off, n, stream);
  }
  DescSlot *slot;
  TAL_TRY(acquire_slot(ctx, desc_bytes, &slot));
  memcpy(slot->h, kv->plane_base, ptr_bytes);
  memcpy(slot->h + ptr_bytes, page_off, off_bytes);
  memcpy(slot->h + ptr_bytes + off_bytes, bt, (size_t)n * sizeof(int32_t));
  TAL_TRY(upload_slot(ctx, slot, desc_bytes, stream));
  p.plane_base = (const void *const *)slot->d;
  p.table = (const int32_t *)(slot->d + ptr_bytes + off_bytes);

  if (variant == TALARIA_VARIANT_ZEROCOPY) {
    p.img = (char *)pool_dev;
    p.page_off = (const int64_t *)(slot->d + ptr_bytes);
    p.sd[2] = 0;                              // the block's place comes from its page offset
    p.w0 = 0; p.w1 = n * L * P;
    TAL_TRY(launch_dir(ctx, to_image, p, vec, zc_grid(ctx), stream));
    return release_slot(ctx, slot, stream);
  }

  const int64_t piece = (int64_t)ln.half / slab;          // blocks per bounce half
  p.page_off = nullptr;
  p.sd[2] = slab;
  TAL_CUDA(ctx, cudaEventRecord(ln.fork, stream));
  for (int j = 0; j < 2; ++j) TAL_CUDA(ctx, cudaStreamWaitEvent(ln.s[j], ln.fork, 0));
  int k = 0;
  for (int64_t i0 = 0; i0 < n; i0 += piece, ++k) {
    const int64_t i1 = std::min(n, i0 + piece);
    const int j = k & 1;
    char *half = ln.buf + (size_t)j * ln.half;
    p.img = half - i0 * slab;
    p.w0 = i0 * L * P; p.w1 = i1 * L * P;
    if (to_image) TAL_TRY(launch_dir(ctx, true, p, vec, pack_grid(ctx), ln.s[j]));
    for (int64_t a = i0; a < i1;) {
      int64_t b = a + 1;
      while (b < i1 && page_off[b] == page_off[b - 1] + slab) ++b;
      char *h = (char *)host_pool + page_off[a];
      char *d = half + (a - i0) * slab;
      const size_t bytes = (size_t)((b - a) * slab);
      if (to_image) TAL_CUDA(ctx, cudaMemcpyAsync(h, d, bytes, cudaMemcpyDeviceToHost, ln.s[j]));
      else          TAL_CUDA(ctx, cudaMemcpyAsync(d, h, bytes, cudaMemcpyHostToDevice, ln.s[j]));
      ctx->counters.memcpy_calls++;
      a = b;
    }
    if (!to_image) TAL_TRY(launch_dir(ctx, false, p, vec, pack_grid(ctx), ln.s[j]));
  }
  for (int j = 0; j < 2; ++j) {
    TAL_CUDA(ctx, cudaEventRecord(ln.done[j], ln.s[j]));
    TAL_CUDA(ctx, cudaStreamWaitEvent(stream, ln.done[j], 0));
  }
  return release_slot(ctx, slot, stream);
}

// ---------------------------------------------------------------------------
// Layer-ordered restore (App. C: the layer-first view is the one the attention kernels'
// device-side KV layout follows): the image is brought in layer by
// layer, whatever its host layout, and an event per layer tells a consumer
// (prefill of that layer) that the layer's K and V are in the pool.  Copy-engine
// transfers (1-D or pitched 2-D, one per layer and piece) land in a bounce half;
// the unpack kernel scatters it; the two halves alternate on two internal streams.
static talaria_status_t kv_restore_layered(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                           const int32_t *table, int64_t first, int64_t n, const void *img,
                                           const talaria_host_layout_t *hl, void *const *layer_events,
                                           cudaStream_t stream) {
  if (!kv || !hl || first < 0 || n < 0 || !layer_events) return TALARIA_ERR_INVALID_ARG;
  if (kv->num_layers <= 0) return TALARIA_ERR_INVALID_ARG;
  for (int32_t l = 0; l < kv->num_layers; ++l)
    if (!layer_events[l]) return TALARIA_ERR_INVALID_ARG;
  auto record_all = [&]() -> talaria_status_t {
    for (int32_t l = 0; l < kv->num_layers; ++l) TAL_CUDA(ctx, cudaEventRecord((cudaEvent_t)layer_events[l], stream));
    return TALARIA_OK;
  };
  if (n == 0) return record_all();
  if (!table || !img) return TALARIA_ERR_INVALID_ARG;
  Plan pl;
  TAL_TRY(make_plan(kv, n, img, hl, &pl));
  BounceLane &ln = ctx->lane[1];
  const int64_t C = pl.C, P = pl.P, L = pl.L;
  const int64_t sL = hl->stride_layer, sP = hl->stride_plane, sI = hl->stride_block;
  const int64_t payload = pl.chunks * C, dma_min = ctx->cfg.dma_min_bytes > 0 ? ctx->cfg.dma_min_bytes : (8ll << 20);
  const int64_t max_pitch = 1ll << 30;
  // rows the copy engine can move: planes adjacent (a row per block) or blocks adjacent (a row per plane)
  const bool rows_by_block = (P == 1 || sP == C);
  const bool rows_by_plane = !rows_by_block && (n == 1 || sI == C);
  const bool dma_ok = pl.vec != 0 && (int64_t)ln.half >= P * C && (rows_by_block || rows_by_plane) &&
                      sI < max_pitch && sP < max_pitch && ctx->cfg.variant != TALARIA_VARIANT_ZEROCOPY &&
                      (payload >= dma_min || ctx->cfg.variant == TALARIA_VARIANT_BOUNCE);
  if (!dma_ok) {
    // small or oddly laid out images: the ordinary restore, then every layer is ready at once
    TAL_TRY(kv_transfer(ctx, kv, table, first, n, (void *)img, hl, stream, false, false));
    return record_all();
  }
  const int32_t *bt = table + first;
  TAL_TRY(validate_table(ctx, kv, bt, n, /*reject_dups=*/true));
  TAL_TRY(check_planes(ctx, kv, pl));
  void *alias;
  TAL_TRY(mapped_range(ctx, img, hl->capacity_bytes, &alias));

  const size_t ptr_bytes = (size_t)(L * P) * sizeof(void *);
  const size_t desc_bytes = ptr_bytes + (size_t)n * sizeof(int32_t);
  DescSlot *slot;
  TAL_TRY(acquire_slot(ctx, desc_bytes, &slot));
  memcpy(slot->h, kv->plane_base, ptr_bytes);
  memcpy(slot->h + ptr_bytes, bt, (size_t)n * sizeof(int32_t));
  TAL_TRY(upload_slot(ctx, slot, desc_bytes, stream));
  ctx->counters.payload_bytes += payload;
  ctx->counters.last_variant = TALARIA_VARIANT_BOUNCE;

  // pieces: whole layers while a layer fits a bounce half, else block ranges of one layer
  const int64_t layer_bytes = P * n * C;
  const int64_t layers_per_piece = std::max<int64_t>(1, (int64_t)ln.half / layer_bytes);
  const int64_t blocks_per_piece = layer_bytes <= (int64_t)ln.half ? n : std::max<int64_t>(1, (int64_t)ln.half / (P * C));

  TAL_CUDA(ctx, cudaEventRecord(ln.fork, stream));
  for (int j = 0; j < 2; ++j) TAL_CUDA(ctx, cudaStreamWaitEvent(ln.s[j], ln.fork, 0));
  int k = 0;
  for (int64_t l0 = 0; l0 < L;) {
    const int64_t l1 = (blocks_per_piece == n) ? std::min(L, l0 + layers_per_piece) : l0 + 1;
    for (int64_t i0 = 0; i0 < n; i0 += blocks_per_piece, ++k) {
      const int64_t i1 = std::min(n, i0 + blocks_per_piece), nn = i1 - i0, LL = l1 - l0;
      const int j = k & 1;
      char *half = ln.buf + (size_t)j * ln.half;
      // host -> bounce half, one transfer per layer
      for (int64_t l = l0; l < l1; ++l) {
        const char *src = (const char *)img + l * sL + i0 * sI;
        char *dst = half + (l - l0) * P * nn * C;
        if (rows_by_block) {
          if (nn == 1 || sI == P * C) {
            TAL_CUDA(ctx, cudaMemcpyAsync(dst, src, (size_t)(nn * P * C), cudaMemcpyHostToDevice, ln.s[j]));
          } else {
            TAL_CUDA(ctx, cudaMemcpy2DAsync(dst, (size_t)(P * C), src, (size_t)sI, (size_t)(P * C), (size_t)nn,
                                            cudaMemcpyHostToDevice, ln.s[j]));
          }
        } else {
          if (P == 1 || sP == nn * C) {
            TAL_CUDA(ctx, cudaMemcpyAsync(dst, src, (size_t)(P * nn * C), cudaMemcpyHostToDevice, ln.s[j]));
          } else {
            TAL_CUDA(ctx, cudaMemcpy2DAsync(dst, (size_t)(nn * C), src, (size_t)sP, (size_t)(nn * C), (size_t)P,
                                            cudaMemcpyHostToDevice, ln.s[j]));
          }
        }
        ctx->counters.memcpy_calls++;
      }
      // bounce half -> pool: the half holds [layer][block][plane] or [layer][plane][block]
      KvCopyParams p{};
      p.num_blocks = kv->num_blocks;
      p.status = ctx->status_dev;
      p.plane_base = (const void *const *)slot->d + l0 * P;
      p.table = (const int32_t *)(slot->d + ptr_bytes) + i0;
      p.chunk_bytes = C;
      p.img = half;
      p.w0 = 0;
      p.w1 = LL * P * nn;
      if (rows_by_block) {        // digits: plane, block, layer
        p.ord.e0 = P; p.ord.e1 = nn;
        p.ord.lp_coef[0] = 1; p.ord.lp_coef[1] = 0; p.ord.lp_coef[2] = (int32_t)P;
        p.ord.i_coef[0] = 0; p.ord.i_coef[1] = 1; p.ord.i_coef[2] = 0;
        p.sd[0] = C; p.sd[1] = P * C; p.sd[2] = nn * P * C;
      } else {                    // digits: block, plane, layer
        p.ord.e0 = nn; p.ord.e1 = P;
        p.ord.lp_coef[0] = 0; p.ord.lp_coef[1] = 1; p.ord.lp_coef[2] = (int32_t)P;
        p.ord.i_coef[0] = 1; p.ord.i_coef[1] = 0; p.ord.i_coef[2] = 0;
        p.sd[0] = C; p.sd[1] = nn * C; p.sd[2] = P * nn * C;
      }
      TAL_TRY(launch_dir(ctx, false, p, pl.vec, pack_grid(ctx), ln.s[j]));
      TAL_CUDA(ctx, cudaEventRecord(ln.done[j], ln.s[j]));
      if (i1 == n) {
        // the layers of this piece are complete once the other half's earlier pieces are too
        if (blocks_per_piece != n && k > 0) TAL_CUDA(ctx, cudaStreamWaitEvent(ln.s[j], ln.done[1 - j], 0));
        for (int64_t l = l0; l < l1; ++l) TAL_CUDA(ctx, cudaEventRecord((cudaEvent_t)layer_events[l], ln.s[j]));
      }
    }
    l0 = l1;
  }
  for (int j = 0; j < 2; ++j) {
    TAL_CUDA(ctx, cudaEventRecord(ln.done[j], ln.s[j]));
    TAL_CUDA(ctx, cudaStreamWaitEvent(stream, ln.done[j], 0));
  }
  return release_slot(ctx, slot, stream);
}

}  // namespace tal

using namespace tal;

#define TAL_ENTER(ctx)                                   \
  if (!(ctx)) return TALARIA_ERR_INVALID_ARG;            \
  std::lock_guard<std::mutex> lk__((ctx)->mu);           \
  DeviceGuard guard__((ctx)->device);                    \
  if (!guard__.ok) return TALARIA_ERR_CUDA

extern "C" talaria_status_t talaria_check_block_table(const int32_t *block_table, int64_t n, int64_t num_blocks,
                                                      int32_t reject_duplicates) {
  if (n < 0 || num_blocks <= 0 || (n > 0 && !block_table)) return TALARIA_ERR_INVALID_ARG;
  std::vector<uint64_t> bits;
  return check_table(block_table, n, num_blocks, reject_duplicates != 0, &bits);
}

extern "C" talaria_status_t talaria_check_image_layout(const talaria_kv_layout_t *kv, int64_t n_blocks,
                                                       const talaria_host_layout_t *hl,
                                                       int64_t *contiguous_run_bytes) {
  if (!kv || !hl || n_blocks < 0) return TALARIA_ERR_INVALID_ARG;
  if (n_blocks == 0) {
    if (contiguous_run_bytes) *contiguous_run_bytes = 0;
    return TALARIA_OK;
  }
  Plan pl;
  TAL_TRY(make_plan(kv, n_blocks, nullptr, hl, &pl, /*need_planes=*/false));
  if (contiguous_run_bytes) *contiguous_run_bytes = pl.run_chunks * pl.C;
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_kv_offload(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                               const int32_t *block_table, int64_t first_block,
                                               int64_t n_blocks, void *host_dst,
                                               const talaria_host_layout_t *hl, void *stream) {
  TAL_ENTER(ctx);
  CallTimer timer__(ctx, (cudaStream_t)stream, 1);
  return kv_transfer(ctx, kv, block_table, first_block, n_blocks, host_dst, hl, (cudaStream_t)stream, true, false);
}

extern "C" talaria_status_t talaria_kv_restore(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                               const int32_t *new_block_table, int64_t first_block,
                                               int64_t n_blocks, const void *host_src,
                                               const talaria_host_layout_t *hl, void *stream) {
  TAL_ENTER(ctx);
  CallTimer timer__(ctx, (cudaStream_t)stream, 2);
  return kv_transfer(ctx, kv, new_block_table, first_block, n_blocks, (void *)host_src, hl,
                     (cudaStream_t)stream, false, false);
}

extern "C" talaria_status_t talaria_kv_restore_layered(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                                       const int32_t *new_block_table, int64_t first_block,
                                                       int64_t n_blocks, const void *host_src,
                                                       const talaria_host_layout_t *hl,
                                                       void *const *layer_events, void *stream) {
  TAL_ENTER(ctx);
  CallTimer timer__(ctx, (cudaStream_t)stream, 2);
  return kv_restore_layered(ctx, kv, new_block_table, first_block, n_blocks, host_src, hl, layer_events,
                            (cudaStream_t)stream);
}

extern "C" talaria_status_t talaria_kv_offload_pages(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                                     const int32_t *block_table, int64_t first_block,
                                                     int64_t n_blocks, void *host_pool, int64_t pool_bytes,
                                                     const int64_t *page_offsets, void *stream) {
  TAL_ENTER(ctx);
  CallTimer timer__(ctx, (cudaStream_t)stream, 1);
  return kv_transfer_pages(ctx, kv, block_table, first_block, n_blocks, host_pool, pool_bytes, page_offsets,
                           (cudaStream_t)stream, true);
}

extern "C" talaria_status_t talaria_kv_restore_pages(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                                     const int32_t *new_block_table, int64_t first_block,
                                                     int64_t n_blocks, const void *host_pool, int64_t pool_bytes,
                                                     const int64_t *page_offsets, void *stream) {
  TAL_ENTER(ctx);
  CallTimer timer__(ctx, (cudaStream_t)stream, 2);
  return kv_transfer_pages(ctx, kv, new_block_table, first_block, n_blocks, (void *)host_pool, pool_bytes,
                           page_offsets, (cudaStream_t)stream, false);
}

extern "C" talaria_status_t talaria_kv_gather(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                              const int32_t *block_table, int64_t first_block,
                                              int64_t n_blocks, void *d_image,
                                              const talaria_host_layout_t *il, void *stream) {
  TAL_ENTER(ctx);
  return kv_transfer(ctx, kv, block_table, first_block, n_blocks, d_image, il, (cudaStream_t)stream, true, true);
}

extern "C" talaria_status_t talaria_kv_scatter(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                               const int32_t *new_block_table, int64_t first_block,
                                               int64_t n_blocks, const void *d_image,
                                               const talaria_host_layout_t *il, void *stream) {
  TAL_ENTER(ctx);
  return kv_transfer(ctx, kv, new_block_table, first_block, n_blocks, (void *)d_image, il,
                     (cudaStream_t)stream, false, true);
}

// Restore tables of different sessions must not share a block either.
static talaria_status_t batch_dup_check(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                        const talaria_kv_xfer_t *x, int32_t n) {
  if (!ctx->cfg.validate || !kv || kv->num_blocks <= 0) return TALARIA_OK;
  std::vector<uint64_t> bits((size_t)((kv->num_blocks + 63) / 64), 0);
  for (int32_t s = 0; s < n; ++s) {
    if (x[s].n_blocks < 0 || x[s].first_block < 0) return TALARIA_ERR_INVALID_ARG;
    if (x[s].n_blocks == 0) continue;
    if (!x[s].block_table) return TALARIA_ERR_INVALID_ARG;
    for (int64_t i = 0; i < x[s].n_blocks; ++i) {
      int32_t b = x[s].block_table[x[s].first_block + i];
      if (b < 0 || b >= kv->num_blocks) return TALARIA_ERR_BAD_BLOCK_ID;
      uint64_t bit = 1ull << (b & 63);
      if (bits[(size_t)b >> 6] & bit) return TALARIA_ERR_DUP_BLOCK;
      bits[(size_t)b >> 6] |= bit;
    }
  }
  return TALARIA_OK;
}

// Several sessions in one call.  Sessions that would each run the zero-copy kernel (the small
// ones) and share their layer and plane strides are fused into ONE launch: the kernel sees
// one image whose logical blocks are all the sessions' blocks back to back, each block
// carrying the byte offset of its place in its own session's image -- the page-slab form of
// the copy kernel.  Everything else (copy-engine variants, odd shapes) is enqueued in turn.
// All arguments are checked before the first launch.
static talaria_status_t kv_batch(talaria_ctx *ctx, const talaria_kv_layout_t *kv, const talaria_kv_xfer_t *x,
                                 int32_t n_x, cudaStream_t stream, bool to_image) {
  if (n_x < 0 || (n_x > 0 && !x) || !kv) return TALARIA_ERR_INVALID_ARG;
  struct Member { int32_t s; Plan pl; char *img_dev; };
  std::vector<Member> fuse;
  std::vector<int32_t> solo;
  for (int32_t s = 0; s < n_x; ++s) {
    const talaria_kv_xfer_t &t = x[s];
    if (t.n_blocks < 0 || t.first_block < 0) return TALARIA_ERR_INVALID_ARG;
    if (t.n_blocks == 0) continue;
    if (!t.block_table || !t.host) return TALARIA_ERR_INVALID_ARG;
    Plan pl;
    TAL_TRY(make_plan(kv, t.n_blocks, t.host, &t.hl, &pl));
    const int32_t *bt = t.block_table + t.first_block;
    TAL_TRY(validate_table(ctx, kv, bt, t.n_blocks, /*reject_dups=*/!to_image));
    TAL_TRY(check_planes(ctx, kv, pl));
    void *img_dev = nullptr;
    TAL_TRY(mapped_range(ctx, t.host, t.hl.capacity_bytes, &img_dev));
    const bool vec_ok = pl.vec != 0 && (uintptr_t)img_dev % 16 == 0;
    if (vec_ok && choose_variant(ctx, pl, &t.hl, bt, t.n_blocks, to_image) == TALARIA_VARIANT_ZEROCOPY)
      fuse.push_back(Member{s, pl, (char *)img_dev});
    else
      solo.push_back(s);
  }
  // ---- fused groups: members with equal (stride_layer, stride_plane) ------------------
  std::vector<char> done(fuse.size(), 0);
  std::vector<int64_t> page_off;
  std::vector<int32_t> table;
  for (size_t a = 0; a < fuse.size(); ++a) {
    if (done[a]) continue;
    const talaria_host_layout_t &ha = x[fuse[a].s].hl;
    const Plan &pa = fuse[a].pl;
    // a dimension of extent 1 has no meaningful stride: compare only what addresses use
    auto same = [&](const talaria_host_layout_t &h) {
      return (pa.L == 1 || h.stride_layer == ha.stride_layer) && (pa.P == 1 || h.stride_plane == ha.stride_plane);
    };
    char *base = fuse[a].img_dev;
    int vec = 32;
    for (size_t b = a; b < fuse.size(); ++b)
      if (!done[b] && same(x[fuse[b].s].hl)) base = std::min(base, fuse[b].img_dev);
    page_off.clear();
    table.clear();
    int32_t members = 0;
    for (size_t b = a; b < fuse.size(); ++b) {
      if (done[b] || !same(x[fuse[b].s].hl)) continue;
      done[b] = 1;
      ++members;
      const talaria_kv_xfer_t &t = x[fuse[b].s];
      vec = std::min(vec, fuse[b].pl.vec);
      if ((uintptr_t)fuse[b].img_dev % 32 != 0) vec = std::min(vec, 16);
      for (int64_t i = 0; i < t.n_blocks; ++i) {
        page_off.push_back((int64_t)(fuse[b].img_dev - base) + i * t.hl.stride_block);
        table.push_back(t.block_table[t.first_block + i]);
      }
    }
    const int64_t n = (int64_t)table.size(), L = pa.L, P = pa.P, C = pa.C;
    KvCopyParams p{};
    p.num_blocks = kv->num_blocks;
    p.status = ctx->status_dev;
    p.chunk_bytes = C;
    p.img = base;
    // digits: plane, layer, block -- the block's place comes from its offset
    p.ord.e0 = P; p.ord.e1 = L;
    p.ord.lp_coef[0] = 1; p.ord.lp_coef[1] = (int32_t)P; p.ord.lp_coef[2] = 0;
    p.ord.i_coef[0] = 0; p.ord.i_coef[1] = 0; p.ord.i_coef[2] = 1;
    p.sd[0] = P == 1 ? 0 : ha.stride_plane; p.sd[1] = L == 1 ? 0 : ha.stride_layer; p.sd[2] = 0;
    p.w0 = 0; p.w1 = n * L * P;
    ctx->counters.payload_bytes += n * L * P * C;
    ctx->counters.last_variant = TALARIA_VARIANT_ZEROCOPY;
    if (fits_inline(L * P, n, vec, base)) {
      TAL_TRY(launch_inline(ctx, to_image, p, vec, zc_grid(ctx), kv->plane_base, L * P, table.data(), page_off.data(), n, stream));
      continue;
    }
    const size_t ptr_bytes = (size_t)(L * P) * sizeof(void *), off_bytes = (size_t)n * sizeof(int64_t);
    const size_t desc_bytes = ptr_bytes + off_bytes + (size_t)n * sizeof(int32_t);
    DescSlot *slot;
    TAL_TRY(acquire_slot(ctx, desc_bytes, &slot));
    memcpy(slot->h, kv->plane_base, ptr_bytes);
    memcpy(slot->h + ptr_bytes, page_off.data(), off_bytes);
    memcpy(slot->h + ptr_bytes + off_bytes, table.data(), (size_t)n * sizeof(int32_t));
    TAL_TRY(upload_slot(ctx, slot, desc_bytes, stream));
    p.plane_base = (const void *const *)slot->d;
    p.page_off = (const int64_t *)(slot->d + ptr_bytes);
    p.table = (const int32_t *)(slot->d + ptr_bytes + off_bytes);
    TAL_TRY(launch_dir(ctx, to_image, p, vec, zc_grid(ctx), stream));
    TAL_TRY(release_slot(ctx, slot, stream));
    (void)members;
  }
  // ---- the rest, one after the other ------------------------------------------------------
  for (int32_t s : solo)
    TAL_TRY(kv_transfer(ctx, kv, x[s].block_table, x[s].first_block, x[s].n_blocks, x[s].host, &x[s].hl, stream,
                        to_image, false));
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_kv_offload_batch(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                                     const talaria_kv_xfer_t *xfers, int32_t n_xfers,
                                                     void *stream) {
  TAL_ENTER(ctx);
  CallTimer timer__(ctx, (cudaStream_t)stream, 1);
  return kv_batch(ctx, kv, xfers, n_xfers, (cudaStream_t)stream, true);
}

extern "C" talaria_status_t talaria_kv_restore_batch(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                                     const talaria_kv_xfer_t *xfers, int32_t n_xfers,
                                                     void *stream) {
  TAL_ENTER(ctx);
  CallTimer timer__(ctx, (cudaStream_t)stream, 2);
  if (n_xfers < 0 || (n_xfers > 0 && !xfers)) return TALARIA_ERR_INVALID_ARG;
  TAL_TRY(batch_dup_check(ctx, kv, xfers, n_xfers));
  return kv_batch(ctx, kv, xfers, n_xfers, (cudaStream_t)stream, false);
}
