/*
 * talaria.h -- C ABI of the instance-local KV substrate hot path.
 *
 * Four operations from the Talaria paper's memory substrate (Sec. 3.5, 4.3, 4.4):
 *   (1) chained block hashing and prefix matching of a continuation against a
 *       stored session stream,
 *   (2) KV offload: gather of a session's paged KV blocks from the HBM pool
 *       into pinned host memory (the host KV registry's checkpoint),
 *   (3) KV restore: scatter from pinned host memory into newly allocated pool
 *       blocks,
 *   (4) D2D staging: copy of staged weight / KV chunks into stable-address
 *       slots, with dirty or missing chunks reloaded from the host copy.
 *
 * General rules
 *   - Every function returns a talaria_status_t (0 = OK, negative = error).
 *     No exceptions, no aborts, no device traps.  Arguments are validated on
 *     the host before any launch, so a bad table never reaches the GPU.  Extents
 *     are checked the same way: a host image (its declared capacity_bytes), a
 *     pinned pool, every pool plane (num_blocks chunks) and every stage source
 *     and destination must lie, for their whole length, inside the one pinned or
 *     device allocation that holds their first byte (the driver is asked once per
 *     allocation; ranges registered through talaria_host_register are known
 *     exactly).  A range that runs off its allocation is TALARIA_ERR_EXTENT and
 *     nothing is launched.  validate = 0 switches the table, plan and extent
 *     checks off.
 *   - Ownership: the caller owns all memory named in the arguments (pool,
 *     host images, token arrays, tables, staging region, slots).  The library
 *     owns only its context: small descriptor buffers, a device bounce buffer
 *     for the copy-engine variant, internal streams and events.
 *   - "HOST" / "DEVICE" beside a pointer says where it must live.  Host arrays
 *     of tables, offsets and plans are copied before the call returns.
 *   - Work is enqueued on the caller's CUDA stream (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream) and is asynchronous unless
 *     noted.  Completion = talaria_sync() or any stream/event wait.
 *   - A context serialises its own calls with a mutex; two calls that overlap
 *     on the GPU must not touch the same bytes.
 *   - GPU: sm_100a only.  There is no CPU fallback.
 */
#ifndef TALARIA_H_
#define TALARIA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t talaria_status_t;
enum {
  TALARIA_OK = 0,
  TALARIA_ERR_INVALID_ARG = -1,     /* null pointer, negative size, bad shape or strides  */
  TALARIA_ERR_BAD_BLOCK_ID = -2,    /* table entry < 0 or >= num_blocks                   */
  TALARIA_ERR_DUP_BLOCK = -3,       /* duplicate id in a restore/scatter table            */
  TALARIA_ERR_HOST_NOT_PINNED = -4, /* host buffer is not page-locked / device-mapped     */
  TALARIA_ERR_EXTENT = -5,          /* image or buffer smaller than the strides require   */
  TALARIA_ERR_OVERLAP = -6,         /* stage plan: destinations overlap each other or a   */
                                    /* source that is read                                */
  TALARIA_ERR_CUDA = -7,            /* a CUDA call failed: see talaria_last_cuda_error    */
  TALARIA_ERR_NO_MEMORY = -9        /* host or device allocation for the context failed   */
};

/* How offload / restore cross the host link. */
enum {
  TALARIA_VARIANT_AUTO = 0,     /* chosen per transfer size from the measured crossover        */
  TALARIA_VARIANT_ZEROCOPY = 1, /* one kernel reads/writes device-mapped pinned memory         */
  TALARIA_VARIANT_BOUNCE = 2,   /* gather kernel -> device bounce -> large copy-engine copies, */
                                /* double-buffered on two internal streams                     */
  TALARIA_VARIANT_RUNS = 3      /* one copy-engine copy per run of adjacent block ids          */
};

typedef struct talaria_ctx talaria_ctx;

typedef struct {
  int64_t bounce_bytes;   /* device bounce buffer PER DIRECTION (two halves); 0 = 128 MiB     */
  int64_t dma_min_bytes;  /* AUTO: payloads >= this use BOUNCE; 0 = built-in measured value   */
  int32_t variant;        /* TALARIA_VARIANT_*; overridden by env TALARIA_VARIANT=1|2|3       */
  int32_t validate;       /* 0 = skip host-side table / plan validation; default 1            */
  int32_t zc_ctas;        /* grid size of zero-copy kernels; 0 = built-in (leaves SMs free)   */
  int32_t pack_ctas;      /* grid size of the bounce variant's pack / unpack kernels; 0 = 64  */
  int64_t host_match_bytes; /* staging (pinned + device, allocated once at create) of            */
                            /* talaria_prefix_match_host; 0 = 16 MiB, at least 1 MiB             */
  int32_t reload_ctas;      /* grid of the staged switch's host-reload kernel; 0 = built-in.     */
                            /* Fewer CTAs leave more of the host link to a concurrent restore.   */
  int32_t reserved;
} talaria_config_t;

/* Device-side paged KV pool (Sec. 4.3; descriptor fields of App. C "Attention-layout
 * metadata": page size, dtype width, slab shape).  Plane (l, p) is one layer's K
 * (p = 0) or V (p = 1) tensor laid out [num_blocks, kv_heads, block_tokens, head_dim];
 * a "chunk" is one block of one plane: kv_heads*block_tokens*head_dim*elt_bytes
 * contiguous bytes.  The addresses are stable for the life of the pool. */
typedef struct {
  int32_t num_layers, num_kv_heads, block_tokens, head_dim, elt_bytes;
  int32_t num_planes;        /* 2 = paired K/V slabs (MHA); 1 = one latent slab (MLA)        */
  int64_t num_blocks;        /* pool capacity per plane                                      */
  void *const *plane_base;   /* HOST array [num_layers*num_planes] of DEVICE pointers        */
} talaria_kv_layout_t;

/* Image of n logical blocks outside the pool (App. C "Layer-first and page-first
 * movement").  Chunk (l, p, i) lives at byte offset l*stride_layer + p*stride_plane
 * + i*stride_block.  Layer-first: stride_block = C, stride_plane = n*C, stride_layer
 * = planes*n*C.  Page-first: stride_plane = C, stride_layer = planes*C, stride_block
 * = layers*planes*C.  Padded variants are allowed as long as the three dimensions
 * nest without overlap; every stride and the image base must be 16-byte aligned
 * unless the chunk size itself is not a multiple of 16. */
typedef struct {
  int64_t stride_layer, stride_plane, stride_block; /* bytes */
  int64_t capacity_bytes;                           /* size of the image buffer */
} talaria_host_layout_t;

/* Result of matching one continuation against one stored stream (App. A "Prefix
 * reuse"; Sec. 4.3 blocks keyed by cumulative prefix hash). */
typedef struct {
  int64_t lcp_tokens;          /* token-level longest common prefix                          */
  int64_t matched_blocks;      /* leading full blocks whose chained hashes are equal         */
  int64_t reusable_tokens;     /* block_tokens * min(matched_blocks, lcp_tokens/block_tokens)*/
  int32_t hash_token_disagree; /* 1 if hashes and tokens disagree on the block count         */
  int32_t reserved;
} talaria_match_t;

/* One entry of a staged-switch copy plan (Sec. 4.4). */
typedef struct {
  const void *src_dev;   /* DEVICE staged copy of the chunk; NULL = chunk was never staged   */
  const void *src_host;  /* HOST (pinned) authoritative copy; may be NULL if never needed    */
  void *dst_dev;         /* DEVICE stable-address slot                                       */
  int64_t bytes;
  int32_t chunk_id;      /* bit index into the dirty bitmap; < 0 = never dirty               */
  int32_t reserved;
} talaria_copy_t;

/* App. D "Path classification": staged-byte coverage and dirty bytes of a switch. */
typedef struct {
  int64_t d2d_bytes, h2d_bytes, dirty_chunks, missing_chunks;
} talaria_stage_stats_t;

/* App. D "Path classification" also records the D2D and H2D gather times of a switch, and the
 * router charges a measured restore cost (Sec. 3.3): optional per-call timing from CUDA events
 * on the streams the work runs on.  op: 1 offload, 2 restore, 3 stage, 4 prefix match from host
 * memory (the _host and _resident forms: first copy to last kernel); the leg fields that do
 * not apply are 0.  For a stage, d2d_ms is the gather kernel and h2d_ms the host reloads, which
 * overlap, so total_ms is less than their sum. */
typedef struct {
  float total_ms;           /* from the call's first to its last piece of work on `stream`   */
  float d2d_ms, h2d_ms, d2h_ms;
  int32_t op;
  int32_t reserved;
} talaria_timing_t;

typedef struct {
  int64_t kernel_launches;  /* kernels of this library launched since create / reset         */
  int64_t memcpy_calls;     /* copy-engine copies enqueued (payload and descriptors)         */
  int64_t payload_bytes;    /* KV / weight payload bytes moved                               */
  int32_t last_variant;     /* variant the last offload / restore actually used              */
  int32_t reserved;
} talaria_counters_t;

/* ---- context ------------------------------------------------------------ */

/* Create a context on CUDA device `device` (cfg may be NULL).  Allocates the
 * descriptor ring, the internal streams and the bounce buffers. */
talaria_status_t talaria_create(talaria_ctx **out, int32_t device, const talaria_config_t *cfg);
/* Waits for the context's own streams, frees everything it owns. */
talaria_status_t talaria_destroy(talaria_ctx *ctx);

/* Page-lock and device-map an existing HOST range so offload / restore / stage
 * may use it (the paper's "unified pinned-memory pool", Sec. 4.3).  Memory from
 * cudaHostAlloc / torch pinned tensors needs no registration. */
talaria_status_t talaria_host_register(talaria_ctx *ctx, void *host, size_t bytes);
talaria_status_t talaria_host_unregister(talaria_ctx *ctx, void *host);

/* ---- (1) chained block hash and prefix match ------------------------------ */

/* Sec. 4.3 / App. B: cumulative hash at page (block) boundaries.  For each full
 * block k of d_tokens:
 *     digest_k = sum_{j<B} mix64( u32(tok[kB+j]) + G*(j+1) )        (mod 2^64)
 *     s_k = s_{k-1}*P + digest_k,  s_{-1} = seed;   hash_k = mix64(s_k)
 * with mix64 the SplitMix64 finaliser, G = 0x9E3779B97F4A7C15, P = 0xD1342543DE82EF95.
 * `seed` stands for the model-name part of the key.  The partial tail block has no
 * hash.  d_tokens: DEVICE int32[n_tokens]; d_hashes_out: DEVICE uint64[n_tokens /
 * block_tokens].  block_tokens >= 1. */
talaria_status_t talaria_block_hash(talaria_ctx *ctx, const int32_t *d_tokens, int64_t n_tokens,
                                    int32_t block_tokens, uint64_t seed, uint64_t *d_hashes_out,
                                    void *stream);

/* Batched match of n_pairs continuations, each against its own session's stored
 * stream (App. A: LCP of the new prompt and the prior prompt plus response).
 *   d_cont_tokens / d_sess_tokens : DEVICE int32, all pairs back to back
 *   cont_offsets / sess_offsets   : HOST int64[n_pairs+1], token offsets (CSR)
 *   d_sess_hashes    : DEVICE uint64 or NULL.  Stored chained hashes of each
 *                      session's full blocks, pairs back to back (pair q starts at
 *                      sum_{r<q} floor(Ts_r/B)).  NULL = derive them from tokens.
 *   d_cont_hashes_out: DEVICE uint64 or NULL, same CSR rule with floor(Tc_r/B).
 *   d_results        : DEVICE talaria_match_t[n_pairs].
 * Fields are defined as in the struct above; matched_blocks counts k <
 * min(floor(Tc/B), floor(Ts/B)). */
talaria_status_t talaria_prefix_match(talaria_ctx *ctx, int32_t n_pairs,
                                      const int32_t *d_cont_tokens, const int64_t *cont_offsets,
                                      const int32_t *d_sess_tokens, const int64_t *sess_offsets,
                                      const uint64_t *d_sess_hashes, int32_t block_tokens,
                                      uint64_t seed, uint64_t *d_cont_hashes_out,
                                      talaria_match_t *d_results, void *stream);

/* Same computation with every array in HOST memory (pageable or pinned).  The inputs are
 * gathered into the context's pinned staging buffer, go to the device in ONE copy, are
 * matched by the same kernels, and hashes and results are written by those kernels straight
 * into the pinned staging (no device-to-host copy).  Nothing is
 * allocated or freed: staging was sized at talaria_create (host_match_bytes).  A batch
 * larger than the staging is processed as several sub-batches of whole pairs; a single
 * pair that does not fit is TALARIA_ERR_EXTENT.  Synchronous: returns after the results
 * are in host memory. */
talaria_status_t talaria_prefix_match_host(talaria_ctx *ctx, int32_t n_pairs,
                                           const int32_t *h_cont_tokens, const int64_t *cont_offsets,
                                           const int32_t *h_sess_tokens, const int64_t *sess_offsets,
                                           const uint64_t *h_sess_hashes, int32_t block_tokens,
                                           uint64_t seed, uint64_t *h_cont_hashes_out,
                                           talaria_match_t *h_results, void *stream);

/* Match against streams that already live on the device (Sec. 4.3: the instance keeps a
 * session's state between its calls; App. A: the new prompt is compared with what the session
 * held).  The caller owns one DEVICE token array and one DEVICE hash array and hands out places
 * ("slots", element offsets) in them.  For each pair the new prompt comes from HOST memory
 * (pageable or pinned), is copied to d_tokens[cont_slot ..) through the context's pinned staging,
 * is matched there against the stored stream d_tokens[sess_slot .. +sess_tokens), and its
 * floor(cont_tokens / B) block hashes are written to d_hashes[cont_hash_slot ..): prompt and hashes
 * stay where the session's next call can name them as its stored stream, so a stored stream never
 * crosses the host link again.  sess_hash_slot names the stored stream's block hashes in d_hashes;
 * -1 derives them (all pairs of a call that have a stored block must agree on this, else
 * TALARIA_ERR_INVALID_ARG).  sess_tokens = 0 is a session with nothing stored.
 * Checked before anything is copied or launched: every range lies inside its array
 * (TALARIA_ERR_EXTENT; the arrays themselves inside their device allocations); no prompt or hash
 * destination overlaps another one or a stored range this call reads (TALARIA_ERR_OVERLAP).
 * A prompt larger than the staging (host_match_bytes) is TALARIA_ERR_EXTENT; a batch larger than
 * it runs as sub-batches of whole pairs.  Nothing is allocated.  Returns after the records are in
 * h_results and the hashes in d_hashes; the prompts reach their places in d_tokens in stream order
 * (work enqueued on `stream` afterwards sees them; another stream must be ordered after `stream`
 * first, e.g. by talaria_sync). */
typedef struct {
  const int32_t *h_cont_tokens;   /* HOST [cont_tokens] */
  int64_t cont_tokens;
  int64_t cont_slot;              /* where the prompt is stored in d_tokens */
  int64_t cont_hash_slot;         /* where its block hashes are stored in d_hashes */
  int64_t sess_slot, sess_tokens; /* the stored stream in d_tokens */
  int64_t sess_hash_slot;         /* its block hashes in d_hashes, or -1 */
} talaria_resident_pair_t;
talaria_status_t talaria_prefix_match_resident(talaria_ctx *ctx, int32_t n_pairs,
                                               const talaria_resident_pair_t *pairs /* HOST */,
                                               int32_t *d_tokens, int64_t tokens_capacity,
                                               uint64_t *d_hashes, int64_t hashes_capacity,
                                               int32_t block_tokens, uint64_t seed,
                                               talaria_match_t *h_results /* HOST */, void *stream);

/* No counterpart in the paper: an allocation-free form of talaria_prefix_match.
 *
 * Who needs it: a serving process that has handed all of HBM to its own memory
 * manager, or a latency-critical thread inside a serving loop.  Such callers must
 * not reach the CUDA allocator: a device allocation may simply fail when no HBM is
 * left, and allocating or freeing device memory makes every stream of the device
 * wait.  They also may not want a talaria context, whose creation allocates.
 *
 * This entry point takes no context and allocates nothing, on the device or on the
 * host: no cudaMalloc / cudaFree, no pinned staging, no copies.  Its scratch (block
 * digests and per-tile mismatch positions) is a fixed 1 MiB array inside the library
 * image, held by every GPU that loads the library until the process exits, and the
 * pair descriptors travel in the kernel parameters.  Arguments and results are
 * exactly those of talaria_prefix_match; the caller still owns every buffer.
 *
 * Limits (TALARIA_ERR_EXTENT beyond them, nothing is launched):
 *   n_pairs <= 8, and
 *   sum over pairs of floor(Tc/B) [+ floor(Ts/B) when d_sess_hashes is NULL]
 *     + ceil(max(Tc,Ts)/2048)  <=  131,072 scratch words
 *   (for example one pair of two 1,000,000-token streams at B = 16).
 * The work runs on the CURRENT device (cudaSetDevice is the caller's business).
 * The first call on each device looks up the scratch array's device address; make
 * that first call before any stream capture.  All calls in a process share the one
 * scratch array per device: two calls whose kernels can overlap on the GPU
 * (different streams, no ordering between them) race on it and must be serialised
 * by the caller.  Host threads may call concurrently: the two launches of a call are
 * issued under one internal lock.  The array keeps the previous call's contents; nothing in it
 * needs clearing because every word that is read is written first in the same
 * call. */
talaria_status_t talaria_prefix_match_static(int32_t n_pairs, const int32_t *d_cont_tokens,
                                             const int64_t *cont_offsets,
                                             const int32_t *d_sess_tokens,
                                             const int64_t *sess_offsets,
                                             const uint64_t *d_sess_hashes, int32_t block_tokens,
                                             uint64_t seed, uint64_t *d_cont_hashes_out,
                                             talaria_match_t *d_results, void *stream);

/* App. B "Prefix agreement": the longest leading block range on which all R
 * ranks committed a block and hold the same chained hash.  Pure host arithmetic.
 * committed_blocks: HOST int64[R]; hashes: HOST uint64[R][stride]. */
int64_t talaria_prefix_agree(int32_t n_ranks, const int64_t *committed_blocks,
                             const uint64_t *hashes, int64_t stride);

/* Host-side page registry (Sec. 4.3: a block's key is the model name together with the
 * cumulative prefix hash, at the radix tree's chunk granularity).  Maps a chained block hash
 * (the model key is its seed) to the byte offset of the block's page-first slab in the
 * pinned host pool.  Pure host code, internally locked; all arrays are HOST arrays.
 *   insert        : keys already present keep their value (first wins); *n_new (nullable)
 *                   receives the number of new keys.
 *   lookup_prefix : number of LEADING hashes that are present; their page offsets are
 *                   written to page_offsets_out (nullable).  Because the hashes are
 *                   cumulative, this is the longest restorable prefix of the stream.
 *   erase         : removes the keys that are present; *n_erased (nullable) counts them.
 * The table grows by itself. */
typedef struct talaria_registry talaria_registry;
talaria_status_t talaria_registry_create(talaria_registry **out, int64_t expected_pages);
talaria_status_t talaria_registry_destroy(talaria_registry *reg);
talaria_status_t talaria_registry_insert(talaria_registry *reg, const uint64_t *hashes,
                                         const int64_t *page_offsets, int64_t n, int64_t *n_new);
int64_t talaria_registry_lookup_prefix(talaria_registry *reg, const uint64_t *hashes, int64_t n,
                                       int64_t *page_offsets_out);
talaria_status_t talaria_registry_erase(talaria_registry *reg, const uint64_t *hashes, int64_t n,
                                        int64_t *n_erased);
int64_t talaria_registry_size(talaria_registry *reg);

/* ---- (2)/(3) block-table copies ------------------------------------------- */

/* Sec. 4.3 checkpoint: host_dst[l,p,i] <- pool_{l,p}[block_table[first_block+i]]
 * for i < n_blocks, whole chunks.  block_table: HOST int32 (at least first_block +
 * n_blocks entries); duplicates allowed.  host_dst: HOST pinned (cudaHostAlloc,
 * torch pinned, or talaria_host_register) image described by hl.  The pool is only
 * read.  Errors: BAD_BLOCK_ID, EXTENT (image exceeds capacity_bytes),
 * HOST_NOT_PINNED, INVALID_ARG. */
talaria_status_t talaria_kv_offload(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                    const int32_t *block_table, int64_t first_block,
                                    int64_t n_blocks, void *host_dst,
                                    const talaria_host_layout_t *hl, void *stream);

/* Sec. 4.3 restore into new device slots: pool_{l,p}[new_block_table[first_block+i]]
 * <- host_src[l,p,i] for i < n_blocks; every other pool byte is left unchanged.
 * Duplicate ids are rejected (DUP_BLOCK) because the result would depend on copy
 * order. */
talaria_status_t talaria_kv_restore(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                    const int32_t *new_block_table, int64_t first_block,
                                    int64_t n_blocks, const void *host_src,
                                    const talaria_host_layout_t *hl, void *stream);

/* The same restore, delivered layer by layer (App. C: the layer-first view matches the
 * device-side layout used by attention kernels; Sec. 3.4 charges the restore to the
 * prefill budget, so prefill of layer l should start as soon as layer l has landed).
 * The result in the pool is exactly that of talaria_kv_restore.  In addition
 * layer_events[l] (HOST array of num_layers cudaEvent_t handles created by the
 * caller, passed as void*) is recorded once every chunk of layer l, both planes, is
 * in the pool; a consumer stream calls cudaStreamWaitEvent on it.  Layers complete in
 * increasing order for large images (copy-engine path, any host layout: contiguous or
 * pitched transfers per layer); for small images, zero-copy contexts or layouts with
 * neither planes nor blocks adjacent, all events are recorded after one ordinary
 * restore.  Work enqueued on `stream` after the call still waits for the whole
 * restore. */
talaria_status_t talaria_kv_restore_layered(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                            const int32_t *new_block_table, int64_t first_block,
                                            int64_t n_blocks, const void *host_src,
                                            const talaria_host_layout_t *hl,
                                            void *const *layer_events, void *stream);

/* Page-first registry slabs (App. C: the host copy is organised by logical prefix page,
 * one page descriptor covering that page's fragments of every layer; Sec. 4.3: slabs of
 * one unified pinned pool).  Logical block i is ONE slab of
 * num_layers*num_planes*C bytes, fragments ordered [layer][plane], at byte offset
 * page_offsets[i] (HOST int64[n_blocks]) of the pinned HOST pool (host_pool, pool_bytes).
 * Slabs may sit anywhere in the pool, in any order: the registry commits, invalidates
 * and restores at page granularity.
 *   offload_pages: slab_i <- pool_{l,p}[block_table[first_block+i]]   (slabs must not overlap: OVERLAP)
 *   restore_pages: pool_{l,p}[new_block_table[first_block+i]] <- slab_i  (DUP_BLOCK as in restore)
 * Errors also: EXTENT (a slab leaves the pool), HOST_NOT_PINNED, BAD_BLOCK_ID. */
talaria_status_t talaria_kv_offload_pages(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                          const int32_t *block_table, int64_t first_block,
                                          int64_t n_blocks, void *host_pool, int64_t pool_bytes,
                                          const int64_t *page_offsets, void *stream);
talaria_status_t talaria_kv_restore_pages(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                          const int32_t *new_block_table, int64_t first_block,
                                          int64_t n_blocks, const void *host_pool, int64_t pool_bytes,
                                          const int64_t *page_offsets, void *stream);

/* Several sessions in one call.  Every argument of every session is checked before anything is
 * enqueued; restore tables are also checked against each other (no block may be claimed
 * twice).  Sessions small enough for the zero-copy kernel whose images share their layer and
 * plane strides (any page-first images; layer-first images of equal block count) are moved by
 * ONE fused launch; with at most 256 blocks in total even its descriptor travels in the kernel
 * parameters.  Larger sessions use the copy-engine variants, one after the other on `stream`. */
typedef struct {
  const int32_t *block_table; /* HOST */
  int64_t first_block, n_blocks;
  void *host;                 /* HOST pinned image (written by offload, read by restore) */
  talaria_host_layout_t hl;
} talaria_kv_xfer_t;
talaria_status_t talaria_kv_offload_batch(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                          const talaria_kv_xfer_t *xfers, int32_t n_xfers,
                                          void *stream);
talaria_status_t talaria_kv_restore_batch(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                          const talaria_kv_xfer_t *xfers, int32_t n_xfers,
                                          void *stream);

/* The same block-table gather / scatter with the image in DEVICE memory (the
 * in-HBM leg of the bounce variant, exposed for callers that pack KV pages on
 * the device, App. C "pack and unpack KV pages"). */
talaria_status_t talaria_kv_gather(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                   const int32_t *block_table, int64_t first_block,
                                   int64_t n_blocks, void *d_image,
                                   const talaria_host_layout_t *il, void *stream);
talaria_status_t talaria_kv_scatter(talaria_ctx *ctx, const talaria_kv_layout_t *kv,
                                    const int32_t *new_block_table, int64_t first_block,
                                    int64_t n_blocks, const void *d_image,
                                    const talaria_host_layout_t *il, void *stream);

/* ---- (4) staged switching -------------------------------------------------- */

/* Sec. 4.4 gather plan: for each of the n entries, dst_dev[0..bytes) <- src_dev
 * if the chunk is clean and present, else <- src_host (dirty: bit chunk_id of
 * dirty_bitmap set, LSB-first bytes; missing: src_dev == NULL).  plan and
 * dirty_bitmap are HOST arrays (bitmap may be NULL = all clean; it must cover the
 * largest chunk_id).  src_host must be pinned where it is used.  Destinations must
 * be pairwise disjoint and disjoint from every staged source that is read
 * (OVERLAP).  stats (HOST, nullable) is filled before return.
 * The clean entries are one D2D kernel on `stream`.  The host-sourced entries run
 * beside it on an internal stream that `stream` then waits for: up to 32 merged runs
 * as copy-engine copies of at most 32 MiB, more than that as a second, small launch
 * of the same kernel that reads the pinned copies through their device mapping (the
 * call returns at once instead of feeding thousands of copies to a full queue, and
 * a restore issued meanwhile keeps a share of the host link). */
talaria_status_t talaria_stage(talaria_ctx *ctx, const talaria_copy_t *plan, int64_t n,
                               const uint8_t *dirty_bitmap, talaria_stage_stats_t *stats,
                               void *stream);

/* The same switch with the planning taken off the critical path.  A cold-pool instance switches
 * among a fixed set of models, so the gather plan of a model is known long before the switch
 * (Sec. 4.4: staging goes on in the background of the model that is serving).  create validates the
 * plan once (destinations pairwise disjoint and disjoint from EVERY staged source, whatever
 * a later bitmap says) and keeps its descriptors in device memory; run then costs one bitmap
 * upload, one launch and the copy-engine copies of the chunks that are dirty or missing this
 * time.  Results and stats are those of talaria_stage with the same plan and bitmap.  The
 * bitmap must cover the largest chunk_id of the plan.  Runs of one prepared plan must be
 * ordered on the GPU by the caller (same stream, or events). */
typedef struct talaria_stage_plan talaria_stage_plan;
talaria_status_t talaria_stage_plan_create(talaria_ctx *ctx, const talaria_copy_t *plan, int64_t n,
                                           talaria_stage_plan **out);
talaria_status_t talaria_stage_plan_run(talaria_ctx *ctx, talaria_stage_plan *prepared,
                                        const uint8_t *dirty_bitmap, talaria_stage_stats_t *stats,
                                        void *stream);
talaria_status_t talaria_stage_plan_destroy(talaria_ctx *ctx, talaria_stage_plan *prepared);

/* Sec. 4.4 pre-staging, the step that runs while the current model is still serving:
 * for every plan entry, the authoritative HOST bytes (src_host, pinned) are written to
 * the chunk's place in the staging region (src_dev, a DEVICE address inside unused KV
 * rows), unless bit chunk_id of blocked_bitmap is set (those rows currently belong to
 * a KV allocation, so the chunk stays unstaged).  chunk_id must be >= 0.  For each
 * chunk written, its bit in staged_bitmap (HOST, in/out, nullable) is set and its
 * bit in dirty_bitmap (HOST, in/out, nullable) is cleared.  dst_dev is ignored.
 * stats (nullable): h2d_bytes = bytes written, missing_chunks = chunks skipped,
 * dirty_chunks = dirty bits cleared, d2d_bytes = 0.  Copy-engine transfers on
 * `stream`; bitmaps are updated before return, the data lands when the stream gets
 * there.  Errors: INVALID_ARG, HOST_NOT_PINNED, OVERLAP (two written staging ranges
 * intersect). */
talaria_status_t talaria_prestage(talaria_ctx *ctx, const talaria_copy_t *plan, int64_t n,
                                  const uint8_t *blocked_bitmap, uint8_t *staged_bitmap,
                                  uint8_t *dirty_bitmap, talaria_stage_stats_t *stats, void *stream);

/* Sec. 4.4: a staged chunk becomes dirty when a prefill allocation made meanwhile claims
 * rows inside the chunk's staging range.  Pure host arithmetic: sets the dirty bit of
 * every staged chunk (all chunks when staged_bitmap is NULL) whose staging bytes
 * [src_dev, src_dev+bytes) intersect [alloc_base, alloc_base+alloc_bytes).  Returns the
 * number of bits that changed from clean to dirty. */
int64_t talaria_mark_dirty(const talaria_copy_t *plan, int64_t n, const void *alloc_base,
                           int64_t alloc_bytes, const uint8_t *staged_bitmap, uint8_t *dirty_bitmap);

/* ---- stable-address HBM layout (Sec. 4.2, Sec. 4.4) -------------------------------- */

/* One managed region for every model of a cold-pool instance (Sec. 4.2): for the active model
 * the weights grow up from the low-address end, the runtime buffers are anchored at the
 * high-address end, and the gap between them is the paged KV pool.  Pure host arithmetic:
 * region_base is a DEVICE address that is only ever added to, never dereferenced.
 *
 * Layout of model m in a region of S bytes (A = align, a power of two; C = chunk_bytes, a
 * multiple of A; LP = num_layers*num_planes):
 *     weights  [0, weight_bytes)
 *     runtime  [R, R + runtime_bytes)          R = floor((S - runtime_bytes) / A) * A
 *     KV pool  plane k = [K + k*NB*C, +NB*C)   K = ceil(weight_bytes / A) * A,
 *                                              NB = floor((R - K) / (LP*C)) >= 1 (else EXTENT)
 * Every address is a function of (region, model) only: a model finds its weights, KV planes and
 * runtime buffers where they were the last time (the restore-time pointer check of Sec. 4.2
 * compares exactly these bases).
 *
 * activate(m)    : m becomes the active model; all of its NB blocks are free; any staging
 *                  placement is forgotten (the switch consumed it).
 * alloc_blocks   : n block ids, lowest free ids first (Sec. 4.4: low addresses are reused first,
 *                  which keeps the plane tails clean), passing over rows under an active staging
 *                  write.  A block id is a row of EVERY plane; for each staged chunk (bit set in
 *                  staged_bitmap, or every placed chunk if that is NULL) that loses a row to the
 *                  allocation, its bit in dirty_bitmap (nullable, in/out) is set; *n_dirtied
 *                  (nullable) counts bits that changed.  NO_MEMORY if fewer than n ids are
 *                  available (nothing is taken).
 * free_blocks    : INVALID_ARG for an id that is out of range, already free or given twice.
 * stage_place    : plans pre-staging of model `next` (Sec. 4.4): its weights are cut into chunks
 *                  of chunk_bytes (the last may be short); chunk j goes to the next usable tail
 *                  slot, slots being taken tail slot by tail slot across all planes (slot t of a
 *                  plane = rows [NB-(t+1)*r, NB-t*r), r = ceil(chunk_bytes / C)).  A slot is
 *                  usable when all its rows are free and unlocked and none of its bytes lies in
 *                  [0, ceil(next.weight_bytes / A) * A), where the switch will write.  plan_out[j]
 *                  (HOST array, capacity >= *n_chunks_out, else EXTENT) = { src_dev = the slot's
 *                  address or NULL if no slot was left, src_host = host_weights + j*chunk_bytes
 *                  (NULL when host_weights is NULL), dst_dev = next's weights base + j*chunk_bytes,
 *                  bytes, chunk_id = j }: ready for talaria_prestage, talaria_mark_dirty and
 *                  talaria_stage / talaria_stage_plan_create.
 * lock_chunk     : marks a placed chunk as being written (locked != 0) or done (0).
 * staging_slack  : bytes of weights that could still be staged for `next` at this chunk size
 *                  (usable slots not holding a chunk, times chunk_bytes): the paper's staging
 *                  slack signal. */
typedef struct talaria_bump talaria_bump;
typedef struct {
  int64_t weight_bytes, runtime_bytes;
  int32_t num_layers, num_planes;
  int64_t chunk_bytes;
} talaria_model_desc_t;
typedef struct {
  void *weights_base;
  int64_t weights_bytes;
  void *kv_base;
  int64_t kv_bytes;          /* num_layers * num_planes * num_blocks * chunk_bytes */
  void *runtime_base;
  int64_t runtime_bytes;
  int64_t num_blocks;        /* rows per plane = pool capacity in blocks */
} talaria_bump_view_t;
talaria_status_t talaria_bump_create(talaria_bump **out, void *region_base, int64_t region_bytes, int64_t align,
                                     const talaria_model_desc_t *models, int32_t n_models);
talaria_status_t talaria_bump_destroy(talaria_bump *b);
/* plane_base_out: HOST array [num_layers*num_planes] or NULL; usable as talaria_kv_layout_t.plane_base. */
talaria_status_t talaria_bump_view(talaria_bump *b, int32_t model, talaria_bump_view_t *view, void **plane_base_out);
talaria_status_t talaria_bump_activate(talaria_bump *b, int32_t model, talaria_bump_view_t *view /*nullable*/);
talaria_status_t talaria_bump_alloc_blocks(talaria_bump *b, int64_t n, int32_t *ids_out, const uint8_t *staged_bitmap,
                                           uint8_t *dirty_bitmap, int64_t *n_dirtied);
talaria_status_t talaria_bump_free_blocks(talaria_bump *b, const int32_t *ids, int64_t n);
int64_t talaria_bump_free_count(talaria_bump *b);
talaria_status_t talaria_bump_stage_place(talaria_bump *b, int32_t next_model, int64_t chunk_bytes,
                                          const void *host_weights, talaria_copy_t *plan_out, int64_t plan_capacity,
                                          int64_t *n_chunks_out, int64_t *n_placed_out /*nullable*/);
talaria_status_t talaria_bump_lock_chunk(talaria_bump *b, int32_t chunk_id, int32_t locked);
int64_t talaria_bump_staging_slack(talaria_bump *b, int32_t next_model, int64_t chunk_bytes);

/* ---- argument checks that need no GPU ------------------------------------------ */

/* The same host-side validation the copy and stage calls apply, callable on its own
 * (for example when a table or plan is built, long before it is used).
 *   check_block_table  : BAD_BLOCK_ID, and DUP_BLOCK when reject_duplicates != 0.
 *   check_image_layout : the three strides must nest without overlap (INVALID_ARG) and the
 *                        image must fit capacity_bytes (EXTENT); plane_base may be NULL.
 *                        *contiguous_run_bytes (nullable) receives the length of the image's
 *                        contiguous runs, which decides whether large copy-engine
 *                        transfers are possible.
 *   check_stage_plan   : INVALID_ARG / OVERLAP as in talaria_stage; fills stats. */
talaria_status_t talaria_check_block_table(const int32_t *block_table, int64_t n, int64_t num_blocks,
                                           int32_t reject_duplicates);
talaria_status_t talaria_check_image_layout(const talaria_kv_layout_t *kv, int64_t n_blocks,
                                            const talaria_host_layout_t *hl, int64_t *contiguous_run_bytes);
talaria_status_t talaria_check_stage_plan(const talaria_copy_t *plan, int64_t n, const uint8_t *dirty_bitmap,
                                          talaria_stage_stats_t *stats);

/* ---- completion, errors, counters ------------------------------------------ */

/* Sec. 4.3 / App. B "Switch barrier": block the host until everything enqueued on
 * `stream` (offloads included) has finished.  Also the place where a device-side
 * finding surfaces: the copy kernels never touch memory outside the pool -- a table
 * entry outside [0, num_blocks) that reaches them (only possible with validate = 0)
 * makes them skip that chunk and set a status word, and the next talaria_sync of the
 * context returns TALARIA_ERR_BAD_BLOCK_ID once (the word is then cleared).  The word
 * belongs to the context, not to a stream: whichever stream is synchronised first
 * reports it. */
talaria_status_t talaria_sync(talaria_ctx *ctx, void *stream);

const char *talaria_strerror(talaria_status_t status);
/* cudaError_t value of the last failed CUDA call in this context (0 if none). */
int32_t talaria_last_cuda_error(talaria_ctx *ctx);
talaria_status_t talaria_get_counters(talaria_ctx *ctx, talaria_counters_t *out);
/* Timing is off by default (events cost a little on every call).  With it on, every offload,
 * restore (all forms) and stage records its events; talaria_get_timing waits for the last timed
 * call to finish and returns its times (INVALID_ARG if no call was timed yet). */
talaria_status_t talaria_set_timing(talaria_ctx *ctx, int32_t enabled);
talaria_status_t talaria_get_timing(talaria_ctx *ctx, talaria_timing_t *out);
talaria_status_t talaria_reset_counters(talaria_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* TALARIA_H_ */
