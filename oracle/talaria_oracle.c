/*
 * CPU oracle for the instance-local KV substrate of the Talaria paper.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, single-threaded, plain
 * definition of every result the CUDA library produces.  It is used by the
 * tests, by the smoke check and by the benchmark's CPU-baseline leg; nothing
 * on the product path may call it, and it shares no code, header, table or
 * constant generator with the CUDA sources.
 *
 * Parity status of each function against the paper:
 *   orc_lcp_tokens        pinned   (App. A "Prefix reuse": longest common
 *                                   prefix after tokenisation; brute force,
 *                                   numpy cross-check, constructed cases)
 *   orc_kv_offload_* /
 *   orc_kv_restore_*      pinned   (Sec. 4.3 + App. C: block-table copies;
 *                                   round-trip invariants, element-wise vs
 *                                   chunk form, numpy fancy indexing)
 *   orc_stage             pinned   (Sec. 4.4: clean chunks copied device to
 *                                   device, dirty/missing chunks from host;
 *                                   numpy slice cross-check, corrupted-dirty
 *                                   staging test)
 *   orc_prefix_agree      pinned   (App. B "Prefix agreement": brute force)
 *   orc_kv_offload_pages /
 *   orc_kv_restore_pages  pinned   (App. C page-first: one slab per logical page; reduces
 *                                   to the dense page-first image when pages are
 *                                   consecutive, numpy check for shuffled pages)
 *   orc_prestage /
 *   orc_mark_dirty        pinned   (Sec. 4.4 pre-staging protocol: numpy slice and
 *                                   interval brute force)
 *   orc_block_hash        PARITY UNPINNED against the paper: Sec. 4.3 only says
 *                                   "cumulative prefix hash" per block and
 *                                   prints no function, width or value.  The
 *                                   definition below is this build's reading;
 *                                   it is pinned only by mathematics: the
 *                                   published SplitMix64 output sequence
 *                                   (for the finaliser and digest of an
 *                                   all-zero block), the closed form of the
 *                                   affine chain, the prefix property and
 *                                   exhaustive injectivity on tiny alphabets.
 *
 * All pointers are host pointers.  Nothing here allocates except
 * orc_stage_validate (a temporary index array).
 */
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ */
/* Chained block hash (reading of Sec. 4.3 "cumulative prefix hash",    */
/* App. B "cumulative prefix hash at page boundaries")                  */
/* ------------------------------------------------------------------ */

/* 64-bit finaliser of SplitMix64 (Steele, Lea, Flood 2014). */
uint64_t orc_mix64(uint64_t z)
{
    z ^= z >> 30;
    z *= 0xBF58476D1CE4E5B9ULL;
    z ^= z >> 27;
    z *= 0x94D049BB133111EBULL;
    z ^= z >> 31;
    return z;
}

#define ORC_G 0x9E3779B97F4A7C15ULL /* position weight (golden-ratio gamma) */
#define ORC_P 0xD1342543DE82EF95ULL /* chain multiplier, odd                */

/* digest_k = sum_{j<B} mix64( u32(tok[kB+j]) + G*(j+1) )   (mod 2^64) */
uint64_t orc_block_digest(const int32_t *tok, int32_t B)
{
    uint64_t acc = 0;
    for (int32_t j = 0; j < B; ++j) {
        uint64_t t = (uint64_t)(uint32_t)tok[j];
        acc += orc_mix64(t + ORC_G * (uint64_t)(j + 1));
    }
    return acc;
}

/* s_{-1} = seed; s_k = s_{k-1}*P + digest_k; hash_k = mix64(s_k).
 * Only full blocks are hashed: out has floor(T/B) entries.  Returns that count. */
int64_t orc_block_hash(const int32_t *tok, int64_t T, int32_t B, uint64_t seed,
                       uint64_t *out)
{
    if (B <= 0 || T < 0) return -1;
    int64_t nb = T / B;
    uint64_t s = seed;
    for (int64_t k = 0; k < nb; ++k) {
        s = s * ORC_P + orc_block_digest(tok + k * (int64_t)B, B);
        out[k] = orc_mix64(s);
    }
    return nb;
}

/* ------------------------------------------------------------------ */
/* Prefix match (App. A "Prefix reuse"; Sec. 4.3 keyed blocks)          */
/* ------------------------------------------------------------------ */

/* Longest common prefix, one token at a time. */
int64_t orc_lcp_tokens(const int32_t *a, int64_t Ta, const int32_t *b, int64_t Tb)
{
    int64_t n = Ta < Tb ? Ta : Tb;
    int64_t k = 0;
    while (k < n && a[k] == b[k]) ++k;
    return k;
}

typedef struct {
    int64_t lcp_tokens;
    int64_t matched_blocks;
    int64_t reusable_tokens;
    int32_t hash_token_disagree;
    int32_t pad_;
} orc_match_t;

/* cont vs one stored session stream.
 * sess_hashes: stored chained hashes of the session's full blocks, or NULL to
 *              derive them from sess tokens here.
 * cont_hashes_out: NULL or room for floor(Tc/B) hashes.
 * scratch: room for floor(Tc/B)+floor(Ts/B) uint64 (caller-owned). */
int32_t orc_prefix_match(const int32_t *cont, int64_t Tc, const int32_t *sess, int64_t Ts,
                         const uint64_t *sess_hashes, int32_t B, uint64_t seed,
                         uint64_t *cont_hashes_out, uint64_t *scratch, orc_match_t *res)
{
    if (B <= 0 || Tc < 0 || Ts < 0) return -1;
    int64_t nbc = Tc / B, nbs = Ts / B;
    uint64_t *hc = scratch;
    uint64_t *hs = scratch + nbc;
    orc_block_hash(cont, Tc, B, seed, hc);
    if (sess_hashes) {
        for (int64_t k = 0; k < nbs; ++k) hs[k] = sess_hashes[k];
    } else {
        orc_block_hash(sess, Ts, B, seed, hs);
    }
    int64_t lim = nbc < nbs ? nbc : nbs;
    int64_t m = 0;
    while (m < lim && hc[m] == hs[m]) ++m;
    int64_t lcp = orc_lcp_tokens(cont, Tc, sess, Ts);
    int64_t lcp_blocks = lcp / B;
    int64_t token_blocks = lcp_blocks < lim ? lcp_blocks : lim;
    res->lcp_tokens = lcp;
    res->matched_blocks = m;
    res->reusable_tokens = (int64_t)B * (m < lcp_blocks ? m : lcp_blocks);
    res->hash_token_disagree = (m != token_blocks) ? 1 : 0;
    res->pad_ = 0;
    if (cont_hashes_out)
        for (int64_t k = 0; k < nbc; ++k) cont_hashes_out[k] = hc[k];
    return 0;
}

/* App. B "Prefix agreement": every rank reports its committed full-block count
 * and its chained hashes; the published prefix is the longest leading block
 * range on which all ranks hold the same hash.  hashes is [R][stride]. */
int64_t orc_prefix_agree(int32_t R, const int64_t *committed_blocks,
                         const uint64_t *hashes, int64_t stride)
{
    if (R <= 0) return 0;
    int64_t lim = committed_blocks[0];
    for (int32_t r = 1; r < R; ++r)
        if (committed_blocks[r] < lim) lim = committed_blocks[r];
    if (lim < 0) lim = 0;
    int64_t k = 0;
    for (; k < lim; ++k) {
        int same = 1;
        for (int32_t r = 1; r < R; ++r)
            if (hashes[(int64_t)r * stride + k] != hashes[k]) { same = 0; break; }
        if (!same) break;
    }
    return k;
}

/* ------------------------------------------------------------------ */
/* Block-table copies (Sec. 4.3 checkpoint / restore; App. C LF / PF)    */
/* ------------------------------------------------------------------ */

typedef struct {
    int32_t num_layers, num_kv_heads, block_tokens, head_dim, elt_bytes, num_planes;
    int64_t num_blocks;
    uint8_t *const *plane_base; /* [num_layers*num_planes] host pointers, each
                                   [num_blocks, kv_heads, block_tokens, head_dim] */
} orc_kv_layout_t;

typedef struct {
    int64_t stride_layer, stride_plane, stride_block; /* bytes */
    int64_t capacity_bytes;
} orc_host_layout_t;

static int64_t orc_chunk_bytes(const orc_kv_layout_t *kv)
{
    return (int64_t)kv->num_kv_heads * kv->block_tokens * kv->head_dim * kv->elt_bytes;
}

/* Element-wise definition: host[l,p,i][h,t,d] <- pool_{l,p}[bt[first+i]][h,t,d]. */
int32_t orc_kv_offload_elem(const orc_kv_layout_t *kv, const int32_t *bt, int64_t first,
                            int64_t n, uint8_t *host, const orc_host_layout_t *hl)
{
    const int64_t H = kv->num_kv_heads, B = kv->block_tokens, D = kv->head_dim, e = kv->elt_bytes;
    for (int32_t l = 0; l < kv->num_layers; ++l)
        for (int32_t p = 0; p < kv->num_planes; ++p) {
            const uint8_t *plane = kv->plane_base[l * kv->num_planes + p];
            for (int64_t i = 0; i < n; ++i) {
                int64_t b = bt[first + i];
                if (b < 0 || b >= kv->num_blocks) return -2;
                uint8_t *img = host + l * hl->stride_layer + p * hl->stride_plane + i * hl->stride_block;
                for (int64_t h = 0; h < H; ++h)
                    for (int64_t t = 0; t < B; ++t)
                        for (int64_t d = 0; d < D; ++d) {
                            int64_t src = (((b * H + h) * B + t) * D + d) * e;
                            int64_t dst = ((h * B + t) * D + d) * e;
                            for (int64_t q = 0; q < e; ++q) img[dst + q] = plane[src + q];
                        }
            }
        }
    return 0;
}

/* Element-wise definition: pool_{l,p}[bt[first+i]][h,t,d] <- host[l,p,i][h,t,d]. */
int32_t orc_kv_restore_elem(const orc_kv_layout_t *kv, const int32_t *bt, int64_t first,
                            int64_t n, const uint8_t *host, const orc_host_layout_t *hl)
{
    const int64_t H = kv->num_kv_heads, B = kv->block_tokens, D = kv->head_dim, e = kv->elt_bytes;
    for (int32_t l = 0; l < kv->num_layers; ++l)
        for (int32_t p = 0; p < kv->num_planes; ++p) {
            uint8_t *plane = kv->plane_base[l * kv->num_planes + p];
            for (int64_t i = 0; i < n; ++i) {
                int64_t b = bt[first + i];
                if (b < 0 || b >= kv->num_blocks) return -2;
                const uint8_t *img = host + l * hl->stride_layer + p * hl->stride_plane + i * hl->stride_block;
                for (int64_t h = 0; h < H; ++h)
                    for (int64_t t = 0; t < B; ++t)
                        for (int64_t d = 0; d < D; ++d) {
                            int64_t dst = (((b * H + h) * B + t) * D + d) * e;
                            int64_t src = ((h * B + t) * D + d) * e;
                            for (int64_t q = 0; q < e; ++q) plane[dst + q] = img[src + q];
                        }
            }
        }
    return 0;
}

/* Chunk form: one memcpy per (layer, plane, logical block).  Same result as the
 * element-wise form because a block's [kv_heads, block_tokens, head_dim] slab
 * is contiguous on both sides. */
int32_t orc_kv_offload_chunk(const orc_kv_layout_t *kv, const int32_t *bt, int64_t first,
                             int64_t n, uint8_t *host, const orc_host_layout_t *hl)
{
    const int64_t C = orc_chunk_bytes(kv);
    for (int32_t l = 0; l < kv->num_layers; ++l)
        for (int32_t p = 0; p < kv->num_planes; ++p) {
            const uint8_t *plane = kv->plane_base[l * kv->num_planes + p];
            for (int64_t i = 0; i < n; ++i) {
                int64_t b = bt[first + i];
                if (b < 0 || b >= kv->num_blocks) return -2;
                memcpy(host + l * hl->stride_layer + p * hl->stride_plane + i * hl->stride_block,
                       plane + b * C, (size_t)C);
            }
        }
    return 0;
}

int32_t orc_kv_restore_chunk(const orc_kv_layout_t *kv, const int32_t *bt, int64_t first,
                             int64_t n, const uint8_t *host, const orc_host_layout_t *hl)
{
    const int64_t C = orc_chunk_bytes(kv);
    for (int32_t l = 0; l < kv->num_layers; ++l)
        for (int32_t p = 0; p < kv->num_planes; ++p) {
            uint8_t *plane = kv->plane_base[l * kv->num_planes + p];
            for (int64_t i = 0; i < n; ++i) {
                int64_t b = bt[first + i];
                if (b < 0 || b >= kv->num_blocks) return -2;
                memcpy(plane + b * C,
                       host + l * hl->stride_layer + p * hl->stride_plane + i * hl->stride_block,
                       (size_t)C);
            }
        }
    return 0;
}

/* Page-first registry slabs (App. C: "grouped by logical prefix page, with the
 * per-layer fragments for that page stored under one page descriptor"): logical block
 * i lives in one slab of layers*planes*C bytes at byte offset page_off[i] of the host
 * pool, fragments ordered [layer][plane].  to_host: slab <- pool chunk; else pool <- slab. */
int32_t orc_kv_pages(const orc_kv_layout_t *kv, const int32_t *bt, int64_t first, int64_t n,
                     uint8_t *host_pool, int64_t pool_bytes, const int64_t *page_off, int32_t to_host)
{
    const int64_t C = orc_chunk_bytes(kv);
    const int64_t slab = (int64_t)kv->num_layers * kv->num_planes * C;
    for (int64_t i = 0; i < n; ++i) {
        int64_t b = bt[first + i];
        if (b < 0 || b >= kv->num_blocks) return -2;
        if (page_off[i] < 0 || page_off[i] + slab > pool_bytes) return -5;
        for (int32_t l = 0; l < kv->num_layers; ++l)
            for (int32_t p = 0; p < kv->num_planes; ++p) {
                uint8_t *plane = kv->plane_base[l * kv->num_planes + p];
                uint8_t *frag = host_pool + page_off[i] + ((int64_t)l * kv->num_planes + p) * C;
                if (to_host) memcpy(frag, plane + b * C, (size_t)C);
                else         memcpy(plane + b * C, frag, (size_t)C);
            }
    }
    return 0;
}

/* ------------------------------------------------------------------ */
/* Staged switching (Sec. 4.4; App. D path classification)              */
/* ------------------------------------------------------------------ */

typedef struct {
    const uint8_t *src_dev;  /* staged copy ("device" side; NULL = chunk missing) */
    const uint8_t *src_host; /* authoritative host copy (may be NULL if never needed) */
    uint8_t *dst_dev;        /* stable-address slot */
    int64_t bytes;
    int32_t chunk_id;        /* index into the dirty bitmap */
    int32_t pad_;
} orc_copy_t;

typedef struct {
    int64_t d2d_bytes, h2d_bytes, dirty_chunks, missing_chunks;
} orc_stage_stats_t;

static int orc_bit(const uint8_t *bm, int64_t i) { return (bm[i >> 3] >> (i & 7)) & 1; }

/* A clean, present chunk is copied from its staged source; a chunk that is
 * dirty (bit set, LSB-first bytes) or missing (no staged source) comes from
 * the host copy.  Returns -1 if a host copy is needed but absent. */
int32_t orc_stage(const orc_copy_t *plan, int64_t n, const uint8_t *dirty_bitmap,
                  orc_stage_stats_t *st)
{
    orc_stage_stats_t s = {0, 0, 0, 0};
    for (int64_t k = 0; k < n; ++k) {
        const orc_copy_t *c = &plan[k];
        if (c->bytes < 0 || !c->dst_dev) return -1;
        int missing = (c->src_dev == NULL);
        int dirty = (!missing && dirty_bitmap && c->chunk_id >= 0 && orc_bit(dirty_bitmap, c->chunk_id));
        if (missing || dirty) {
            if (!c->src_host) return -1;
            memcpy(c->dst_dev, c->src_host, (size_t)c->bytes);
            s.h2d_bytes += c->bytes;
            if (missing) s.missing_chunks += 1; else s.dirty_chunks += 1;
        } else {
            memcpy(c->dst_dev, c->src_dev, (size_t)c->bytes);
            s.d2d_bytes += c->bytes;
        }
    }
    if (st) *st = s;
    return 0;
}

/* Destination ranges must be pairwise disjoint and must not intersect any
 * staged source range that the plan reads (else the result depends on the
 * order of copies).  O(n^2) on purpose: it is the definition.  1 = valid. */
int32_t orc_stage_validate(const orc_copy_t *plan, int64_t n, const uint8_t *dirty_bitmap)
{
    for (int64_t a = 0; a < n; ++a) {
        if (plan[a].bytes <= 0) continue;
        const uint8_t *d0 = plan[a].dst_dev, *d1 = d0 + plan[a].bytes;
        for (int64_t b = 0; b < n; ++b) {
            if (plan[b].bytes <= 0) continue;
            if (b != a) {
                const uint8_t *e0 = plan[b].dst_dev, *e1 = e0 + plan[b].bytes;
                if (d0 < e1 && e0 < d1) return 0;
            }
            int missing = (plan[b].src_dev == NULL);
            int dirty = (!missing && dirty_bitmap && plan[b].chunk_id >= 0 &&
                         orc_bit(dirty_bitmap, plan[b].chunk_id));
            if (!missing && !dirty) {
                const uint8_t *s0 = plan[b].src_dev, *s1 = s0 + plan[b].bytes;
                if (d0 < s1 && s0 < d1) return 0;
            }
        }
    }
    return 1;
}

/* ------------------------------------------------------------------ */
/* Pre-staging while the current model serves (Sec. 4.4)                */
/* ------------------------------------------------------------------ */

static void orc_set_bit(uint8_t *bm, int64_t i, int v)
{
    if (v) bm[i >> 3] |= (uint8_t)(1u << (i & 7));
    else   bm[i >> 3] &= (uint8_t)~(1u << (i & 7));
}

/* Sec. 4.4, pre-staging: weights are written into the staging region in fixed-size
 * chunks.  For every plan entry
 * whose staging rows are not blocked (bit chunk_id of `blocked`: the rows currently
 * belong to a KV allocation), copy the authoritative host bytes into the chunk's
 * place in the staging region (src_dev), set its staged bit and clear its dirty
 * bit.  Blocked chunks are left alone and stay unstaged.
 * stats: h2d_bytes = bytes written, missing_chunks = chunks skipped,
 *        dirty_chunks = dirty bits cleared by a rewrite, d2d_bytes = 0. */
int32_t orc_prestage(const orc_copy_t *plan, int64_t n, const uint8_t *blocked, uint8_t *staged,
                     uint8_t *dirty, orc_stage_stats_t *st)
{
    orc_stage_stats_t s = {0, 0, 0, 0};
    for (int64_t k = 0; k < n; ++k) {
        const orc_copy_t *c = &plan[k];
        if (c->bytes < 0 || c->chunk_id < 0 || !c->src_dev || !c->src_host) return -1;
        if (blocked && orc_bit(blocked, c->chunk_id)) { s.missing_chunks += 1; continue; }
        memcpy((uint8_t *)c->src_dev, c->src_host, (size_t)c->bytes);
        s.h2d_bytes += c->bytes;
        if (staged) orc_set_bit(staged, c->chunk_id, 1);
        if (dirty && orc_bit(dirty, c->chunk_id)) { orc_set_bit(dirty, c->chunk_id, 0); s.dirty_chunks += 1; }
    }
    if (st) *st = s;
    return 0;
}

/* "marks a chunk dirty if a concurrent prefill allocation takes rows that overlap the
 * chunk's staging range": every STAGED chunk whose staging bytes [src_dev, +bytes)
 * intersect the allocation [alloc_base, +alloc_bytes) gets its dirty bit set.
 * Returns how many bits changed from clean to dirty. */
int64_t orc_mark_dirty(const orc_copy_t *plan, int64_t n, const uint8_t *alloc_base, int64_t alloc_bytes,
                       const uint8_t *staged, uint8_t *dirty)
{
    int64_t changed = 0;
    if (alloc_bytes <= 0) return 0;
    for (int64_t k = 0; k < n; ++k) {
        const orc_copy_t *c = &plan[k];
        if (c->bytes <= 0 || c->chunk_id < 0 || !c->src_dev) continue;
        if (staged && !orc_bit(staged, c->chunk_id)) continue;
        if (c->src_dev < alloc_base + alloc_bytes && alloc_base < c->src_dev + c->bytes) {
            if (!orc_bit(dirty, c->chunk_id)) { orc_set_bit(dirty, c->chunk_id, 1); changed += 1; }
        }
    }
    return changed;
}
