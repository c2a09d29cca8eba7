// Chained block hash and prefix match (Sec. 4.3 "cumulative prefix hash";
// App. A "Prefix reuse"; App. B "at page boundaries").
//
//   digest_k = sum_j mix64(u32(tok[kB+j]) + G*(j+1));  s_k = s_{k-1}*P + digest_k;
//   hash_k   = mix64(s_k)
//
// Up to eight pairs (a session returning) run as ONE fused launch: the CTA that finishes a
// pair's last tile also runs that pair's chain.  Larger batches use two launches:
//   1. tile kernel  -- a CTA per 2048-token tile of a pair: coalesced 16-byte token
//      loads (four tokens per thread, summed in registers), a warp-shuffle
//      segmented sum over the B/4 lanes that share a block, and the first token
//      position where the two streams differ inside the tile.
//   2. chain kernel -- a CTA per pair: the affine recurrence s -> s*P + d is
//      associative under composition, so it is evaluated as a block-wide scan
//      (thread-serial runs, shuffle scan across lanes, shared memory across warps);
//      then hash compare against the stored session's hashes, min-reductions for
//      matched_blocks and the token LCP, and the result record.
// No atomics, no inter-CTA waiting, bit-identical for any grid shape.
#include <algorithm>
#include <cstring>

#include "internal.h"
#include "prefix_common.cuh"

namespace tal {

// Work of one 2,048-token tile; returns the pair the tile belongs to.
__device__ __forceinline__ int tile_body(const PrefixParams &p) {
  __shared__ long long s_min[kTileThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  int q = 0;
  if (p.pairs) {
    q = p.tile_pair[blockIdx.x];
  } else {
    // last inline pair whose first tile is <= this tile
    for (int k = 1; k < p.n_pairs; ++k)
      if (p.inl[k].tile_off <= (int64_t)blockIdx.x) q = k;
  }
  const PairDesc pd = p.pairs ? p.pairs[q] : p.inl[q];
  const int tile_tok = p.tile_tok;
  const int64_t base = ((int64_t)blockIdx.x - pd.tile_off) * tile_tok;
  const int32_t *cont = p.cont + pd.cont_off;
  const int32_t *sess = p.sess + pd.sess_off;
  const int64_t Tmin = pd.Tc < pd.Ts ? pd.Tc : pd.Ts;
  const int B = p.B;
  const int64_t nbc = pd.Tc / B, nbs = pd.Ts / B;
  long long first_mis = kNoMismatch;

  const bool vec_ok = p.log2B >= 2 && ((((uintptr_t)cont) | ((uintptr_t)sess)) & 15) == 0;
  if (vec_ok) {
    // four consecutive tokens per thread (one 16-byte load per stream); the B/4 lanes
    // that share a block finish the sum with xor-shuffles
    const int lanes_per_block = B >> 2;
    // the position weights of this thread's four tokens never change: rounds advance by a
    // multiple of the block size
    const int j_first = (int)((base + (int64_t)tid * 4) & (B - 1));
    uint64_t wt[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) wt[e] = kG * (uint64_t)(j_first + e + 1);
    // interior tile: every token exists in both streams and every block is full, so the
    // loop carries no bounds checks at all
    const int64_t tile_end = base + tile_tok;
    const bool interior = tile_end <= Tmin && tile_end <= nbc * B && (!p.need_sess_digest || tile_end <= nbs * B);
    if (interior) {
      const int4 *c4 = (const int4 *)(cont + base) + tid;
      const int4 *s4 = (const int4 *)(sess + base) + tid;
      uint64_t *dc = p.dig_c + pd.cont_blk_off + ((base + (int64_t)tid * 4) >> p.log2B);
      uint64_t *ds = p.dig_s + pd.sess_blk_off + ((base + (int64_t)tid * 4) >> p.log2B);
      const int blocks_per_round = (kTileThreads * 4) >> p.log2B;
      const int rounds = tile_tok / (kTileThreads * 4);
      if (p.need_sess_digest) {
#pragma unroll 2
        for (int r = 0; r < rounds; ++r) {
          const int4 a = __ldg(c4 + r * kTileThreads), b = __ldg(s4 + r * kTileThreads);
          if ((a.x != b.x) | (a.y != b.y) | (a.z != b.z) | (a.w != b.w)) {
            const int e = a.x != b.x ? 0 : a.y != b.y ? 1 : a.z != b.z ? 2 : 3;
            const long long g = base + ((int64_t)r * kTileThreads + tid) * 4 + e;
            first_mis = g < first_mis ? g : first_mis;
          }
          uint64_t vc = mix64((uint64_t)(uint32_t)a.x + wt[0]) + mix64((uint64_t)(uint32_t)a.y + wt[1]) +
                        mix64((uint64_t)(uint32_t)a.z + wt[2]) + mix64((uint64_t)(uint32_t)a.w + wt[3]);
          uint64_t vs = mix64((uint64_t)(uint32_t)b.x + wt[0]) + mix64((uint64_t)(uint32_t)b.y + wt[1]) +
                        mix64((uint64_t)(uint32_t)b.z + wt[2]) + mix64((uint64_t)(uint32_t)b.w + wt[3]);
          for (int m = 1; m < lanes_per_block; m <<= 1) {
            vc += shfl_xor_u64(vc, m);
            vs += shfl_xor_u64(vs, m);
          }
          if (j_first == 0) {
            dc[r * blocks_per_round] = vc;
            ds[r * blocks_per_round] = vs;
          }
        }
      } else {
#pragma unroll 2
        for (int r = 0; r < rounds; ++r) {
          const int4 a = __ldg(c4 + r * kTileThreads), b = __ldg(s4 + r * kTileThreads);
          if ((a.x != b.x) | (a.y != b.y) | (a.z != b.z) | (a.w != b.w)) {
            const int e = a.x != b.x ? 0 : a.y != b.y ? 1 : a.z != b.z ? 2 : 3;
            const long long g = base + ((int64_t)r * kTileThreads + tid) * 4 + e;
            first_mis = g < first_mis ? g : first_mis;
          }
          uint64_t vc = mix64((uint64_t)(uint32_t)a.x + wt[0]) + mix64((uint64_t)(uint32_t)a.y + wt[1]) +
                        mix64((uint64_t)(uint32_t)a.z + wt[2]) + mix64((uint64_t)(uint32_t)a.w + wt[3]);
          for (int m = 1; m < lanes_per_block; m <<= 1) vc += shfl_xor_u64(vc, m);
          if (j_first == 0) dc[r * blocks_per_round] = vc;
        }
      }
    } else
#pragma unroll 2
    for (int r = 0; r < tile_tok / (kTileThreads * 4); ++r) {
      const int64_t g0 = base + ((int64_t)r * kTileThreads + tid) * 4;
      const int64_t k = g0 >> p.log2B;
      const int j0 = (int)(g0 & (B - 1));
      int tc[4] = {0, 0, 0, 0}, ts[4] = {0, 0, 0, 0};
      if (g0 + 4 <= pd.Tc) {
        const int4 v = __ldg((const int4 *)(cont + g0));
        tc[0] = v.x; tc[1] = v.y; tc[2] = v.z; tc[3] = v.w;
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) if (g0 + e < pd.Tc) tc[e] = __ldg(cont + g0 + e);
      }
      if (g0 + 4 <= pd.Ts) {
        const int4 v = __ldg((const int4 *)(sess + g0));
        ts[0] = v.x; ts[1] = v.y; ts[2] = v.z; ts[3] = v.w;
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) if (g0 + e < pd.Ts) ts[e] = __ldg(sess + g0 + e);
      }
      uint64_t vc = 0, vs = 0;
#pragma unroll
      for (int e = 3; e >= 0; --e)
        if (g0 + e < Tmin && tc[e] != ts[e]) first_mis = (first_mis < g0 + e) ? first_mis : g0 + e;
      const bool full_c = k < nbc, full_s = p.need_sess_digest && k < nbs;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (full_c) vc += mix64((uint64_t)(uint32_t)tc[e] + wt[e]);
        if (full_s) vs += mix64((uint64_t)(uint32_t)ts[e] + wt[e]);
      }
      for (int m = 1; m < lanes_per_block; m <<= 1) {
        vc += shfl_xor_u64(vc, m);
        if (p.need_sess_digest) vs += shfl_xor_u64(vs, m);
      }
      if (j0 == 0) {
        if (full_c) p.dig_c[pd.cont_blk_off + k] = vc;
        if (full_s) p.dig_s[pd.sess_blk_off + k] = vs;
      }
    }
  } else if (p.log2B >= 0) {
    // one token per thread per round; B consecutive lanes own one block
#pragma unroll 4
    for (int r = 0; r < tile_tok / kTileThreads; ++r) {
      const int64_t g = base + r * kTileThreads + tid;
      const int64_t k = g >> p.log2B;
      const int j = (int)(g & (B - 1));
      const uint64_t w = kG * (uint64_t)(j + 1);
      int32_t tc = 0, ts = 0;
      const bool hc = g < pd.Tc, hs = g < pd.Ts;
      if (hc) tc = __ldg(cont + g);
      if (hs) ts = __ldg(sess + g);
      if (g < Tmin && tc != ts && first_mis == kNoMismatch) first_mis = g;
      uint64_t vc = hc ? mix64((uint64_t)(uint32_t)tc + w) : 0ull;
      uint64_t vs = (p.need_sess_digest && hs) ? mix64((uint64_t)(uint32_t)ts + w) : 0ull;
      for (int m = 1; m < B; m <<= 1) {
        vc += shfl_xor_u64(vc, m);
        if (p.need_sess_digest) vs += shfl_xor_u64(vs, m);
      }
      if (j == 0) {
        if (k < nbc) p.dig_c[pd.cont_blk_off + k] = vc;
        if (p.need_sess_digest && k < nbs) p.dig_s[pd.sess_blk_off + k] = vs;
      }
    }
  } else {
    // general block size: a warp per block that STARTS inside this tile
    for (int r = 0; r < tile_tok / kTileThreads; ++r) {
      const int64_t g = base + r * kTileThreads + tid;
      if (g < Tmin && first_mis == kNoMismatch && __ldg(cont + g) != __ldg(sess + g)) first_mis = g;
    }
    const int64_t k_first = (base + B - 1) / B;
    const int64_t nb_max = nbc > nbs ? nbc : nbs;
    for (int64_t k = k_first + wid; k < nb_max && k * B < base + tile_tok; k += kTileThreads / 32) {
      const bool dc = k < nbc, ds = p.need_sess_digest && k < nbs;
      uint64_t vc = 0, vs = 0;
      for (int j = lane; j < B; j += 32) {
        const uint64_t w = kG * (uint64_t)(j + 1);
        if (dc) vc += mix64((uint64_t)(uint32_t)__ldg(cont + k * B + j) + w);
        if (ds) vs += mix64((uint64_t)(uint32_t)__ldg(sess + k * B + j) + w);
      }
      for (int m = 16; m >= 1; m >>= 1) {
        vc += shfl_xor_u64(vc, m);
        vs += shfl_xor_u64(vs, m);
      }
      if (lane == 0) {
        if (dc) p.dig_c[pd.cont_blk_off + k] = vc;
        if (ds) p.dig_s[pd.sess_blk_off + k] = vs;
      }
    }
  }

  // first mismatch inside the tile
  for (int m = 16; m >= 1; m >>= 1) {
    long long o = __shfl_xor_sync(0xffffffffu, first_mis, m);
    first_mis = o < first_mis ? o : first_mis;
  }
  if (lane == 0) s_min[wid] = first_mis;
  __syncthreads();
  if (tid == 0) {
    long long v = s_min[0];
    for (int k = 1; k < kTileThreads / 32; ++k) v = s_min[k] < v ? s_min[k] : v;
    p.tile_mis[blockIdx.x] = v;
  }
  return q;
}

__global__ void __launch_bounds__(kTileThreads) prefix_tile_kernel(const __grid_constant__ PrefixParams p) {
  (void)tile_body(p);
}

// (a1,b1) then (a2,b2):  x -> (x*a1 + b1)*a2 + b2
struct Affine2 {
  uint64_t a, bc, bs;
};
__device__ __forceinline__ Affine2 then(const Affine2 &f, const Affine2 &g) {
  return Affine2{f.a * g.a, f.bc * g.a + g.bc, f.bs * g.a + g.bs};
}

// Chain, compare and result record of one pair, by one CTA of kScanThreads threads.  Digests and
// tile results were written by other CTAs, so they are read through L2 (ld.global.cg).
template <bool DERIVE_S>
__device__ __forceinline__ void chain_body(const PrefixParams &p, const int pair) {
  __shared__ Affine2 s_warp[kScanThreads / 32];
  __shared__ uint64_t s_carry[2];
  __shared__ long long s_red[kScanThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const PairDesc pd = p.pairs ? p.pairs[pair] : p.inl[pair];
  const int B = p.B;
  const int64_t nbc = pd.Tc / B, nbs = pd.Ts / B;
  const int64_t lim = nbc < nbs ? nbc : nbs;                 // blocks that can be compared
  constexpr bool derive_s = DERIVE_S;   // compile-time: the unused stream's registers disappear
  const int64_t nb = derive_s ? (nbc > nbs ? nbc : nbs) : nbc;  // blocks to chain
  const uint64_t *dc = p.dig_c + pd.cont_blk_off;
  const uint64_t *ds = derive_s ? p.dig_s + pd.sess_blk_off : nullptr;
  const uint64_t *hs_in = p.sess_hashes ? p.sess_hashes + pd.sess_hash_off : nullptr;
  uint64_t *hc_out = p.cont_hashes_out ? p.cont_hashes_out + pd.cont_hash_off : nullptr;

  if (tid == 0) { s_carry[0] = p.seed; s_carry[1] = p.seed; }
  __syncthreads();
  long long first_bad = lim;
  // token-level first mismatch over this pair's tiles: loaded first, so the latency of these
  // reads overlaps the scan below
  long long lcp = pd.Tc < pd.Ts ? pd.Tc : pd.Ts;
  {
    const int64_t t0 = pd.tile_off, t1 = p.pairs ? p.pairs[pair + 1].tile_off : p.inl[pair + 1].tile_off;
    for (int64_t t = t0 + tid; t < t1; t += kScanThreads) {
      long long v = __ldcg(p.tile_mis + t);
      lcp = v < lcp ? v : lcp;
    }
  }

  for (int64_t chunk = 0; chunk < nb; chunk += (int64_t)kScanThreads * kScanItems) {
    const int64_t k0 = chunk + (int64_t)tid * kScanItems;
    uint64_t vc[kScanItems], vs[kScanItems], hs_st[kScanItems];
    Affine2 loc{1ull, 0ull, 0ull};
    // all loads of this thread's run are issued up front (the stored hashes too: fetched
    // inside the compare loop they would serialise behind the hash stores)
#pragma unroll
    for (int q = 0; q < kScanItems; ++q) {
      const int64_t k = k0 + q;
      vc[q] = (k < nbc) ? __ldcg(dc + k) : 0ull;
      vs[q] = (derive_s && k < nbs) ? __ldcg(ds + k) : 0ull;
      hs_st[q] = (!derive_s && k < lim) ? __ldg(hs_in + k) : 0ull;
    }
#pragma unroll
    for (int q = 0; q < kScanItems; ++q)
      if (k0 + q < nb) loc = Affine2{loc.a * kP, loc.bc * kP + vc[q], loc.bs * kP + vs[q]};
    // inclusive scan across the warp
    Affine2 inc = loc;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      Affine2 prev{shfl_up_u64(inc.a, d), shfl_up_u64(inc.bc, d), shfl_up_u64(inc.bs, d)};
      if (lane >= d) inc = then(prev, inc);
    }
    if (lane == 31) s_warp[wid] = inc;
    // exclusive prefix inside the warp
    Affine2 exc{shfl_up_u64(inc.a, 1), shfl_up_u64(inc.bc, 1), shfl_up_u64(inc.bs, 1)};
    if (lane == 0) exc = Affine2{1ull, 0ull, 0ull};
    __syncthreads();
    Affine2 before{1ull, 0ull, 0ull};
    for (int w = 0; w < wid; ++w) before = then(before, s_warp[w]);
    before = then(before, exc);
    uint64_t sc = s_carry[0] * before.a + before.bc;
    uint64_t ss = s_carry[1] * before.a + before.bs;
#pragma unroll
    for (int q = 0; q < kScanItems; ++q) {
      const int64_t k = k0 + q;
      if (k < nb) {
        sc = sc * kP + vc[q];
        ss = ss * kP + vs[q];
        const uint64_t hc = mix64(sc);
        if (k < nbc && hc_out) hc_out[k] = hc;
        if (k < lim) {
          const uint64_t hs = derive_s ? mix64(ss) : hs_st[q];
          if (hs != hc && k < first_bad) first_bad = k;
        }
      }
    }
    __syncthreads();                       // everyone has read s_carry and s_warp
    if (tid == kScanThreads - 1) { s_carry[0] = sc; s_carry[1] = ss; }
    __syncthreads();
  }

  for (int m = 16; m >= 1; m >>= 1) {
    long long o = __shfl_xor_sync(0xffffffffu, lcp, m);
    lcp = o < lcp ? o : lcp;
    long long o2 = __shfl_xor_sync(0xffffffffu, first_bad, m);
    first_bad = o2 < first_bad ? o2 : first_bad;
  }
  __syncthreads();
  if (lane == 0) s_red[wid] = lcp;
  __syncthreads();
  if (tid == 0) for (int w = 1; w < kScanThreads / 32; ++w) lcp = s_red[w] < lcp ? s_red[w] : lcp;
  __syncthreads();
  if (lane == 0) s_red[wid] = first_bad;
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kScanThreads / 32; ++w) first_bad = s_red[w] < first_bad ? s_red[w] : first_bad;
    if (p.results) {
      const long long lcp_blocks = lcp / B;
      const long long tok_blocks = lcp_blocks < lim ? lcp_blocks : lim;
      talaria_match_t r;
      r.lcp_tokens = lcp;
      r.matched_blocks = first_bad;
      r.reusable_tokens = (long long)B * (first_bad < lcp_blocks ? first_bad : lcp_blocks);
      r.hash_token_disagree = (first_bad != tok_blocks) ? 1 : 0;
      r.reserved = 0;
      p.results[pair] = r;
    }
  }
}

__global__ void __launch_bounds__(kScanThreads) prefix_chain_kernel(const __grid_constant__ PrefixParams p) {
  // Launched as a programmatic dependent of the tile kernel: CTAs may be resident early,
  // and this wait returns once the tile kernel has finished and its writes are visible.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (p.need_sess_digest) chain_body<true>(p, (int)blockIdx.x);
  else                    chain_body<false>(p, (int)blockIdx.x);
}

// One launch for a handful of pairs (a session returning): every CTA does its tile, and the
// CTA that finishes a pair's last tile also runs that pair's chain.  Completion is counted with
// one atomic per CTA; nobody waits for anybody.  The counter is put back to zero by the CTA
// that saw the last arrival, so the next call finds it clean.
static_assert(kTileThreads == kScanThreads, "the fused kernel runs both bodies with one block size");
__global__ void __launch_bounds__(kTileThreads) prefix_fused_kernel(const __grid_constant__ PrefixParams p) {
  __shared__ int s_last;
  const int q = tile_body(p);
  __threadfence();                       // this thread's digests / tile result are visible device-wide
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned tiles_q = (unsigned)(p.inl[q + 1].tile_off - p.inl[q].tile_off);
    const unsigned prev = atomicAdd(&p.counters[q], 1u);
    s_last = (prev + 1 == tiles_q);
    if (s_last) p.counters[q] = 0;
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    if (p.need_sess_digest) chain_body<true>(p, q);
    else                    chain_body<false>(p, q);
  }
}

// The chain kernel is launched with programmatic stream serialization so its launch latency
// overlaps the tile kernel; it blocks in griddepcontrol.wait until the tile kernel is done.
static cudaError_t launch_chain(const PrefixParams &p, int n_pairs, cudaStream_t stream) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)n_pairs);
  cfg.blockDim = dim3(kScanThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, prefix_chain_kernel, p);
}

// Batches with fewer pairs than SMs: the one-CTA-per-pair kernel takes as long as its longest pair
// (measured 8.5 us + 0.285 us per 1,024 tokens for a CTA that has its SM to itself), the tile and
// chain kernels as long as the whole batch spread over the GPU (21 us + 3.2 us per million token
// positions).  Measured at 16 - 147 pairs of 32,768 - 131,072 tokens; the faster one is predicted
// right or within 3 us everywhere in that range.
static bool pair_kernel_is_faster(int64_t longest, int64_t positions) {
  return 8.5 + 0.285 * (double)longest / 1024.0 <= 21.0 + 3.2 * (double)positions / 1e6;
}

// Host side: validates the pairs, builds the pair table, sizes scratch, launches.
static talaria_status_t prefix_launch_specs(talaria_ctx *ctx, int32_t n_pairs, const PairSpec *specs,
                                            const int32_t *d_cont, const int32_t *d_sess,
                                            const uint64_t *d_sess_hashes, int32_t B, uint64_t seed,
                                            uint64_t *d_cont_hashes, talaria_match_t *d_results,
                                            cudaStream_t stream) {
  if (n_pairs < 0 || B <= 0) return TALARIA_ERR_INVALID_ARG;
  if (n_pairs == 0) return TALARIA_OK;
  if (!specs) return TALARIA_ERR_INVALID_ARG;
  // few pairs: descriptors ride in the kernel parameters (no upload); otherwise a
  // pinned slot holds the pair table followed by one pair index per tile
  const bool inl = n_pairs <= kInlinePairs;
  PrefixParams p{};
  std::vector<PairDesc> big;
  PairDesc *pd = p.inl;
  int log2B = -1;
  if (B <= 32 && (B & (B - 1)) == 0)
    while ((1 << ++log2B) < B) {}
  // More than a handful of pairs: one CTA per pair, one launch, no global scratch -- when there is
  // a pair for every SM, or when no pair is so long that its one CTA would outlast the whole batch
  // spread over the GPU.
  int64_t longest = 0, positions = 0, any_c = 0, any_s = 0;
  for (int32_t q = 0; q < n_pairs; ++q) {
    const PairSpec &sp = specs[q];
    if (sp.Tc < 0 || sp.Ts < 0 || sp.cont_off < 0 || sp.sess_off < 0 || sp.cont_hash_off < 0 || sp.sess_hash_off < 0)
      return TALARIA_ERR_INVALID_ARG;
    const int64_t t = std::max(sp.Tc, sp.Ts);
    longest = std::max(longest, t);
    positions += t;
    any_c |= sp.Tc;
    any_s |= sp.Ts;
  }
  if (any_c && !d_cont) return TALARIA_ERR_INVALID_ARG;
  if (any_s && !d_sess) return TALARIA_ERR_INVALID_ARG;
  if (!inl && log2B >= 2 && (n_pairs >= ctx->sm_count || pair_kernel_is_faster(longest, positions)))
    return pair_launch(ctx, n_pairs, specs, d_cont, d_sess, d_sess_hashes, B, log2B, seed, d_cont_hashes, d_results,
                       stream);
  if (!inl) {
    big.resize((size_t)n_pairs + 1);
    pd = big.data();
  }
  // A handful of pairs run as ONE fused launch (every pair then owns at least one tile, so some
  // CTA always finishes it); batches in between use a tile kernel and a chain kernel.
  bool fused = inl;
  int64_t cb = 0, sb = 0, tiles = 0;
  int tile_tok = kTileTok;
  for (int pass = 0; pass < 2; ++pass) {
    cb = sb = tiles = 0;
    tile_tok = fused ? kTileTok : kBatchTileTok;
    for (int32_t q = 0; q < n_pairs; ++q) {
      const PairSpec &sp = specs[q];
      const int64_t Tc = sp.Tc, Ts = sp.Ts;
      pd[q] = PairDesc{sp.cont_off, sp.sess_off, Tc, Ts, cb, sb, tiles, sp.cont_hash_off, sp.sess_hash_off};
      cb += Tc / B;
      sb += Ts / B;
      const int64_t t = (std::max(Tc, Ts) + tile_tok - 1) / tile_tok;
      tiles += fused ? std::max<int64_t>(t, 1) : t;
    }
    if (!fused || tiles <= kFusedMaxTiles) break;
    fused = false;                        // too much work for one wave of CTAs: lay out again, unfused
  }
  pd[n_pairs] = PairDesc{0, 0, 0, 0, cb, sb, tiles, 0, 0};      // the totals
  if (tiles > 0x7fffffffll) return TALARIA_ERR_INVALID_ARG;

  // The scratch (digests, tile results, counters) is shared by all calls of this context:
  // a call on another stream must not start before the previous call's kernels are done.
  if (ctx->prefix_busy && ctx->prefix_stream != stream) TAL_CUDA(ctx, cudaStreamWaitEvent(stream, ctx->prefix_done, 0));

  const bool derive = (d_sess_hashes == nullptr);
  const size_t dig_c_bytes = (size_t)cb * 8, dig_s_bytes = derive ? (size_t)sb * 8 : 0;
  const size_t need = dig_c_bytes + dig_s_bytes + (size_t)tiles * 8 + 64;
  TAL_TRY(grow(ctx, &ctx->prefix_scratch, need));
  DescSlot *slot = nullptr;
  if (!inl) {
    const size_t pair_bytes = ((size_t)(n_pairs + 1) * sizeof(PairDesc) + 15) & ~(size_t)15;
    const size_t desc_bytes = pair_bytes + (size_t)tiles * sizeof(int32_t);
    TAL_TRY(acquire_slot(ctx, desc_bytes, &slot));
    memcpy(slot->h, big.data(), (size_t)(n_pairs + 1) * sizeof(PairDesc));
    int32_t *tp = (int32_t *)(slot->h + pair_bytes);
    for (int32_t q = 0; q < n_pairs; ++q)
      for (int64_t t = big[q].tile_off; t < big[q + 1].tile_off; ++t) tp[t] = q;
    TAL_TRY(upload_slot(ctx, slot, desc_bytes, stream));
    p.pairs = (const PairDesc *)slot->d;
    p.tile_pair = (const int32_t *)(slot->d + pair_bytes);
  }
  p.n_pairs = n_pairs;
  p.B = B;
  p.log2B = log2B;
  p.need_sess_digest = derive ? 1 : 0;
  p.tile_tok = tile_tok;
  p.cont = d_cont;
  p.sess = d_sess;
  p.dig_c = (uint64_t *)ctx->prefix_scratch.p;
  p.dig_s = (uint64_t *)(ctx->prefix_scratch.p + dig_c_bytes);
  p.tile_mis = (long long *)(ctx->prefix_scratch.p + dig_c_bytes + dig_s_bytes);
  p.sess_hashes = d_sess_hashes;
  p.cont_hashes_out = d_cont_hashes;
  p.results = d_results;
  p.seed = seed;
  p.counters = ctx->prefix_counters;
  if (fused) {
    prefix_fused_kernel<<<(unsigned)tiles, kTileThreads, 0, stream>>>(p);
    TAL_CUDA(ctx, cudaGetLastError());
    ctx->counters.kernel_launches++;
  } else {
    if (tiles > 0) {
      prefix_tile_kernel<<<(unsigned)tiles, kTileThreads, 0, stream>>>(p);
      TAL_CUDA(ctx, cudaGetLastError());
      ctx->counters.kernel_launches++;
    }
    TAL_CUDA(ctx, launch_chain(p, n_pairs, stream));
    ctx->counters.kernel_launches++;
  }
  TAL_CUDA(ctx, cudaEventRecord(ctx->prefix_done, stream));
  ctx->prefix_busy = true;
  ctx->prefix_stream = stream;
  return slot ? release_slot(ctx, slot, stream) : TALARIA_OK;
}

// The same for pairs laid out back to back: pair q spans [off[q], off[q+1]) of its token array and
// its hashes follow those of the pairs before it.
static talaria_status_t prefix_launch(talaria_ctx *ctx, int32_t n_pairs, const int32_t *d_cont,
                                      const int64_t *cont_off, const int32_t *d_sess,
                                      const int64_t *sess_off, const uint64_t *d_sess_hashes, int32_t B,
                                      uint64_t seed, uint64_t *d_cont_hashes, talaria_match_t *d_results,
                                      cudaStream_t stream) {
  if (n_pairs < 0 || B <= 0) return TALARIA_ERR_INVALID_ARG;
  if (n_pairs == 0) return TALARIA_OK;
  if (!cont_off || !sess_off) return TALARIA_ERR_INVALID_ARG;
  PairSpec few[kInlinePairs];
  std::vector<PairSpec> many;
  PairSpec *specs = few;
  if (n_pairs > kInlinePairs) {
    many.resize((size_t)n_pairs);
    specs = many.data();
  }
  int64_t cb = 0, sb = 0;
  for (int32_t q = 0; q < n_pairs; ++q) {
    const int64_t Tc = cont_off[q + 1] - cont_off[q], Ts = sess_off[q + 1] - sess_off[q];
    if (Tc < 0 || Ts < 0 || cont_off[q] < 0 || sess_off[q] < 0) return TALARIA_ERR_INVALID_ARG;
    specs[q] = PairSpec{cont_off[q], Tc, sess_off[q], Ts, cb, sb};
    cb += Tc / B;
    sb += Ts / B;
  }
  return prefix_launch_specs(ctx, n_pairs, specs, d_cont, d_sess, d_sess_hashes, B, seed, d_cont_hashes, d_results,
                             stream);
}

}  // namespace tal

using namespace tal;

#define TAL_ENTER(ctx)                                   \
  if (!(ctx)) return TALARIA_ERR_INVALID_ARG;            \
  std::lock_guard<std::mutex> lk__((ctx)->mu);           \
  DeviceGuard guard__((ctx)->device);                    \
  if (!guard__.ok) return TALARIA_ERR_CUDA

extern "C" talaria_status_t talaria_block_hash(talaria_ctx *ctx, const int32_t *d_tokens, int64_t n_tokens,
                                               int32_t block_tokens, uint64_t seed,
                                               uint64_t *d_hashes_out, void *stream) {
  TAL_ENTER(ctx);
  if (n_tokens < 0 || block_tokens <= 0) return TALARIA_ERR_INVALID_ARG;
  if (n_tokens / block_tokens == 0) return TALARIA_OK;
  if (!d_tokens || !d_hashes_out) return TALARIA_ERR_INVALID_ARG;
  const int64_t co[2] = {0, n_tokens}, so[2] = {0, 0};
  return prefix_launch(ctx, 1, d_tokens, co, d_tokens, so, nullptr, block_tokens, seed, d_hashes_out,
                       nullptr, (cudaStream_t)stream);
}

extern "C" talaria_status_t talaria_prefix_match(talaria_ctx *ctx, int32_t n_pairs,
                                                 const int32_t *d_cont_tokens, const int64_t *cont_offsets,
                                                 const int32_t *d_sess_tokens, const int64_t *sess_offsets,
                                                 const uint64_t *d_sess_hashes, int32_t block_tokens,
                                                 uint64_t seed, uint64_t *d_cont_hashes_out,
                                                 talaria_match_t *d_results, void *stream) {
  TAL_ENTER(ctx);
  if (n_pairs > 0 && !d_results) return TALARIA_ERR_INVALID_ARG;
  return prefix_launch(ctx, n_pairs, d_cont_tokens, cont_offsets, d_sess_tokens, sess_offsets,
                       d_sess_hashes, block_tokens, seed, d_cont_hashes_out, d_results,
                       (cudaStream_t)stream);
}

extern "C" talaria_status_t talaria_prefix_match_host(talaria_ctx *ctx, int32_t n_pairs,
                                                      const int32_t *h_cont, const int64_t *cont_offsets,
                                                      const int32_t *h_sess, const int64_t *sess_offsets,
                                                      const uint64_t *h_sess_hashes, int32_t B,
                                                      uint64_t seed, uint64_t *h_cont_hashes_out,
                                                      talaria_match_t *h_results, void *stream_) {
  TAL_ENTER(ctx);
  cudaStream_t stream = (cudaStream_t)stream_;
  if (n_pairs < 0 || B <= 0) return TALARIA_ERR_INVALID_ARG;
  if (n_pairs == 0) return TALARIA_OK;
  if (!cont_offsets || !sess_offsets || !h_results) return TALARIA_ERR_INVALID_ARG;
  for (int32_t q = 0; q < n_pairs; ++q)
    if (cont_offsets[q + 1] < cont_offsets[q] || sess_offsets[q + 1] < sess_offsets[q] || cont_offsets[q] < 0 ||
        sess_offsets[q] < 0)
      return TALARIA_ERR_INVALID_ARG;
  if ((cont_offsets[n_pairs] > cont_offsets[0] && !h_cont) || (sess_offsets[n_pairs] > sess_offsets[0] && !h_sess))
    return TALARIA_ERR_INVALID_ARG;
  auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
  const size_t cap = ctx->host_tok.cap;
  char *const dev = ctx->host_tok.p, *const pin = ctx->match_pin;
  // a resident match on another stream may still be spreading prompts out of the device staging
  if (ctx->stage_busy && ctx->stage_stream != stream) TAL_CUDA(ctx, cudaStreamWaitEvent(stream, ctx->stage_free, 0));
  std::vector<int64_t> co, so;
  int64_t sb_before = 0, cb_before = 0;           // blocks of the pairs already done (positions in the users' hash arrays)
  for (int32_t q0 = 0; q0 < n_pairs;) {
    // the longest run of whole pairs whose inputs and outputs fit the staging
    int32_t q1 = q0;
    int64_t nc = 0, ns = 0, cb = 0, sb = 0;
    while (q1 < n_pairs) {
      const int64_t Tc = cont_offsets[q1 + 1] - cont_offsets[q1], Ts = sess_offsets[q1 + 1] - sess_offsets[q1];
      const size_t need = up((size_t)(nc + Tc) * 4) + up((size_t)(ns + Ts) * 4) +
                          up(h_sess_hashes ? (size_t)(sb + Ts / B) * 8 : 0) + up((size_t)(cb + Tc / B) * 8) +
                          up((size_t)(q1 + 1 - q0) * sizeof(talaria_match_t));
      if (need > cap) break;
      nc += Tc; ns += Ts; cb += Tc / B; sb += Ts / B;
      ++q1;
    }
    if (q1 == q0) return TALARIA_ERR_EXTENT;       // one pair alone is larger than the staging
    const int32_t m = q1 - q0;
    const size_t o_cont = 0, o_sess = o_cont + up((size_t)nc * 4), o_sh = o_sess + up((size_t)ns * 4),
                 o_ch = o_sh + up(h_sess_hashes ? (size_t)sb * 8 : 0), o_res = o_ch + up((size_t)cb * 8);
    const int64_t c0 = cont_offsets[q0], s0 = sess_offsets[q0];
    co.resize((size_t)m + 1);
    so.resize((size_t)m + 1);
    for (int32_t q = 0; q <= m; ++q) {
      co[(size_t)q] = cont_offsets[q0 + q] - c0;
      so[(size_t)q] = sess_offsets[q0 + q] - s0;
    }
    // gather the inputs into the pinned staging; one copy takes them to the device
    if (nc) memcpy(pin + o_cont, h_cont + c0, (size_t)nc * 4);
    if (ns) memcpy(pin + o_sess, h_sess + s0, (size_t)ns * 4);
    if (h_sess_hashes && sb) memcpy(pin + o_sh, h_sess_hashes + sb_before, (size_t)sb * 8);
    if (ctx->timing && q0 == 0) {      // op 4: from the first copy to the last kernel, host-side packing excluded
      ctx->tm_op = 4;
      ctx->tm_d2d = ctx->tm_h2d = false;
      TAL_CUDA(ctx, cudaEventRecord(ctx->tm[0], stream));
    }
    if (o_ch) {
      TAL_CUDA(ctx, cudaMemcpyAsync(dev, pin, o_ch, cudaMemcpyHostToDevice, stream));
      ctx->counters.memcpy_calls++;
    }
    // Hashes and results are written by the kernels straight into the pinned staging (through its
    // device mapping): a few kilobytes of posted writes, and no device-to-host copy that would
    // queue behind bulk checkpoint traffic on the copy engine.
    char *const pin_dev = ctx->match_pin_dev;
    TAL_TRY(prefix_launch(ctx, m, (const int32_t *)(dev + o_cont), co.data(), (const int32_t *)(dev + o_sess),
                          so.data(), h_sess_hashes ? (const uint64_t *)(dev + o_sh) : nullptr, B, seed,
                          (h_cont_hashes_out && cb) ? (uint64_t *)(pin_dev + o_ch) : nullptr,
                          (talaria_match_t *)(pin_dev + o_res), stream));
    if (ctx->timing) TAL_CUDA(ctx, cudaEventRecord(ctx->tm[1], stream));
    TAL_CUDA(ctx, cudaStreamSynchronize(stream));
    if (h_cont_hashes_out && cb) memcpy(h_cont_hashes_out + cb_before, pin + o_ch, (size_t)cb * 8);
    memcpy(h_results + q0, pin + o_res, (size_t)m * sizeof(talaria_match_t));
    sb_before += sb;
    cb_before += cb;
    q0 = q1;
  }
  return TALARIA_OK;
}


namespace tal {

// Prompts out of the device staging into their places in the caller's token array.
constexpr int kSpreadItems = 64;
struct SpreadParams {
  const int32_t *src;
  int32_t *dst;
  int32_t n;
  int64_t src_off[kSpreadItems], dst_off[kSpreadItems], count[kSpreadItems];   // in elements
};
__global__ void __launch_bounds__(256) resident_spread_kernel(const __grid_constant__ SpreadParams p) {
  const int it = blockIdx.y;
  const int32_t *src = p.src + p.src_off[it];
  int32_t *dst = p.dst + p.dst_off[it];
  const int64_t n = p.count[it], step = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += step) dst[i] = __ldg(src + i);
}

}  // namespace tal

// Match against streams that live on the device (Sec. 4.3: the instance keeps what it knows of a
// session; App. A: the new prompt is compared with it).  Only the new prompt crosses the host
// link, and it is left where the next call will find it as the stored stream.
extern "C" talaria_status_t talaria_prefix_match_resident(talaria_ctx *ctx, int32_t n_pairs,
                                                          const talaria_resident_pair_t *pairs, int32_t *d_tokens,
                                                          int64_t tokens_capacity, uint64_t *d_hashes,
                                                          int64_t hashes_capacity, int32_t B, uint64_t seed,
                                                          talaria_match_t *h_results, void *stream_) {
  TAL_ENTER(ctx);
  cudaStream_t stream = (cudaStream_t)stream_;
  if (n_pairs < 0 || B <= 0 || tokens_capacity < 0 || hashes_capacity < 0) return TALARIA_ERR_INVALID_ARG;
  if (n_pairs == 0) return TALARIA_OK;
  if (!pairs || !h_results) return TALARIA_ERR_INVALID_ARG;
  // ranges written (prompts, their hashes) and read (stored streams, stored hashes), as [lo, hi)
  struct Range { int64_t lo, hi; };
  std::vector<Range> wt, rt, wh, rh;
  bool any_stored = false, any_derived = false;
  for (int32_t q = 0; q < n_pairs; ++q) {
    const talaria_resident_pair_t &r = pairs[q];
    if (r.cont_tokens < 0 || r.sess_tokens < 0 || (r.cont_tokens > 0 && !r.h_cont_tokens)) return TALARIA_ERR_INVALID_ARG;
    const int64_t nbc = r.cont_tokens / B, nbs = r.sess_tokens / B;
    if (r.cont_slot < 0 || r.cont_slot > tokens_capacity - r.cont_tokens) return TALARIA_ERR_EXTENT;
    if (r.sess_tokens > 0 && (r.sess_slot < 0 || r.sess_slot > tokens_capacity - r.sess_tokens)) return TALARIA_ERR_EXTENT;
    if (nbc > 0 && (r.cont_hash_slot < 0 || r.cont_hash_slot > hashes_capacity - nbc)) return TALARIA_ERR_EXTENT;
    if (nbs > 0) {
      if (r.sess_hash_slot < 0) {
        any_derived = true;
      } else {
        if (r.sess_hash_slot > hashes_capacity - nbs) return TALARIA_ERR_EXTENT;
        any_stored = true;
        rh.push_back(Range{r.sess_hash_slot, r.sess_hash_slot + nbs});
      }
    }
    if (r.cont_tokens > 0) wt.push_back(Range{r.cont_slot, r.cont_slot + r.cont_tokens});
    if (r.sess_tokens > 0) rt.push_back(Range{r.sess_slot, r.sess_slot + r.sess_tokens});
    if (nbc > 0) wh.push_back(Range{r.cont_hash_slot, r.cont_hash_slot + nbc});
  }
  if (any_stored && any_derived) return TALARIA_ERR_INVALID_ARG;      // one mode per call
  // a prompt (or its hashes) must not land on another prompt or on anything this call still reads
  auto clash = [](std::vector<Range> &w, const std::vector<Range> &r) {
    std::sort(w.begin(), w.end(), [](const Range &a, const Range &b) { return a.lo < b.lo; });
    for (size_t i = 1; i < w.size(); ++i)
      if (w[i].lo < w[i - 1].hi) return true;
    for (const Range &x : r) {
      auto it = std::upper_bound(w.begin(), w.end(), x.lo, [](int64_t v, const Range &a) { return v < a.hi; });
      if (it != w.end() && it->lo < x.hi) return true;
    }
    return false;
  };
  if (clash(wt, rt) || clash(wh, rh)) return TALARIA_ERR_OVERLAP;
  if ((!wt.empty() || !rt.empty()) && !d_tokens) return TALARIA_ERR_INVALID_ARG;
  if ((!wh.empty() || !rh.empty()) && !d_hashes) return TALARIA_ERR_INVALID_ARG;
  if (ctx->cfg.validate) {
    if (d_tokens && tokens_capacity) TAL_TRY(require_device_range(ctx, d_tokens, tokens_capacity * 4));
    if (d_hashes && hashes_capacity) TAL_TRY(require_device_range(ctx, d_hashes, hashes_capacity * 8));
  }

  auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
  const size_t cap = ctx->host_tok.cap;
  char *const pin = ctx->match_pin, *const pin_dev = ctx->match_pin_dev;
  std::vector<PairSpec> specs;
  if (ctx->stage_busy && ctx->stage_stream != stream) TAL_CUDA(ctx, cudaStreamWaitEvent(stream, ctx->stage_free, 0));
  for (int32_t q0 = 0; q0 < n_pairs;) {
    // the longest run of whole pairs whose prompts and result records fit the pinned staging
    int32_t q1 = q0;
    size_t bytes = 0;
    while (q1 < n_pairs) {
      const size_t need = bytes + up((size_t)pairs[q1].cont_tokens * 4) + up((size_t)(q1 + 1 - q0) * sizeof(talaria_match_t));
      if (need > cap) break;
      bytes += up((size_t)pairs[q1].cont_tokens * 4);
      ++q1;
    }
    if (q1 == q0) return TALARIA_ERR_EXTENT;       // one prompt alone is larger than the staging
    const int32_t m = q1 - q0;
    const size_t o_res = bytes;
    specs.resize((size_t)m);
    // Every command the GPU fetches costs a round trip on the host link, and several times that
    // while a checkpoint keeps the link's other direction full (measured: +40 to +65 us per copy
    // or launch).  So the call's critical path is two commands: ONE copy takes the packed prompts
    // to the device staging and the match kernels read them there.  Spreading them to their places
    // in the caller's array comes after the kernels and is not waited for.
    size_t at = 0;
    int32_t n_spread = 0;
    for (int32_t q = q0; q < q1; ++q) {
      const talaria_resident_pair_t &r = pairs[q];
      specs[(size_t)(q - q0)] = PairSpec{(int64_t)(at / 4), r.cont_tokens, r.sess_tokens > 0 ? r.sess_slot : 0, r.sess_tokens,
                                         r.cont_tokens / B > 0 ? r.cont_hash_slot : 0,
                                         (any_stored && r.sess_tokens / B > 0) ? r.sess_hash_slot : 0};
      if (r.cont_tokens > 0) {
        memcpy(pin + at, r.h_cont_tokens, (size_t)r.cont_tokens * 4);
        at += up((size_t)r.cont_tokens * 4);
        ++n_spread;
      }
    }
    if (ctx->timing && q0 == 0) {      // op 4: from the first copy to the last kernel, host-side packing excluded
      ctx->tm_op = 4;
      ctx->tm_d2d = ctx->tm_h2d = false;
      TAL_CUDA(ctx, cudaEventRecord(ctx->tm[0], stream));
    }
    if (at) {
      TAL_CUDA(ctx, cudaMemcpyAsync(ctx->host_tok.p, pin, at, cudaMemcpyHostToDevice, stream));
      ctx->counters.memcpy_calls++;
    }
    TAL_TRY(prefix_launch_specs(ctx, m, specs.data(), (const int32_t *)ctx->host_tok.p, d_tokens,
                                any_stored ? d_hashes : nullptr, B, seed, d_hashes,
                                (talaria_match_t *)(pin_dev + o_res), stream));
    if (ctx->timing) TAL_CUDA(ctx, cudaEventRecord(ctx->tm[1], stream));
    TAL_CUDA(ctx, cudaEventRecord(ctx->match_done, stream));
    for (int32_t q = q0; q < q1 && n_spread > 0;) {
      SpreadParams sp{};
      sp.src = (const int32_t *)ctx->host_tok.p;
      sp.dst = d_tokens;
      int64_t longest = 0;
      for (; q < q1 && sp.n < kSpreadItems; ++q) {
        if (pairs[q].cont_tokens == 0) continue;
        sp.src_off[sp.n] = specs[(size_t)(q - q0)].cont_off;
        sp.dst_off[sp.n] = pairs[q].cont_slot;
        sp.count[sp.n] = pairs[q].cont_tokens;
        longest = std::max(longest, pairs[q].cont_tokens);
        ++sp.n;
      }
      if (sp.n == 0) break;
      const unsigned gx = (unsigned)std::min<int64_t>((longest + 1023) / 1024, 64);
      resident_spread_kernel<<<dim3(gx, (unsigned)sp.n), 256, 0, stream>>>(sp);
      TAL_CUDA(ctx, cudaGetLastError());
      ctx->counters.kernel_launches++;
    }
    TAL_CUDA(ctx, cudaEventRecord(ctx->stage_free, stream));
    ctx->stage_busy = true;
    ctx->stage_stream = stream;
    // the records are complete once the match kernels are; a further round reuses the pinned
    // staging, whose copy to the device precedes those kernels
    TAL_CUDA(ctx, cudaEventSynchronize(ctx->match_done));
    memcpy(h_results + q0, pin + o_res, (size_t)m * sizeof(talaria_match_t));
    q0 = q1;
  }
  return TALARIA_OK;
}


// ---------------------------------------------------------------------------
// Prefix match without any allocation.
//
// Same two kernels as talaria_prefix_match, but the digests and per-tile mismatch
// positions live in a fixed array that is part of the loaded library image, and
// the pair descriptors travel in the kernel parameters.  Nothing is allocated on
// the device or on the host, no context is needed, and no copy is issued.
namespace tal {

constexpr int64_t kStaticWords = 131072;   // 1 MiB of scratch: 8 bytes per block digest / tile
static __device__ __align__(256) unsigned long long g_static_scratch[kStaticWords];

constexpr int kStaticMaxDevices = 64;
static std::mutex g_static_mu;
static unsigned long long *g_static_addr[kStaticMaxDevices];   // device address, per device

// The array's name is only a host-side handle here; the address a kernel can use has
// to be asked for, once per device, with that device current.  Called with g_static_mu held.
static talaria_status_t static_scratch_address(unsigned long long **out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return TALARIA_ERR_CUDA;
  }
  if (dev < 0 || dev >= kStaticMaxDevices) return TALARIA_ERR_INVALID_ARG;
  if (!g_static_addr[dev]) {
    void *ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess || !ptr) {
      (void)cudaGetLastError();
      return TALARIA_ERR_CUDA;
    }
    g_static_addr[dev] = (unsigned long long *)ptr;
  }
  *out = g_static_addr[dev];
  return TALARIA_OK;
}

}  // namespace tal

extern "C" talaria_status_t talaria_prefix_match_static(int32_t n_pairs, const int32_t *d_cont_tokens,
                                                        const int64_t *cont_offsets,
                                                        const int32_t *d_sess_tokens,
                                                        const int64_t *sess_offsets,
                                                        const uint64_t *d_sess_hashes, int32_t block_tokens,
                                                        uint64_t seed, uint64_t *d_cont_hashes_out,
                                                        talaria_match_t *d_results, void *stream) {
  const int32_t B = block_tokens;
  if (n_pairs < 0 || B <= 0) return TALARIA_ERR_INVALID_ARG;
  if (n_pairs == 0) return TALARIA_OK;
  if (n_pairs > kInlinePairs) return TALARIA_ERR_EXTENT;
  if (!cont_offsets || !sess_offsets || !d_results) return TALARIA_ERR_INVALID_ARG;
  PrefixParams p{};
  int64_t cb = 0, sb = 0, tiles = 0;
  for (int32_t q = 0; q < n_pairs; ++q) {
    const int64_t Tc = cont_offsets[q + 1] - cont_offsets[q], Ts = sess_offsets[q + 1] - sess_offsets[q];
    if (Tc < 0 || Ts < 0 || cont_offsets[q] < 0 || sess_offsets[q] < 0) return TALARIA_ERR_INVALID_ARG;
    p.inl[q] = PairDesc{cont_offsets[q], sess_offsets[q], Tc, Ts, cb, sb, tiles, cb, sb};
    cb += Tc / B;
    sb += Ts / B;
    tiles += (std::max(Tc, Ts) + kTileTok - 1) / kTileTok;
  }
  p.inl[n_pairs] = PairDesc{0, 0, 0, 0, cb, sb, tiles, 0, 0};
  if (cont_offsets[n_pairs] > cont_offsets[0] && !d_cont_tokens) return TALARIA_ERR_INVALID_ARG;
  if (sess_offsets[n_pairs] > sess_offsets[0] && !d_sess_tokens) return TALARIA_ERR_INVALID_ARG;
  const bool derive = (d_sess_hashes == nullptr);
  const int64_t words = cb + (derive ? sb : 0) + tiles;
  if (words > kStaticWords) return TALARIA_ERR_EXTENT;   // beyond the built-in scratch
  // One host mutex (it allocates nothing) covers the address lookup and BOTH launches: the chain
  // kernel is a programmatic dependent of the tile kernel enqueued just before it, so two host
  // threads must not interleave their launches, not even on one stream.
  std::lock_guard<std::mutex> lk(g_static_mu);
  unsigned long long *scratch = nullptr;
  TAL_TRY(static_scratch_address(&scratch));
  p.pairs = nullptr;
  p.tile_pair = nullptr;
  p.n_pairs = n_pairs;
  p.B = B;
  p.log2B = -1;
  if (B <= 32 && (B & (B - 1)) == 0) {
    int l = 0;
    while ((1 << l) < B) ++l;
    p.log2B = l;
  }
  p.need_sess_digest = derive ? 1 : 0;
  p.tile_tok = kTileTok;
  p.cont = d_cont_tokens;
  p.sess = d_sess_tokens;
  // Every word that is read is written earlier in the same call (digests of full
  // blocks and one mismatch position per tile), so nothing has to start at zero.
  p.dig_c = (uint64_t *)scratch;
  p.dig_s = (uint64_t *)scratch + cb;
  p.tile_mis = (long long *)(scratch + cb + (derive ? sb : 0));
  p.sess_hashes = d_sess_hashes;
  p.cont_hashes_out = d_cont_hashes_out;
  p.results = d_results;
  p.seed = seed;
  cudaStream_t st = (cudaStream_t)stream;
  if (tiles > 0) {
    prefix_tile_kernel<<<(unsigned)tiles, kTileThreads, 0, st>>>(p);
    if (cudaGetLastError() != cudaSuccess) return TALARIA_ERR_CUDA;
  }
  if (launch_chain(p, n_pairs, st) != cudaSuccess) {
    (void)cudaGetLastError();
    return TALARIA_ERR_CUDA;
  }
  return TALARIA_OK;
}
