// Prefix match of a large batch (Sec. 4.3 cumulative hash at page boundaries; App. A token
// LCP): one CTA per pair, one launch, nothing written to global scratch.
//
// Only the continuation is hashed.  The CTA walks its pair in chunks of 1,024 blocks.  Per chunk:
//   (1) every thread hashes whole blocks of the continuation, one block per round, four rounds:
//       the position weights G*(j+1) are compile-time immediates (the kernel is instantiated
//       per block size), a block's digest is one thread's running sum (no shuffles), tokens
//       arrive as 16-byte loads kept two quads ahead of the mixing, and the session's tokens
//       are compared with them until the first difference, whose position is tracked in a register;
//   (2) the chain over the chunk's 1,024 digests (exchanged through shared memory) is a
//       block-wide scan in which only the additive part travels: composing n blocks always
//       multiplies by P^n, so the multiplier of every scan step is a compile-time constant
//       and the carry from earlier chunks enters through two per-thread powers of P;
//   (3) hashes are written and compared with the stored session hashes, and the running state
//       moves on to the next chunk.  When the session hashes are to be derived instead, every
//       block before the first differing token has equal hashes by construction; from the
//       block that holds it one warp walks both chains until their states differ.
// Pairs are taken longest first.  Streams that do not start on a 16-byte boundary (the usual
// case in a concatenated batch) are read with aligned loads and re-aligned in registers.
// Measured: 56 - 57 % of the HBM copy rate on a 268 MB batch; a token costs 43 warp instructions,
// 23 of them its mix, and every lane reads its own block (16 bytes at a stride of 64).
#include <algorithm>
#include <vector>

#include "prefix_common.cuh"

namespace tal {

// Shape of the CTA.  Measured on the 1,024 x 32,768-token batch: 64 / 128 / 256 threads with
// 12 / 8 / 3-4 CTAs per SM land within a few per cent of each other; more than two quads in
// flight per stream, or eight rounds per chunk, spill at the 80-register budget and are slower.
constexpr int kPairThreads = 256;
constexpr int kPairCtasPerSm = 3;      // register budget of 80 per thread
constexpr int kDepth = 2;              // quads in flight per stream
constexpr int kPairWarps = kPairThreads / 32;
constexpr int kChunkBlocks = 1024;                         // blocks per chunk
constexpr int kRounds = kChunkBlocks / kPairThreads;       // blocks per thread per chunk
static_assert(kRounds * kPairThreads == kChunkBlocks && (kPairWarps & (kPairWarps - 1)) == 0 && kPairWarps <= 32,
              "a chunk is a whole number of rounds and the warp totals are scanned by a power-of-two group of lanes");

__host__ __device__ constexpr uint64_t pow_p(unsigned n) {
  uint64_t r = 1, b = kP;
  while (n) {
    if (n & 1u) r *= b;
    b *= b;
    n >>= 1;
  }
  return r;
}

// Four tokens starting at element address p, whatever its alignment: one or two aligned
// 16-byte loads, then a shift by m = (address / 4) mod 4 elements.  A 16-byte vector whose
// first needed element is inside the array never leaves that element's page.
template <bool ALIGNED>
__device__ __forceinline__ int4 load_quad(const int32_t *p, const int m, const bool need_hi) {
  if (ALIGNED) return __ldg((const int4 *)p);
  const int4 *v = (const int4 *)((uintptr_t)p & ~(uintptr_t)15);
  const int4 lo = __ldg(v);
  if (m == 0) return lo;
  int4 hi = make_int4(0, 0, 0, 0);
  if (need_hi) hi = __ldg(v + 1);
  const bool m2 = (m & 2) != 0, m1 = (m & 1) != 0;
  const int f0 = m2 ? lo.z : lo.x, f1 = m2 ? lo.w : lo.y, f2 = m2 ? hi.x : lo.z, f3 = m2 ? hi.y : lo.w,
            f4 = m2 ? hi.z : hi.x;
  return make_int4(m1 ? f1 : f0, m1 ? f2 : f1, m1 ? f3 : f2, m1 ? f4 : f3);
}

// sum of the four mixes of a quad whose first token sits at position J0 of its block
template <int J0>
__device__ __forceinline__ uint64_t quad_digest(const int4 v) {
  return mix64((uint64_t)(uint32_t)v.x + kG * (uint64_t)(J0 + 1)) + mix64((uint64_t)(uint32_t)v.y + kG * (uint64_t)(J0 + 2)) +
         mix64((uint64_t)(uint32_t)v.z + kG * (uint64_t)(J0 + 3)) + mix64((uint64_t)(uint32_t)v.w + kG * (uint64_t)(J0 + 4));
}

__device__ __forceinline__ void note_mismatch(const int4 a, const int4 b, const long long g0, long long &first_mis) {
  if (((a.x ^ b.x) | (a.y ^ b.y) | (a.z ^ b.z) | (a.w ^ b.w)) != 0) {
    const long long g = g0 + (a.x != b.x ? 0 : a.y != b.y ? 1 : a.z != b.z ? 2 : 3);
    first_mis = g < first_mis ? g : first_mis;
  }
}

// Rounds [r0, r1) of a chunk in which every token exists wherever it is used and every block is
// full.  In round r this thread owns block r*256 + tid of the chunk.  MODE 0: hash cont.
// MODE 1: hash cont, compare with sess.  Quads are requested DEPTH quads before they are used
// (a rolling buffer of DEPTH quads per stream).
template <int LOG2B, int MODE, bool ALIGNED>
__device__ __forceinline__ void hash_blocks(const int32_t *cont, const int32_t *sess, const int mc, const int ms,
                                            const int64_t tbase, const int r0, const int r1, uint64_t *dig_c,
                                            long long &first_mis) {
  constexpr int Q = (1 << LOG2B) / 4;                    // quads per block
  constexpr int DEPTH = Q < kDepth ? Q : kDepth;         // quads in flight per stream
  constexpr int kRoundTok = kPairThreads << LOG2B;       // tokens between this thread's blocks of two rounds
  if (r0 >= r1) return;
  const int tid = threadIdx.x;
  const int64_t g_first = tbase + ((int64_t)tid << LOG2B);
  const int32_t *pc = cont + g_first, *ps = sess + g_first;
  int4 a[DEPTH], b[DEPTH];
#pragma unroll
  for (int i = 0; i < DEPTH; ++i) {
    const int dr = i / Q, u = i % Q;
    a[i] = b[i] = make_int4(0, 0, 0, 0);
    if (r0 + dr < r1) {
      a[i] = load_quad<ALIGNED>(pc + (int64_t)(r0 + dr) * kRoundTok + 4 * u, mc, true);
      if (MODE != 0) b[i] = load_quad<ALIGNED>(ps + (int64_t)(r0 + dr) * kRoundTok + 4 * u, ms, true);
    }
  }
  for (int r = r0; r < r1; ++r) {
    uint64_t vc = 0;
#pragma unroll
    for (int u = 0; u < Q; ++u) {
      const int slot = u % DEPTH;
      const int4 qa = a[slot], qb = b[slot];
      const int dr = (u + DEPTH) / Q, un = (u + DEPTH) % Q;   // the quad DEPTH steps ahead
      if (r + dr < r1) {
        a[slot] = load_quad<ALIGNED>(pc + (int64_t)(r + dr) * kRoundTok + 4 * un, mc, true);
        if (MODE != 0) b[slot] = load_quad<ALIGNED>(ps + (int64_t)(r + dr) * kRoundTok + 4 * un, ms, true);
      }
      if (MODE != 0) note_mismatch(qa, qb, g_first + (int64_t)r * kRoundTok + 4 * u, first_mis);
      switch (u) {      // the position weights are immediates
#define TAL_QUAD(U) case U: vc += quad_digest<4 * U>(qa); break;
        TAL_QUAD(0) TAL_QUAD(1) TAL_QUAD(2) TAL_QUAD(3) TAL_QUAD(4) TAL_QUAD(5) TAL_QUAD(6) TAL_QUAD(7)
#undef TAL_QUAD
      }
    }
    dig_c[r * kPairThreads + tid] = vc;
  }
}

// The same rounds with every token and block checked against the ends of the two streams.
template <int LOG2B>
__device__ __forceinline__ void hash_blocks_checked(const int32_t *cont, const int32_t *sess, const int mc,
                                                    const int ms, const int64_t tbase, const int r0, const int r1,
                                                    const int64_t Tc, const int64_t Ts, const int64_t hash_c_end,
                                                    const int64_t cmp_end, uint64_t *dig_c, long long &first_mis) {
  constexpr int B = 1 << LOG2B;
  constexpr int kRoundTok = kPairThreads << LOG2B;
  const int tid = threadIdx.x;
  for (int r = r0; r < r1; ++r) {
    const int64_t gb = tbase + (int64_t)r * kRoundTok + ((int64_t)tid << LOG2B);   // first token of the block
    const bool full_c = gb < hash_c_end;                                           // a block is full or not hashed
    uint64_t vc = 0;
    if (full_c || gb < cmp_end) {
      for (int j0 = 0; j0 < B; j0 += 4) {
        const int64_t g0 = gb + j0;
        int4 a = make_int4(0, 0, 0, 0), b = make_int4(0, 0, 0, 0);
        if (g0 < Tc && (full_c || g0 < cmp_end)) a = load_quad<false>(cont + g0, mc, g0 + 4 - mc < Tc);
        if (g0 < Ts && g0 < cmp_end) b = load_quad<false>(sess + g0, ms, g0 + 4 - ms < Ts);
        const int ta[4] = {a.x, a.y, a.z, a.w}, tb[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int e = 3; e >= 0; --e)
          if (g0 + e < cmp_end && ta[e] != tb[e]) first_mis = (first_mis < g0 + e) ? first_mis : g0 + e;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const uint64_t w = kG * (uint64_t)(j0 + e + 1);
          if (full_c) vc += mix64((uint64_t)(uint32_t)ta[e] + w);
        }
      }
    }
    dig_c[r * kPairThreads + tid] = vc;
  }
}

// Inclusive scan over the CTA's threads of x_t (each the zero-carry chain of that thread's
// kRounds blocks).  Returns the zero-carry chain of everything BEFORE the thread's run, split in two
// parts so that  state_before_run = carry * P^(kRounds tid) + before_warps * P^(kRounds lane) + before_lanes;
// total = chain of the whole chunk.  s_tot: one word of shared memory per warp.
__device__ __forceinline__ void chunk_scan(uint64_t x, uint64_t *s_tot, uint64_t &before_warps,
                                           uint64_t &before_lanes, uint64_t &total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint64_t y = shfl_up_u64(x, d);
    if (lane >= d) x = y * pow_p(kRounds * d) + x;
  }
  if (lane == 31) s_tot[wid] = x;
  before_lanes = shfl_up_u64(x, 1);
  if (lane == 0) before_lanes = 0;
  __syncthreads();
  uint64_t v = s_tot[lane & (kPairWarps - 1)];
#pragma unroll
  for (int d = 1; d < kPairWarps; d <<= 1) {
    const uint64_t y = shfl_up_u64(v, d);
    if ((lane & (kPairWarps - 1)) >= d) v = y * pow_p(kRounds * 32 * d) + v;
  }
  total = (uint64_t)__shfl_sync(0xffffffffu, (unsigned long long)v, kPairWarps - 1);
  before_warps = (uint64_t)__shfl_sync(0xffffffffu, (unsigned long long)v, (wid + kPairWarps - 1) & (kPairWarps - 1));
  if (wid == 0) before_warps = 0;
}

template <bool DERIVE, int LOG2B>
__global__ void __launch_bounds__(kPairThreads, kPairCtasPerSm) prefix_pair_kernel(const __grid_constant__ PrefixParams p) {
  constexpr int B = 1 << LOG2B;
  constexpr int kRoundTok = kPairThreads << LOG2B;     // tokens hashed per round by the whole CTA
  constexpr int kChunkShift = 10 + LOG2B;              // tokens per chunk = 1024 * B
  __shared__ __align__(16) uint64_t s_dig[kChunkBlocks];
  __shared__ uint64_t s_tot[kPairWarps];
  __shared__ long long s_red[2][kPairThreads / 32];
  __shared__ unsigned long long s_first;     // DERIVE: the first differing token seen by any thread
  __shared__ uint64_t s_state;               // DERIVE: chain state before the block that holds it
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const PairDesc pd = p.pairs[blockIdx.x];             // sorted longest first; tile_off = the pair's index
  const int pair = (int)pd.tile_off;
  const int32_t *cont = p.cont + pd.cont_off;
  const int32_t *sess = p.sess + pd.sess_off;
  const int mc = (int)(((uintptr_t)cont >> 2) & 3), ms = (int)(((uintptr_t)sess >> 2) & 3);
  const bool aligned = (mc | ms) == 0;
  const int64_t Tc = pd.Tc, Ts = pd.Ts, Tmin = Tc < Ts ? Tc : Ts;
  const int64_t nbc = Tc >> LOG2B, nbs = Ts >> LOG2B, lim = nbc < nbs ? nbc : nbs;
  // Only the continuation is hashed.  With stored hashes the chain compares block by block; when
  // they are to be derived, every block before the first differing token has equal hashes by
  // construction, and the session is hashed from that block on until the hashes differ.
  const int64_t hash_c_end = nbc << LOG2B;
  if (DERIVE && tid == 0) s_first = (unsigned long long)kNoMismatch;
  const uint64_t *hs_in = DERIVE ? nullptr : p.sess_hashes + pd.sess_hash_off;
  uint64_t *hc_out = p.cont_hashes_out ? p.cont_hashes_out + pd.cont_hash_off : nullptr;

  // P^(kRounds lane) and P^(kRounds tid): where this thread's run starts inside its warp and inside the chunk
  uint64_t pow_lane = 1, pow_tid = 1;
  {
    uint64_t b = pow_p(kRounds);
    for (int n = lane; n; n >>= 1, b *= b)
      if (n & 1) pow_lane *= b;
    b = pow_p(kRounds * 32);
    pow_tid = pow_lane;
    for (int n = wid; n; n >>= 1, b *= b)
      if (n & 1) pow_tid *= b;
  }

  if (DERIVE) __syncthreads();                        // s_first is set before anyone lowers it
  uint64_t carry_c = p.seed;
  long long first_mis = kNoMismatch, first_bad = lim;
  bool diverged = false;                              // CTA-uniform: a token mismatch has been seen
  for (int64_t ch = 0;; ++ch) {
    const int64_t tbase = ch << kChunkShift;
    // once the streams have diverged, later session tokens matter only if their hashes are derived
    const int64_t cmp_end = diverged ? 0 : Tmin;
    const int64_t need_end = hash_c_end > cmp_end ? hash_c_end : cmp_end;
    if (tbase >= need_end) break;
    // round r covers tokens [tbase + r*kRoundTok, +kRoundTok): rounds_below(t) of them end at or
    // before t, rounds_reaching(t) of them start before t
    auto rounds_below = [&](int64_t t) {
      return (int)(t <= tbase ? 0 : ((t - tbase) / kRoundTok < kRounds ? (t - tbase) / kRoundTok : kRounds));
    };
    auto rounds_reaching = [&](int64_t t) { return rounds_below(t + kRoundTok - 1); };
    const int r_end = rounds_reaching(need_end);
    // [0, r_a): both streams fully present (hash the continuation, compare) -- no checks;
    // [r_a, r_b): rounds that straddle the end of the compared range -- checked;
    // [r_b, r_c): only the continuation is left and its blocks are full -- no checks;
    // [r_c, r_end): its ragged tail -- checked.
    const int64_t both_end = hash_c_end < cmp_end ? hash_c_end : cmp_end;
    const int r_a = rounds_below(both_end);
    int r_b = rounds_reaching(cmp_end);                 // beyond cmp_end the session is not read
    r_b = r_b < r_a ? r_a : (r_b > r_end ? r_end : r_b);
    int r_c = rounds_below(hash_c_end);
    r_c = r_c < r_b ? r_b : r_c;
    uint64_t *dc = s_dig;
    if (aligned) hash_blocks<LOG2B, 1, true>(cont, sess, mc, ms, tbase, 0, r_a, dc, first_mis);
    else         hash_blocks<LOG2B, 1, false>(cont, sess, mc, ms, tbase, 0, r_a, dc, first_mis);
    hash_blocks_checked<LOG2B>(cont, sess, mc, ms, tbase, r_a, r_b, Tc, Ts, hash_c_end, cmp_end, dc, first_mis);
    if (mc == 0) hash_blocks<LOG2B, 0, true>(cont, sess, mc, ms, tbase, r_b, r_c, dc, first_mis);
    else         hash_blocks<LOG2B, 0, false>(cont, sess, mc, ms, tbase, r_b, r_c, dc, first_mis);
    hash_blocks_checked<LOG2B>(cont, sess, mc, ms, tbase, r_c, r_end, Tc, Ts, hash_c_end, cmp_end, dc, first_mis);
    const bool was_diverged = diverged;
    if (DERIVE && !was_diverged && first_mis != kNoMismatch) atomicMin(&s_first, (unsigned long long)first_mis);
    diverged = __syncthreads_or(first_mis != kNoMismatch) != 0;
    // DERIVE: the block that holds the first differing token, if it is one of this chunk's blocks
    // that both streams have in full (it can only be found in the chunk that holds it)
    int q_div = -1;                                      // ... and this thread's run holds it at q_div
    bool resolve = false;
    if (DERIVE && diverged && !was_diverged) {
      const int64_t d = (int64_t)(s_first >> LOG2B);
      resolve = d < lim;
      const int64_t rel = d - (ch * kChunkBlocks + (int64_t)tid * kRounds);
      if (resolve && rel >= 0 && rel < kRounds) q_div = (int)rel;
    }
    // its tokens are requested now and used after the chain phase
    uint32_t div_c = 0, div_s = 0;
    if (DERIVE && resolve && wid == 0 && lane < B) {
      const int64_t g = (int64_t)((s_first >> LOG2B) << LOG2B) + lane;
      div_c = (uint32_t)__ldg(cont + g);
      div_s = (uint32_t)__ldg(sess + g);
    }

    // ---- chain over this chunk's blocks ----------------------------------
    const int64_t k0 = ch * kChunkBlocks + tid * kRounds;
    if (ch * kChunkBlocks < nbc) {
      uint64_t vc[kRounds], hst[kRounds];
#pragma unroll
      for (int q = 0; q < kRounds; ++q) {
        vc[q] = dc[tid * kRounds + q];
        hst[q] = (!DERIVE && k0 + q < lim) ? __ldg(hs_in + k0 + q) : 0ull;
      }
      uint64_t xc = 0;
#pragma unroll
      for (int q = 0; q < kRounds; ++q) xc = xc * kP + vc[q];
      uint64_t bw_c, bl_c, tot_c;
      chunk_scan(xc, s_tot, bw_c, bl_c, tot_c);
      uint64_t sc = carry_c * pow_tid + bw_c * pow_lane + bl_c;
#pragma unroll
      for (int q = 0; q < kRounds; ++q) {
        const int64_t k = k0 + q;
        if (DERIVE && q == q_div) s_state = sc;
        sc = sc * kP + vc[q];
        if (k < nbc) {
          const uint64_t hc = mix64(sc);
          if (hc_out) hc_out[k] = hc;
          if (!DERIVE && k < lim && hst[q] != hc && k < first_bad) first_bad = k;
        }
      }
      carry_c = carry_c * pow_p(kChunkBlocks) + tot_c;
    }
    if (DERIVE && resolve) {     // CTA-uniform, at most once per pair
      __syncthreads();
      if (wid == 0) {
        // Both chains enter block d in the same state.  mix64 is a bijection, so two block hashes
        // are equal exactly when the states are: walk on until the states differ (the first step,
        // unless two different blocks have equal digests).
        uint64_t st_c = s_state, st_s = st_c;
        int64_t k = (int64_t)(s_first >> LOG2B);
        const uint64_t w = kG * (uint64_t)(lane + 1);
        for (; k < lim; ++k) {
          uint64_t dgc = lane < B ? mix64((uint64_t)div_c + w) : 0ull, dgs = lane < B ? mix64((uint64_t)div_s + w) : 0ull;
          for (int m = 16; m >= 1; m >>= 1) {
            dgc += shfl_xor_u64(dgc, m);
            dgs += shfl_xor_u64(dgs, m);
          }
          st_c = st_c * kP + dgc;
          st_s = st_s * kP + dgs;
          if (st_c != st_s) break;
          if (k + 1 < lim && lane < B) {
            div_c = (uint32_t)__ldg(cont + ((k + 1) << LOG2B) + lane);
            div_s = (uint32_t)__ldg(sess + ((k + 1) << LOG2B) + lane);
          }
        }
        first_bad = k < first_bad ? k : first_bad;
      }
    }
  }

  // ---- result record ---------------------------------------------------------
  long long lcp = first_mis < Tmin ? first_mis : Tmin;
  for (int m = 16; m >= 1; m >>= 1) {
    const long long o = __shfl_xor_sync(0xffffffffu, lcp, m);
    lcp = o < lcp ? o : lcp;
    const long long o2 = __shfl_xor_sync(0xffffffffu, first_bad, m);
    first_bad = o2 < first_bad ? o2 : first_bad;
  }
  if (lane == 0) {
    s_red[0][wid] = lcp;
    s_red[1][wid] = first_bad;
  }
  __syncthreads();
  if (tid == 0 && p.results) {
    for (int w = 1; w < kPairThreads / 32; ++w) {
      lcp = s_red[0][w] < lcp ? s_red[0][w] : lcp;
      first_bad = s_red[1][w] < first_bad ? s_red[1][w] : first_bad;
    }
    const long long lcp_blocks = lcp >> LOG2B;
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

template <bool DERIVE>
static void launch_pair_kernel(const PrefixParams &p, int log2B, unsigned grid, cudaStream_t stream) {
  switch (log2B) {
    case 2: prefix_pair_kernel<DERIVE, 2><<<grid, kPairThreads, 0, stream>>>(p); break;
    case 3: prefix_pair_kernel<DERIVE, 3><<<grid, kPairThreads, 0, stream>>>(p); break;
    case 4: prefix_pair_kernel<DERIVE, 4><<<grid, kPairThreads, 0, stream>>>(p); break;
    default: prefix_pair_kernel<DERIVE, 5><<<grid, kPairThreads, 0, stream>>>(p); break;
  }
}

// The pair table is written longest pair first (so the last CTAs to start are the short ones),
// each entry carrying its pair's index in tile_off; one launch.
// log2B must be 2..5 (block sizes 4, 8, 16, 32).
talaria_status_t pair_launch(talaria_ctx *ctx, int32_t n_pairs, const PairSpec *specs, const int32_t *d_cont,
                             const int32_t *d_sess, const uint64_t *d_sess_hashes, int32_t B, int log2B,
                             uint64_t seed, uint64_t *d_cont_hashes, talaria_match_t *d_results,
                             cudaStream_t stream) {
  if (log2B < 2 || log2B > 5) return TALARIA_ERR_INVALID_ARG;
  const size_t pair_bytes = ((size_t)n_pairs * sizeof(PairDesc) + 15) & ~(size_t)15;
  const size_t desc_bytes = 2 * pair_bytes;          // second half: the table in call order, before sorting
  DescSlot *slot = nullptr;
  TAL_TRY(acquire_slot(ctx, desc_bytes, &slot));
  PairDesc *pd = (PairDesc *)slot->h;
  PairDesc *in_order = (PairDesc *)(slot->h + pair_bytes);
  bool sorted = true;
  for (int32_t q = 0; q < n_pairs; ++q) {
    const PairSpec &sp = specs[q];
    in_order[q] = PairDesc{sp.cont_off, sp.sess_off, sp.Tc, sp.Ts, 0, 0, q, sp.cont_hash_off, sp.sess_hash_off};
    if (q && std::max(sp.Tc, sp.Ts) > std::max(in_order[q - 1].Tc, in_order[q - 1].Ts)) sorted = false;
  }
  if (sorted) {
    pd = in_order;
  } else {
    std::vector<int32_t> order(n_pairs);
    for (int32_t q = 0; q < n_pairs; ++q) order[q] = q;
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
      return std::max(in_order[a].Tc, in_order[a].Ts) > std::max(in_order[b].Tc, in_order[b].Ts);
    });
    for (int32_t q = 0; q < n_pairs; ++q) pd[q] = in_order[order[q]];
  }
  // Each CTA reads its one descriptor straight from the pinned slot (56 bytes over the host
  // link): no upload stands between this launch and the previous kernel on the stream.
  PrefixParams p{};
  p.pairs = pd;
  p.n_pairs = n_pairs;
  p.B = B;
  p.log2B = log2B;
  p.need_sess_digest = d_sess_hashes ? 0 : 1;
  p.cont = d_cont;
  p.sess = d_sess;
  p.sess_hashes = d_sess_hashes;
  p.cont_hashes_out = d_cont_hashes;
  p.results = d_results;
  p.seed = seed;
  if (d_sess_hashes) launch_pair_kernel<false>(p, log2B, (unsigned)n_pairs, stream);
  else               launch_pair_kernel<true>(p, log2B, (unsigned)n_pairs, stream);
  TAL_CUDA(ctx, cudaGetLastError());
  ctx->counters.kernel_launches++;
  return release_slot(ctx, slot, stream);
}

}  // namespace tal
