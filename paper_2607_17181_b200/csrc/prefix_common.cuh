// Declarations shared by the prefix-match sources: constants of the chained block hash
// (Sec. 4.3 / App. B), the pair descriptor, kernel parameters and small device helpers.
#pragma once
#include "internal.h"

namespace tal {

constexpr uint64_t kG = 0x9E3779B97F4A7C15ull;
constexpr uint64_t kP = 0xD1342543DE82EF95ull;
constexpr int kTileTok = 2048;        // tokens per tile: latency path (fused kernel, static entry point)
constexpr int kBatchTileTok = 8192;   // tokens per tile in big batches: amortises the per-CTA start-up
constexpr int kTileThreads = 256;
constexpr int kScanThreads = 256;
constexpr int kScanItems = 8;
constexpr long long kNoMismatch = 0x7fffffffffffffffll;

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
  z ^= z >> 30;
  z *= 0xBF58476D1CE4E5B9ull;
  z ^= z >> 27;
  z *= 0x94D049BB133111EBull;
  z ^= z >> 31;
  return z;
}

struct PairDesc {
  int64_t cont_off, sess_off;          // token offsets into the concatenated arrays
  int64_t Tc, Ts;                      // token counts
  int64_t cont_blk_off, sess_blk_off;  // block offsets into the scratch digest arrays (packed pair after pair)
  int64_t tile_off;                    // first tile of this pair (tiled kernels); the pair's index
                                       // in the call (one-CTA-per-pair kernel, whose table is sorted)
  int64_t cont_hash_off, sess_hash_off;  // where the pair's block hashes sit in the callers' hash arrays
};

// One pair as the host entry points describe it: where its two streams and their block hashes
// sit in the token and hash arrays (element offsets).
struct PairSpec {
  int64_t cont_off, Tc, sess_off, Ts;
  int64_t cont_hash_off, sess_hash_off;
};

constexpr int kInlinePairs = 8;    // up to this many pairs travel in the kernel parameters
constexpr int64_t kFusedMaxTiles = 296;    // 2 CTAs per SM x 148 SMs: about one wave of the fused kernel

struct PrefixParams {
  const PairDesc *pairs;      // DEVICE [n_pairs + 1] (last entry holds the totals); null when inline
  const int32_t *tile_pair;   // DEVICE [tiles]: pair of each tile; null when inline
  PairDesc inl[kInlinePairs + 1];
  int32_t n_pairs;
  int32_t B;
  int32_t log2B;              // >= 0 when B is a power of two <= 32, else -1
  int32_t need_sess_digest;   // 1 when stored hashes are not supplied
  int32_t tile_tok;           // tokens per tile (a multiple of 1024)
  const int32_t *cont, *sess; // DEVICE tokens
  uint64_t *dig_c, *dig_s;    // DEVICE scratch digests
  long long *tile_mis;        // DEVICE scratch [total tiles]
  const uint64_t *sess_hashes;// DEVICE or null
  uint64_t *cont_hashes_out;  // DEVICE or null
  talaria_match_t *results;   // DEVICE [n_pairs] or null
  uint64_t seed;
  unsigned int *counters;     // DEVICE [kInlinePairs], zero between calls (fused kernel only)
};

__device__ __forceinline__ uint64_t shfl_xor_u64(uint64_t v, int m) {
  return (uint64_t)__shfl_xor_sync(0xffffffffu, (unsigned long long)v, m);
}
__device__ __forceinline__ uint64_t shfl_up_u64(uint64_t v, int d) {
  return (uint64_t)__shfl_up_sync(0xffffffffu, (unsigned long long)v, d);
}


// One CTA per pair, for batches with at least one pair per SM (prefix_pair.cu).
talaria_status_t pair_launch(talaria_ctx *ctx, int32_t n_pairs, const PairSpec *specs, const int32_t *d_cont,
                             const int32_t *d_sess, const uint64_t *d_sess_hashes, int32_t B, int log2B,
                             uint64_t seed, uint64_t *d_cont_hashes, talaria_match_t *d_results,
                             cudaStream_t stream);

}  // namespace tal
