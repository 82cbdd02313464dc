// Order-preserving integer keys of group scores, shared by the scorer (which counts the keys'
// leading digit while it produces the scores) and the TopK kernels (Sec. 4.3).
#pragma once

#include <stdint.h>

namespace kvswap {

constexpr int kKeyTopBits = 12;                        // leading digit counted by the scorer
constexpr int kKeyTopBins = 1 << kKeyTopBits;          // bins of the per-problem histogram

// Larger score <=> larger key; -0 and +0 are the same score.
__device__ __forceinline__ uint32_t score_key(float f) {
  uint32_t u = __float_as_uint(f);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Leading digit of a score's key.  (The TopK kernels lift the one key that is 0, the pattern of
// a negative NaN with all bits set, to 1 so that padding stays below every real key; both have
// leading digit 0.)
__device__ __forceinline__ uint32_t score_key_top(float f) { return score_key(f) >> (32 - kKeyTopBits); }

}  // namespace kvswap
