// Merge of the split-K partials of one (sequence, head) row: the body shared by the stand-alone
// combine kernel (sparse_decode.cu) and the kernel that runs it beside a TopK (topk_select.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace kvswap {

constexpr int kMaxSplits = 256;

// D threads (c = 0..D-1) merge row `row` of partial [rows, splits, D + 2] = (m, l, acc[D]) into
// out[row, :] and lse[row].  Every load of the row is issued before anything is computed (one
// memory round trip); the split weights are formed once by the first warp of the D threads and
// shared through w_s [kMaxSplits] and norm_s [2].  The D threads meet at named barrier `barrier`
// (0 = the CTA-wide one: then the CTA has exactly D threads).  `live` false: the threads only keep
// the barrier company.
template <int D>
__device__ __forceinline__ void combine_row(const float* __restrict__ partial, float* __restrict__ out,
                                            float* __restrict__ lse, int splits, int64_t row, bool live, int c,
                                            float* w_s, float* norm_s, int barrier) {
  constexpr float kLn2 = 0.6931471805599453f;
  constexpr int kUnroll = 16;
  const float* src = partial + row * splits * (D + 2);
  float a_first[kUnroll];
#pragma unroll
  for (int s = 0; s < kUnroll; ++s) a_first[s] = (live && s < splits) ? src[s * (D + 2) + 2 + c] : 0.f;
  if (live && c < 32) {
    // weights: lane s handles splits s, s + 32, ...
    float mx = -INFINITY;
    for (int s = c; s < splits; s += 32) mx = fmaxf(mx, src[s * (D + 2)]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    float lsum = 0.f;
    for (int s = c; s < splits; s += 32) {
      const float w = (mx > -INFINITY) ? exp2f(src[s * (D + 2)] - mx) : 0.f;
      w_s[s] = w;
      lsum = fmaf(src[s * (D + 2) + 1], w, lsum);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, off);
    if (c == 0) {
      norm_s[0] = (lsum > 0.f) ? 1.f / lsum : 0.f;
      norm_s[1] = (lsum > 0.f) ? (mx + log2f(lsum)) * kLn2 : -INFINITY;
    }
  }
  if (barrier == 0) __syncthreads();
  else asm volatile("bar.sync %0, %1;" ::"r"(barrier), "r"(D) : "memory");
  if (!live) return;
  float a = 0.f;
#pragma unroll
  for (int s = 0; s < kUnroll; ++s) if (s < splits) a = fmaf(a_first[s], w_s[s], a);
  for (int s = kUnroll; s < splits; ++s) a = fmaf(src[s * (D + 2) + 2 + c], w_s[s], a);
  out[row * D + c] = a * norm_s[0];
  if (lse != nullptr && c == 0) lse[row] = norm_s[1];
}

}  // namespace kvswap
