// Summed low-rank queries (Eq. 1, the query side): u = sum over heads h of q_h A_g(h), one row per
// selection scope.  The device code is shared by the streaming scorer, which builds the queries of
// its own row sets (score_stream.cu), and by the kernel that builds them one layer ahead beside the
// split-K combine (topk_select.cu): both therefore produce the same bits.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"

namespace kvswap {

constexpr int kQueryThreads = 512;                        // threads that call build_queries together
constexpr int kQueryWarps = kQueryThreads / 32;
constexpr int kQueryCols = 8;                             // query rows (scopes) per row set
constexpr int kQuerySumFloats = 8 * 128;                  // shared scratch: summed queries of up to 8 KV heads
constexpr int kQueryPartFloats = 32 * 32;                 // shared scratch: partial products, [item][column]

__device__ __forceinline__ float load_q(const void* q, int dtype, int64_t i) {
  if (dtype == KVSWAP_F32) return static_cast<const float*>(q)[i];
  if (dtype == KVSWAP_BF16) return __bfloat162float(static_cast<const __nv_bfloat16*>(q)[i]);
  return __half2float(static_cast<const __half*>(q)[i]);
}

// (sequence, metadata head, scope block) of a row set.
struct RowSet { int b, hm, sub; };
__device__ __forceinline__ RowSet row_set(const Problem& p, int rest, int n_sub) {
  const int hm_count = (p.Hm == 1) ? 1 : p.Hkv;
  const int bh = rest / n_sub;
  return RowSet{bh / hm_count, bh % hm_count, rest % n_sub};
}

// Summed low-rank queries of one row set into urow[8][32] (rows beyond the set's scopes are zero).
// The KV heads that feed the rows are taken eight at a time.  An item is 32 channels of one head:
// a warp multiplies the head's summed query by the adapter rows (coalesced 128-byte reads of A_g);
// it requests the adapter rows of its (at most two) items first, then the CTA sums the query
// heads into shared memory, so that both loads share one round trip.  The partial products are
// added in a fixed order.  Threads 0 .. kQueryThreads - 1 of the CTA call, and meet at barrier BAR
// (0: the CTA has exactly kQueryThreads threads).  qsum [kQuerySumFloats] and upart [kQueryPartFloats]
// are shared-memory scratch, urow [8 * 32] receives the result.
template <int BAR>
__device__ void build_queries(const Problem& p, const void* q, const float* __restrict__ proj, RowSet rs,
                              float* qsum, float* upart, float* urow) {
  auto sync = [] {
    if constexpr (BAR == 0) __syncthreads();
    else asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(kQueryThreads) : "memory");
  };
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool joint = p.Hm == 1;
  const bool all_heads = joint && p.scope == KVSWAP_SCOPE_ALL_HEADS;
  // term t of the row set: (row it adds to, KV head it reads)
  const int n_terms = all_heads ? p.Hkv : joint ? min(kQueryCols, p.S - rs.sub * kQueryCols) : 1;
  const int head0 = all_heads ? 0 : joint ? rs.sub * kQueryCols : rs.hm;      // head of term t: head0 + t
  const bool row_per_term = joint && !all_heads;                          // row of term t: t, else 0
  const int ch_shift = (p.d == 128) ? 2 : (p.d == 64) ? 1 : 0;            // 32-channel pieces of a head: 4, 2 or 1
  const int chunks = 1 << ch_shift;
  const int d_shift = ch_shift + 5;
  for (int t0 = 0; t0 < n_terms; t0 += 8) {
    const int nt = min(8, n_terms - t0);
    const int n_items = nt << ch_shift;                            // <= 32: items warp and warp + 16
    const int it0 = warp, it1 = warp + kQueryWarps;
    float a0[32], a1[32];
    {
      const float* P0 = proj + (int64_t(head0 + t0 + (it0 >> ch_shift)) * p.d + (it0 & (chunks - 1)) * 32) * p.r + lane;
      const float* P1 = proj + (int64_t(head0 + t0 + (it1 >> ch_shift)) * p.d + (it1 & (chunks - 1)) * 32) * p.r + lane;
#pragma unroll
      for (int cc = 0; cc < 32; ++cc) a0[cc] = (it0 < n_items) ? P0[cc * 32] : 0.f;
#pragma unroll
      for (int cc = 0; cc < 32; ++cc) a1[cc] = (it1 < n_items) ? P1[cc * 32] : 0.f;
    }
    for (int i = tid; i < (nt << d_shift); i += kQueryThreads) {
      const int tt = i >> d_shift, c = i & (p.d - 1);
      const int64_t at = (int64_t(rs.b) * p.Hq + int64_t(head0 + t0 + tt) * p.rho) * p.d + c;
      float s = 0.f;
      for (int h0 = 0; h0 < p.rho; h0 += 4) {                      // the loads of four heads go out together
        float v[4];
#pragma unroll
        for (int hh = 0; hh < 4; ++hh) v[hh] = (h0 + hh < p.rho) ? load_q(q, p.q_dtype, at + int64_t(h0 + hh) * p.d) : 0.f;
        s += (v[0] + v[1]) + (v[2] + v[3]);
      }
      qsum[tt * 128 + c] = s;
    }
    sync();
    if (it0 < n_items) {
      const float* qs = qsum + (it0 >> ch_shift) * 128 + (it0 & (chunks - 1)) * 32;
      float acc = 0.f;
#pragma unroll
      for (int cc = 0; cc < 32; ++cc) acc = fmaf(qs[cc], a0[cc], acc);
      upart[it0 * 32 + lane] = acc;
    }
    if (it1 < n_items) {
      const float* qs = qsum + (it1 >> ch_shift) * 128 + (it1 & (chunks - 1)) * 32;
      float acc = 0.f;
#pragma unroll
      for (int cc = 0; cc < 32; ++cc) acc = fmaf(qs[cc], a1[cc], acc);
      upart[it1 * 32 + lane] = acc;
    }
    sync();
    if (tid < kQueryCols * 32) {
      const int row = tid >> 5, j = tid & 31;
      float s = (t0 == 0) ? 0.f : urow[tid];
      if (row_per_term) {                                          // the items of term `row`
        if (row < nt)
          for (int ch = 0; ch < chunks; ++ch) s += upart[((row << ch_shift) + ch) * 32 + j];
      } else if (row == 0) {
        for (int it = 0; it < n_items; ++it) s += upart[it * 32 + j];
      }
      urow[tid] = s;
    }
    sync();
  }
}

// Rows of urow[8][32] (build_queries, r = 32) to the query buffer uq [B, Su, r] that the scorer reads
// when it does not build the queries itself: row i of a joint row set is scope sub * 8 + i, the one
// row of a per-head row set is head hm.  Threads 0 .. 255 of the callers of build_queries store.
__device__ __forceinline__ void store_queries(const Problem& p, RowSet rs, const float* urow, float* __restrict__ uq) {
  const int tid = threadIdx.x;
  if (tid >= kQueryCols * 32) return;
  const int row = tid >> 5, j = tid & 31;
  const int dst = (p.Hm == 1) ? rs.sub * kQueryCols + row : rs.hm;
  const bool have = (p.Hm == 1) ? (dst < p.Su) : (row == 0);
  if (have) uq[(int64_t(rs.b) * p.Su + dst) * p.r + j] = urow[tid];
}

}  // namespace kvswap
