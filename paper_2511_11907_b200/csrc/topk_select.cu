// K3: TopK over group scores (Sec. 4.3): per (sequence, scope) the M' = min(M, NG) groups with
// the largest score, lower index first among equal scores, written in ascending index order.
//
// One CTA per problem.  Scores become order-preserving 32-bit keys; an MSB-first radix select
// finds the key of rank M' and how many groups equal to it are still needed; a stable compaction
// in index order then emits the selection.
//   topk_select_regs_kernel   NG <= 16384: every thread keeps its 1, 4 or 16 consecutive keys in
//                             registers; digits of 12, 12 and 8 bits, so that the first pass
//                             already isolates a few hundred candidates and later passes touch
//                             only those; stops as soon as a digit bin is taken whole.
//   topk_select_kernel        longer rows: keys in shared memory (or re-read), 8-bit digits.
#include "async_copy.cuh"
#include "combine.cuh"
#include "lowrank_query.cuh"
#include "common.cuh"
#include "topk_keys.cuh"
#include "topk_parts.cuh"

namespace kvswap {
namespace {

constexpr int kThreads = 1024;
constexpr int kMaxSmemKeys = 48 * 1024;   // 192 KB of keys kept on chip; longer rows re-read L2

// Inclusive prefix sum over the CTA (all threads must call).  `warp_tot` holds 32 ints.
__device__ __forceinline__ int block_inclusive_scan(int v, int* warp_tot) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, v, off);
    if (lane >= off) v += t;
  }
  __syncthreads();                 // protect warp_tot from the previous use
  if (lane == 31) warp_tot[warp] = v;
  __syncthreads();
  if (warp == 0) {
    int w = (lane < kThreads / 32) ? warp_tot[lane] : 0;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, w, off);
      if (lane >= off) w += t;
    }
    warp_tot[lane] = w;            // inclusive totals
  }
  __syncthreads();
  return v + (warp > 0 ? warp_tot[warp - 1] : 0);
}

__global__ void __launch_bounds__(kThreads)
topk_select_kernel(Problem p, const float* __restrict__ scores, int32_t* __restrict__ group_idx,
                   int32_t* __restrict__ n_selected, int keys_in_smem) {
  extern __shared__ uint32_t keys[];
  __shared__ int hist[256];
  __shared__ int warp_tot[32];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_want;

  pdl_wait();
  pdl_trigger();
  const int prob = blockIdx.x;                 // b * S + s
  const float* R = scores + int64_t(prob) * p.score_pitch;
  int32_t* out = group_idx + int64_t(prob) * p.M;
  const int NG = p.NG, Mp = p.Mp;

  if (threadIdx.x == 0) n_selected[prob] = Mp;
  for (int i = Mp + threadIdx.x; i < p.M; i += kThreads) out[i] = -1;
  if (Mp == 0) return;
  if (Mp == NG) {                              // everything is selected
    for (int i = threadIdx.x; i < NG; i += kThreads) out[i] = i;
    return;
  }

  if (keys_in_smem)
    for (int i = threadIdx.x; i < NG; i += kThreads) keys[i] = score_key(R[i]);
  if (threadIdx.x == 0) { sh_prefix = 0u; sh_want = Mp; }
  __syncthreads();

  // ---- radix select: key of descending rank Mp ------------------------------------------
  uint32_t mask = 0u;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (threadIdx.x < 256) hist[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t prefix = sh_prefix;
    const int want = sh_want;
    for (int i = threadIdx.x; i < NG; i += kThreads) {
      const uint32_t k = keys_in_smem ? keys[i] : score_key(R[i]);
      if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 255u], 1);
    }
    __syncthreads();
    // thread t looks at digit 255 - t: inclusive count of candidates with a digit >= its own
    const int mine = (threadIdx.x < 256) ? hist[255 - threadIdx.x] : 0;
    const int incl = block_inclusive_scan(mine, warp_tot);
    if (threadIdx.x < 256 && incl >= want && incl - mine < want) {
      sh_prefix = prefix | (uint32_t(255 - threadIdx.x) << shift);
      sh_want = want - (incl - mine);
    }
    mask |= 255u << shift;
    __syncthreads();
  }
  const uint32_t kth = sh_prefix;
  const int need_eq = sh_want;                 // groups equal to kth still to take (lowest indices)

  // ---- stable compaction in index order ---------------------------------------------------
  const int per = (NG + kThreads - 1) / kThreads;
  const int lo = min(NG, int(threadIdx.x) * per), hi = min(NG, lo + per);
  int n_gt = 0, n_eq = 0;
  for (int i = lo; i < hi; ++i) {
    const uint32_t k = keys_in_smem ? keys[i] : score_key(R[i]);
    n_gt += (k > kth);
    n_eq += (k == kth);
  }
  const int eq_before = block_inclusive_scan(n_eq, warp_tot) - n_eq;
  int eq_take = max(0, min(n_eq, need_eq - eq_before));
  const int n_sel = n_gt + eq_take;
  int pos = block_inclusive_scan(n_sel, warp_tot) - n_sel;
  for (int i = lo; i < hi; ++i) {
    const uint32_t k = keys_in_smem ? keys[i] : score_key(R[i]);
    bool take = k > kth;
    if (k == kth && eq_take > 0) { take = true; --eq_take; }
    if (take) out[pos++] = i;
  }
}


// ------------------------------------------------------------------------------------------
// Register-resident select for NG <= kThreads * KPT.
// ------------------------------------------------------------------------------------------
constexpr int kBins = 4096;

// Among the candidates counted in hist[0..n_bins) find, from the top, the bin that holds the
// candidate of descending rank `want` (1-based).  Thread t owns `per` consecutive bins counted
// down from the top.  Results: sh_bin, sh_want (rank inside that bin), sh_cnt (its population).
__device__ __forceinline__ void find_bin(const int* hist, int n_bins, int want, int* warp_tot, int* sh_bin,
                                         int* sh_want, int* sh_cnt) {
  const int per = (n_bins + kThreads - 1) / kThreads;          // 4 for 4096 bins, 1 for 256
  const int top = n_bins - 1 - int(threadIdx.x) * per;         // highest bin of this thread
  int local = 0;
  for (int i = 0; i < per; ++i) { const int bin = top - i; if (bin >= 0) local += hist[bin]; }
  const int incl = block_inclusive_scan(local, warp_tot);
  const int before = incl - local;                             // candidates in bins above mine
  if (before < want && incl >= want) {
    int acc = before;
    for (int i = 0; i < per; ++i) {
      const int bin = top - i;
      const int c = (bin >= 0) ? hist[bin] : 0;
      if (acc + c >= want) { *sh_bin = bin; *sh_want = want - acc; *sh_cnt = c; break; }
      acc += c;
    }
  }
}

template <int KPT>
__global__ void __launch_bounds__(kThreads)
topk_select_regs_kernel(Problem p, const float* __restrict__ scores, int32_t* __restrict__ group_idx,
                        int32_t* __restrict__ n_selected) {
  __shared__ int hist[kBins];
  __shared__ int warp_tot[32];
  __shared__ int sh_bin, sh_want, sh_cnt;

  const int prob = blockIdx.x;                 // b * S + s
  const int NG = p.NG, Mp = p.Mp;
  for (int i = threadIdx.x; i < kBins; i += kThreads) hist[i] = 0;
  pdl_wait();
  pdl_trigger();
  const float* R = scores + int64_t(prob) * p.score_pitch;
  int32_t* out = group_idx + int64_t(prob) * p.M;

  if (threadIdx.x == 0) n_selected[prob] = Mp;
  for (int i = Mp + threadIdx.x; i < p.M; i += kThreads) out[i] = -1;
  if (Mp == 0) return;
  if (Mp == NG) {                              // everything is selected
    for (int i = threadIdx.x; i < NG; i += kThreads) out[i] = i;
    return;
  }

  // ---- this thread's KPT consecutive keys (0 = below every real key, for the padding) ----------
  const int i0 = int(threadIdx.x) * KPT;
  uint32_t key[KPT];
  if constexpr (KPT >= 4) {
    if ((p.score_pitch & 3) == 0) {              // rows start 16-byte aligned and are padded to whole vectors
#pragma unroll
      for (int v = 0; v < KPT / 4; ++v) {
        if (i0 + 4 * v < NG) {
          const float4 f = *reinterpret_cast<const float4*>(R + i0 + 4 * v);
          key[4 * v] = score_key(f.x);
          key[4 * v + 1] = (i0 + 4 * v + 1 < NG) ? score_key(f.y) : 0u;      // row padding, never a key
          key[4 * v + 2] = (i0 + 4 * v + 2 < NG) ? score_key(f.z) : 0u;
          key[4 * v + 3] = (i0 + 4 * v + 3 < NG) ? score_key(f.w) : 0u;
        } else {
          key[4 * v] = key[4 * v + 1] = key[4 * v + 2] = key[4 * v + 3] = 0u;
        }
      }
    } else {
#pragma unroll
      for (int e = 0; e < KPT; ++e) key[e] = (i0 + e < NG) ? score_key(R[i0 + e]) : 0u;
    }
  } else {
#pragma unroll
    for (int e = 0; e < KPT; ++e) key[e] = (i0 + e < NG) ? score_key(R[i0 + e]) : 0u;
  }
  // A real key is never 0: score_key maps -NaN (all ones) to 0 only for the pattern 0xffffffff;
  // give that one pattern the next key up so that padding stays strictly below every real key.
#pragma unroll
  for (int e = 0; e < KPT; ++e) if (i0 + e < NG && key[e] == 0u) key[e] = 1u;
  __syncthreads();                             // hist is cleared

  // ---- pass 1: top 12 bits of every key -----------------------------------------------------------
#pragma unroll
  for (int e = 0; e < KPT; ++e) if (i0 + e < NG) atomicAdd(&hist[key[e] >> 20], 1);
  __syncthreads();
  find_bin(hist, kBins, Mp, warp_tot, &sh_bin, &sh_want, &sh_cnt);
  __syncthreads();
  uint32_t prefix = uint32_t(sh_bin) << 20;    // known high bits of the M'-th key
  uint32_t known = 0xfff00000u;
  int want = sh_want, cnt = sh_cnt;
  uint32_t kth;                                // keys > kth are selected, plus need_eq keys == kth
  int need_eq;
  if (cnt == want) { kth = prefix - 1u; need_eq = 0; }        // the whole bin is taken (prefix > 0 here)
  else {
    // ---- pass 2: next 12 bits of the candidates ------------------------------------------------------
    for (int i = threadIdx.x; i < kBins; i += kThreads) hist[i] = 0;
    __syncthreads();
#pragma unroll
    for (int e = 0; e < KPT; ++e)
      if ((key[e] & known) == prefix && i0 + e < NG) atomicAdd(&hist[(key[e] >> 8) & 0xfffu], 1);
    __syncthreads();
    find_bin(hist, kBins, want, warp_tot, &sh_bin, &sh_want, &sh_cnt);
    __syncthreads();
    prefix |= uint32_t(sh_bin) << 8;
    known = 0xffffff00u;
    want = sh_want; cnt = sh_cnt;
    if (cnt == want) { kth = prefix - 1u; need_eq = 0; }
    else {
      // ---- pass 3: last 8 bits ---------------------------------------------------------------------
      if (threadIdx.x < 256) hist[threadIdx.x] = 0;
      __syncthreads();
#pragma unroll
      for (int e = 0; e < KPT; ++e)
        if ((key[e] & known) == prefix && i0 + e < NG) atomicAdd(&hist[key[e] & 0xffu], 1);
      __syncthreads();
      find_bin(hist, 256, want, warp_tot, &sh_bin, &sh_want, &sh_cnt);
      __syncthreads();
      kth = prefix | uint32_t(sh_bin);
      need_eq = sh_want;                       // equal keys to take, lowest indices first
    }
  }

  // ---- stable compaction in index order: one scan carries both counts ----------------------------------
  int n_gt = 0, n_eq = 0;
#pragma unroll
  for (int e = 0; e < KPT; ++e) { n_gt += (key[e] > kth); n_eq += (key[e] == kth); }
  const int packed = block_inclusive_scan((n_gt << 16) | n_eq, warp_tot) - ((n_gt << 16) | n_eq);
  const int gt_before = packed >> 16, eq_before = packed & 0xffff;
  int eq_take = max(0, min(n_eq, need_eq - eq_before));
  int pos = gt_before + min(eq_before, need_eq);
#pragma unroll
  for (int e = 0; e < KPT; ++e) {
    bool take = key[e] > kth;
    if (key[e] == kth && eq_take > 0) { take = true; --eq_take; }
    if (take) out[pos++] = i0 + e;
  }
}


}  // namespace

cudaError_t launch_topk_select(const Problem& p, const float* scores, int32_t* group_idx, int32_t* n_selected,
                               cudaStream_t st) {
  const dim3 grid(p.B * p.S), block(kThreads);
  if (p.NG <= kThreads) return launch_pdl(topk_select_regs_kernel<1>, grid, block, 0, st, p, scores, group_idx, n_selected);
  if (p.NG <= 4 * kThreads) return launch_pdl(topk_select_regs_kernel<4>, grid, block, 0, st, p, scores, group_idx, n_selected);
  if (p.NG <= 16 * kThreads) return launch_pdl(topk_select_regs_kernel<16>, grid, block, 0, st, p, scores, group_idx, n_selected);
  const int keys_in_smem = (p.NG <= kMaxSmemKeys) ? 1 : 0;
  const size_t smem = keys_in_smem ? sizeof(uint32_t) * size_t(p.NG) : 0;
  if (smem > 40 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(topk_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
  }
  return launch_pdl(topk_select_kernel, grid, block, smem, st, p, scores, group_idx, n_selected, keys_in_smem);
}

namespace {

template <int P>
__global__ void __launch_bounds__(kPartThreads)
topk_parts_kernel(Problem p, const float* __restrict__ scores, uint32_t* __restrict__ top_hist,
                  int32_t* __restrict__ group_idx, int32_t* __restrict__ n_selected) {
  topk_parts_body<P>(p, scores, top_hist, group_idx, n_selected, blockIdx.x, blockIdx.y, gridDim.y);
}

// Rows of partials one CTA merges, D threads and one named barrier (1 .. 14) each; barrier 15 is the
// query build's.
template <int D> constexpr int kCombineRows = (kPartThreads / D < 14) ? kPartThreads / D : 14;

// The select of one layer beside the split-K combine of another in one launch: the first CTAs merge
// kCombineRows (sequence, head) rows of partials each, the other P * problems CTAs select.  Both are short,
// latency-bound kernels; side by side they cost the longer of the two, and one launch gap.
//
// The combine CTAs have nothing to do until the gather before them has finished.  With q_ahead they
// use that time for the summed low-rank queries of the layer whose scorer is enqueued next (row sets
// cta, cta + n_comb, ..): half of the CTA's threads run the scorer's own build_queries() and store the
// rows where that scorer looks for them, so that it starts on its tiles as soon as this kernel ends.
template <int P, int D>
__global__ void __launch_bounds__(kPartThreads)
combine_select_kernel(Problem p, const float* __restrict__ scores, uint32_t* __restrict__ top_hist,
                      int32_t* __restrict__ group_idx, int32_t* __restrict__ n_selected, int n_probs,
                      const float* __restrict__ partial, float* __restrict__ out, float* __restrict__ lse, int splits,
                      int n_rows, int n_comb, const void* __restrict__ q_ahead, const float* __restrict__ proj_ahead,
                      float* __restrict__ uq_ahead, int n_rests, int n_sub) {
  constexpr int kRows = kCombineRows<D>;             // rows of partials merged per CTA
  if (int(blockIdx.x) >= n_comb) {
    const int t = int(blockIdx.x) - n_comb;
    topk_parts_body<P>(p, scores, top_hist, group_idx, n_selected, t % P, t / P, n_probs);
    return;
  }
  __shared__ float w_s[kRows][kMaxSplits];
  __shared__ float norm_s[kRows][2];
  __shared__ float qsum[kQuerySumFloats], upart[kQueryPartFloats], urow[kQueryCols * 32];
  pdl_trigger();
  if (q_ahead != nullptr && threadIdx.x < kQueryThreads) {
    for (int rest = blockIdx.x; rest < n_rests; rest += n_comb) {
      const RowSet rs = row_set(p, rest, n_sub);
      build_queries<15>(p, q_ahead, proj_ahead, rs, qsum, upart, urow);
      store_queries(p, rs, urow, uq_ahead);
      asm volatile("bar.sync 15, %0;" ::"n"(kQueryThreads) : "memory");       // urow is free for the next row set
    }
  }
  pdl_wait();
  const int slot = int(threadIdx.x) / D;
  if (slot >= kRows) return;
  const int64_t row = int64_t(blockIdx.x) * kRows + slot;
  combine_row<D>(partial, out, lse, splits, row, row < n_rows, int(threadIdx.x) % D, w_s[slot], norm_s[slot], 1 + slot);
}

}  // namespace

bool topk_parts_supported(const Problem& p) { return plan_topk_parts(p) > 0; }

cudaError_t launch_topk_parts(const Problem& p, const float* scores, uint32_t* top_hist, int32_t* group_idx,
                              int32_t* n_selected, cudaStream_t st) {
  const int P = plan_topk_parts(p);
  if (P == 0) return cudaErrorInvalidValue;
  const dim3 grid(P, p.B * p.S), block(kPartThreads);
  auto go = [&](auto kern) { return launch_pdl(kern, grid, block, 0, st, p, scores, top_hist, group_idx, n_selected); };
  return P == 1 ? go(topk_parts_kernel<1>) : P == 2 ? go(topk_parts_kernel<2>) : go(topk_parts_kernel<4>);
}

cudaError_t launch_combine_select(const Problem& p, const float* scores, uint32_t* top_hist, int32_t* group_idx,
                                  int32_t* n_selected, const float* partial, float* out, float* lse, int splits,
                                  int n_rows, int d, const void* q_ahead, const float* proj_ahead, float* uq_ahead,
                                  cudaStream_t st) {
  const int P = plan_topk_parts(p);
  if (P == 0 || (d != 64 && d != 128) || splits > kMaxSplits) return cudaErrorInvalidValue;
  int n_rests = 0, n_sub = 1;
  if (q_ahead != nullptr) {
    if (!score_stream_fuses_query(p) || proj_ahead == nullptr || uq_ahead == nullptr) return cudaErrorInvalidValue;
    score_stream_row_sets(p, &n_rests, &n_sub);
  }
  const int n_probs = p.B * p.S;
  const int rows_per_cta = (d == 128) ? kCombineRows<128> : kCombineRows<64>;
  const int n_comb = (n_rows + rows_per_cta - 1) / rows_per_cta;
  const dim3 grid(n_comb + P * n_probs), block(kPartThreads);
  auto go = [&](auto kern) {
    return launch_pdl(kern, grid, block, 0, st, p, scores, top_hist, group_idx, n_selected, n_probs, partial, out, lse,
                      splits, n_rows, n_comb, q_ahead, proj_ahead, uq_ahead, n_rests, n_sub);
  };
  if (d == 128) return P == 1 ? go(combine_select_kernel<1, 128>) : P == 2 ? go(combine_select_kernel<2, 128>) : go(combine_select_kernel<4, 128>);
  return P == 1 ? go(combine_select_kernel<1, 64>) : P == 2 ? go(combine_select_kernel<2, 64>) : go(combine_select_kernel<4, 64>);
}

}  // namespace kvswap
