// K3: TopK over group scores (Sec. 4.3): per (sequence, scope) the M' = min(M, NG) groups with
// the largest score, lower index first among equal scores, written in ascending index order.
//
// One CTA per problem.  Scores become order-preserving 32-bit keys; an MSB-first radix select
// (8 bits per pass) finds the key of rank M' and how many groups equal to it are still needed;
// a stable compaction in index order then emits the selection.
#include "common.cuh"

namespace kvswap {
namespace {

constexpr int kThreads = 1024;
constexpr int kMaxSmemKeys = 48 * 1024;   // 192 KB of keys kept on chip; longer rows re-read L2

__device__ __forceinline__ uint32_t score_key(float f) {
  uint32_t u = __float_as_uint(f);
  if (u == 0x80000000u) u = 0u;                       // -0 and +0 are the same score
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // larger score <=> larger key
}

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

  const int prob = blockIdx.x;                 // b * S + s
  const float* R = scores + int64_t(prob) * p.NG;
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

}  // namespace

cudaError_t launch_topk_select(const Problem& p, const float* scores, int32_t* group_idx, int32_t* n_selected,
                               cudaStream_t st) {
  const int keys_in_smem = (p.NG <= kMaxSmemKeys) ? 1 : 0;
  const size_t smem = keys_in_smem ? sizeof(uint32_t) * size_t(p.NG) : 0;
  if (smem > 40 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(topk_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
  }
  topk_select_kernel<<<p.B * p.S, kThreads, smem, st>>>(p, scores, group_idx, n_selected, keys_in_smem);
  return cudaGetLastError();
}

}  // namespace kvswap
