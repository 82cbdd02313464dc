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
#include "common.cuh"
#include "topk_keys.cuh"

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


// ------------------------------------------------------------------------------------------
// Select for rows whose first digit the scorer has already counted (top_hist: per problem a
// histogram of the keys' leading 12 bits, 16-bit counters), spread over P CTAs per problem.
//
// A row is cut into P parts of 4096 keys.  Every CTA of a problem (1024 threads) keeps all of the
// row's keys in registers -- thread t holds keys 4t..4t+3 of each part, one 16-byte load per part
// -- finds the bin of the M'-th key in the scorer's histogram and runs the remaining digits over
// its registers, so the CTAs of a problem agree on the threshold without exchanging a word.  Each
// then writes the selected groups of its own part only: where they go is the number of selected
// groups in the parts before it (a block-wide sum over the same registers) plus a scan inside the
// part.  The scorer never writes -0 and no finite score maps to key 0, so here a key is two
// instructions (the -0 and key-0 cases of score_key() cannot occur) and 0 marks padding.
// ------------------------------------------------------------------------------------------
constexpr int kPartThreads = 1024;
constexpr int kPartWarps = kPartThreads / 32;
constexpr int kPartKeys = 4 * kPartThreads;  // keys per part
constexpr int kMaxParts = 4;
constexpr int kFewKeys = 32;                 // candidates that one warp ranks directly instead of by another digit

// Thread t holds the populations c[0..3] of bins base .. base + 3, base = 4096 - 4 (t + 1): the
// CTA's threads cover the histogram from the top.  Finds the bin that holds the candidate of
// descending rank `want` (1-based) and publishes (bin, rank inside the bin, its population).
// Warp sums (one reduction instruction each) meet in shared memory; every warp scans the 32 sums
// itself, and only the warp that holds the rank looks inside its threads.  One barrier inside;
// the caller's next barrier publishes the result and frees `warp_tot` for the next use.
__device__ __forceinline__ void part_find_bin(const int (&c)[4], int base, int want, int* warp_tot, int* sh_bin,
                                              int* sh_want, int* sh_cnt) {
  constexpr uint32_t kAll = 0xffffffffu;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int local = (c[0] + c[1]) + (c[2] + c[3]);
  const int wsum = __reduce_add_sync(kAll, local);
  if (lane == 0) warp_tot[warp] = wsum;
  __syncthreads();
  const int w = warp_tot[lane];
  int incl = w;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int t = __shfl_up_sync(kAll, incl, off);
    if (lane >= off) incl += t;
  }
  const uint32_t reached = __ballot_sync(kAll, incl >= want);
  if (reached == 0u) return;                                   // fewer candidates than `want`: leave the defaults
  const int holder = __ffs(reached) - 1;
  if (warp != holder) return;
  int acc = __shfl_sync(kAll, incl - w, holder);               // candidates in the warps above this one
  int mine = local;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int t = __shfl_up_sync(kAll, mine, off);
    if (lane >= off) mine += t;
  }
  acc += mine - local;                                         // ... and in the threads above this one
  if (acc < want && acc + local >= want) {
#pragma unroll
    for (int i = 3; i >= 0; --i) {
      if (acc < want && acc + c[i] >= want) { *sh_bin = base + i; *sh_want = want - acc; *sh_cnt = c[i]; }
      acc += c[i];
    }
  }
}

// Key of a score the streaming scorer wrote (never -0): larger score <=> larger key.
__device__ __forceinline__ uint32_t fast_key(float f) {
  const int32_t u = __float_as_int(f);
  return uint32_t(u) ^ (uint32_t(u >> 31) | 0x80000000u);
}

template <int P>
__global__ void __launch_bounds__(kPartThreads)
topk_parts_kernel(Problem p, const float* __restrict__ scores, uint32_t* __restrict__ top_hist,
                  int32_t* __restrict__ group_idx, int32_t* __restrict__ n_selected) {
  static_assert(kKeyTopBins == kBins && kBins == 4 * kPartThreads, "layout of the bin search");
  __shared__ int hist[kBins];
  __shared__ int warp_tot[kPartWarps];
  __shared__ uint32_t warp_own[kPartWarps], warp_before[kPartWarps];
  __shared__ int sh_bin, sh_want, sh_cnt, sh_few, sh_last;
  __shared__ uint32_t few[32];
  constexpr uint32_t kAll = 0xffffffffu;

  const int part = blockIdx.x, prob = blockIdx.y;   // prob = b * S + s
  const int NG = p.NG, Mp = p.Mp;
  const int tid = threadIdx.x;
  reinterpret_cast<int4*>(hist)[tid] = make_int4(0, 0, 0, 0);
  if (tid == 0) { sh_bin = 0; sh_want = 1; sh_cnt = 0; sh_few = 0; }
  pdl_wait();
  pdl_trigger();
  const float* R = scores + int64_t(prob) * p.score_pitch;
  int32_t* out = group_idx + int64_t(prob) * p.M;

  // ---- the scorer's histogram of leading digits: the thread's 4 bins, counted from the top, and all
  // keys of the row (0 = padding, below every real key): every load of the kernel goes out here ----------
  const int base = kBins - 4 * (tid + 1);
  uint2* H = reinterpret_cast<uint2*>(top_hist + int64_t(prob) * (kKeyTopBins / 2) + base / 2);
  uint32_t* ticket = top_hist + int64_t(gridDim.y) * (kKeyTopBins / 2) + prob;
  const uint2 h = *H;
  uint32_t key[P][4];
  const bool vec = (p.score_pitch & 3) == 0;   // rows start 16-byte aligned and are padded to whole vectors
#pragma unroll
  for (int q = 0; q < P; ++q) {
    const int i = q * kPartKeys + 4 * tid;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (vec) {
      if (i < NG) x = *reinterpret_cast<const float4*>(R + i);
    } else {
      if (i < NG) x.x = R[i];
      if (i + 1 < NG) x.y = R[i + 1];
      if (i + 2 < NG) x.z = R[i + 2];
      if (i + 3 < NG) x.w = R[i + 3];
    }
    key[q][0] = (i < NG) ? fast_key(x.x) : 0u;
    key[q][1] = (i + 1 < NG) ? fast_key(x.y) : 0u;
    key[q][2] = (i + 2 < NG) ? fast_key(x.z) : 0u;
    key[q][3] = (i + 3 < NG) ? fast_key(x.w) : 0u;
  }
  int c[4] = {int(h.x & 0xffffu), int(h.x >> 16), int(h.y & 0xffffu), int(h.y >> 16)};
  const int local = (c[0] + c[1]) + (c[2] + c[3]);
  // The histogram must be zero again when the next call's scorer counts into it: the CTA of the
  // problem that draws the last ticket -- every CTA has read its counters by then -- clears it.
  uint32_t drawn = 0u;
  auto leave_hist_clear = [&]() {              // all threads call, once, after the CTA's last other barrier
    if (tid == 0) sh_last = (P == 1 || drawn == uint32_t(P - 1)) ? 1 : 0;
    __syncthreads();
    if (sh_last) {
      *H = make_uint2(0u, 0u);
      if (tid == 0 && P > 1) *ticket = 0u;
    }
  };
  // (a barrier whose predicate needs the loaded counters: every thread passes it with them in registers;
  // it also publishes the cleared shared histogram and sh_*)
  const int never = __syncthreads_or(local < 0);
  if (tid == 0 && P > 1 && !never) drawn = atomicAdd(ticket, 1u);
  if (part == 0) {
    if (tid == 0) n_selected[prob] = Mp;
    for (int i = Mp + tid; i < p.M; i += kPartThreads) out[i] = -1;
  }
  if (Mp == 0) { leave_hist_clear(); return; }
  if (Mp == NG) {                              // everything is selected
    for (int i = part * kPartKeys + tid; i < min(NG, (part + 1) * kPartKeys); i += kPartThreads) out[i] = i;
    leave_hist_clear();
    return;
  }

  part_find_bin(c, base, Mp, warp_tot, &sh_bin, &sh_want, &sh_cnt);
  __syncthreads();
  uint32_t prefix = uint32_t(sh_bin) << 20;    // known high bits of the M'-th key
  int want = sh_want, cnt = sh_cnt;
  uint32_t kth;                                // keys > kth are selected, plus need_eq keys == kth
  int need_eq;
  if (cnt == want) { kth = prefix - 1u; need_eq = 0; }        // the whole bin is taken
  else {
    // ---- next 12 bits of the candidates ----------------------------------------------------------------
    const uint32_t top = prefix >> 20;
#pragma unroll
    for (int q = 0; q < P; ++q)
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if ((key[q][e] >> 20) == top) atomicAdd(&hist[(key[q][e] >> 8) & 0xfffu], 1);
    __syncthreads();
    {
      const int4 hv = reinterpret_cast<const int4*>(hist)[kPartThreads - 1 - tid];   // bins base .. base + 3
      c[0] = hv.x; c[1] = hv.y; c[2] = hv.z; c[3] = hv.w;
    }
    part_find_bin(c, base, want, warp_tot, &sh_bin, &sh_want, &sh_cnt);
    __syncthreads();
    prefix |= uint32_t(sh_bin) << 8;
    want = sh_want; cnt = sh_cnt;
    if (cnt == want) { kth = prefix - 1u; need_eq = 0; }
    else if (cnt <= kFewKeys) {
      // ---- a handful of keys share the 24 bits: the first warp ranks their last bytes directly ---------
#pragma unroll
      for (int q = 0; q < P; ++q)
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if ((key[q][e] & 0xffffff00u) == prefix) {
            const int slot = atomicAdd(&sh_few, 1);
            if (slot < 32) few[slot] = key[q][e] & 0xffu;
          }
      __syncthreads();
      if (tid < 32) {
        const uint32_t v = (tid < cnt) ? few[tid] : 0u;
        int gt = 0, ge = 0;                          // of the cnt bytes: how many exceed mine, how many reach it
        for (int j = 0; j < cnt; ++j) {
          const uint32_t o = __shfl_sync(kAll, v, j);
          gt += (o > v); ge += (o >= v);
        }
        const uint32_t is_kth = __ballot_sync(kAll, tid < cnt && gt < want && want <= ge);
        if (is_kth != 0u && tid == __ffs(is_kth) - 1) { sh_bin = int(v); sh_want = want - gt; }
      }
      __syncthreads();
      kth = prefix | uint32_t(sh_bin);
      need_eq = sh_want;
    } else {
      // ---- last 8 bits: the top 256 bins of the cleared histogram ---------------------------------------
      reinterpret_cast<int4*>(hist)[tid] = make_int4(0, 0, 0, 0);
      __syncthreads();
#pragma unroll
      for (int q = 0; q < P; ++q)
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if ((key[q][e] & 0xffffff00u) == prefix) atomicAdd(&hist[kBins - 256 + int(key[q][e] & 0xffu)], 1);
      __syncthreads();
      {
        const int4 hv = reinterpret_cast<const int4*>(hist)[kPartThreads - 1 - tid];
        c[0] = hv.x; c[1] = hv.y; c[2] = hv.z; c[3] = hv.w;
      }
      part_find_bin(c, base, want, warp_tot, &sh_bin, &sh_want, &sh_cnt);
      __syncthreads();
      kth = prefix | uint32_t(sh_bin - (kBins - 256));
      need_eq = sh_want;                       // equal keys to take, lowest indices first
    }
  }

  // ---- stable compaction of this CTA's part: a scan inside the part (counts of keys > kth and == kth,
  // packed 16 + 16 bits) plus the totals of the parts before it ------------------------------------------------------
  uint32_t own = 0u, before = 0u;
#pragma unroll
  for (int q = 0; q < P; ++q) {
    uint32_t n_gt = 0, n_eq = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) { n_gt += (key[q][e] > kth); n_eq += (key[q][e] == kth); }
    const uint32_t pair = (n_gt << 16) | n_eq;
    if (q < part) before += pair;
    else if (q == part) own = pair;
  }
  const int lane = tid & 31, warp = tid >> 5;
  uint32_t incl = own;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t t = __shfl_up_sync(kAll, incl, off);
    if (lane >= off) incl += t;
  }
  const uint32_t before_w = __reduce_add_sync(kAll, before);
  if (lane == 31) warp_own[warp] = incl;
  if (lane == 0) warp_before[warp] = before_w;
  __syncthreads();
  uint32_t w_incl = warp_own[lane];
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t t = __shfl_up_sync(kAll, w_incl, off);
    if (lane >= off) w_incl += t;
  }
  const uint32_t warps_above = __shfl_sync(kAll, w_incl, (warp + 31) & 31);
  const uint32_t excl = incl - own + (warp > 0 ? warps_above : 0u);
  const uint32_t total_before = __reduce_add_sync(kAll, warp_before[lane]);
  const int gt_before = int(total_before >> 16) + int(excl >> 16);
  const int eq_before = int(total_before & 0xffffu) + int(excl & 0xffffu);
  int eq_take = max(0, need_eq - eq_before);   // equal keys this thread may still take
  int pos = gt_before + min(eq_before, need_eq);
#pragma unroll
  for (int q = 0; q < P; ++q) {
    if (q == part) {
      const int i0 = q * kPartKeys + 4 * tid;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        bool take = key[q][e] > kth;
        if (key[q][e] == kth && eq_take > 0) { take = true; --eq_take; }
        if (take && pos < p.M) out[pos++] = i0 + e;
      }
    }
  }
  leave_hist_clear();
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

// CTAs per problem of the select that starts from the scorer's histogram: parts of 4096 keys;
// 0 when the row is too long for it.
static int plan_topk_parts(const Problem& p) {
  if (p.NG < 1 || p.NG > kMaxParts * kPartKeys || int64_t(p.B) * p.S > 65535) return 0;
  const int need = (p.NG + kPartKeys - 1) / kPartKeys;
  return need <= 1 ? 1 : need <= 2 ? 2 : 4;
}

bool topk_parts_supported(const Problem& p) { return plan_topk_parts(p) > 0; }

cudaError_t launch_topk_parts(const Problem& p, const float* scores, uint32_t* top_hist, int32_t* group_idx,
                              int32_t* n_selected, cudaStream_t st) {
  const int P = plan_topk_parts(p);
  if (P == 0) return cudaErrorInvalidValue;
  const dim3 grid(P, p.B * p.S), block(kPartThreads);
  auto go = [&](auto kern) { return launch_pdl(kern, grid, block, 0, st, p, scores, top_hist, group_idx, n_selected); };
  return P == 1 ? go(topk_parts_kernel<1>) : P == 2 ? go(topk_parts_kernel<2>) : go(topk_parts_kernel<4>);
}

}  // namespace kvswap
