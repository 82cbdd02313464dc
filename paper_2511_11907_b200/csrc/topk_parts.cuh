// TopK over group scores whose leading digit the scorer has already counted: the per-CTA body, shared
// by the stand-alone kernel and by the kernel that runs it beside the split-K combine (topk_select.cu).
#pragma once

#include "async_copy.cuh"
#include "common.cuh"
#include "topk_keys.cuh"

namespace kvswap {

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

// Body of the select for CTA `part` of problem `prob` (of n_probs); all kPartThreads threads of the CTA call.
template <int P>
__device__ __forceinline__ void topk_parts_body(const Problem& p, const float* __restrict__ scores,
                                                uint32_t* __restrict__ top_hist, int32_t* __restrict__ group_idx,
                                                int32_t* __restrict__ n_selected, int part, int prob, int n_probs) {
  constexpr int kBins = kKeyTopBins;
  static_assert(kBins == 4 * kPartThreads, "layout of the bin search");
  __shared__ int hist[kBins];
  __shared__ int warp_tot[kPartWarps];
  __shared__ uint32_t warp_own[kPartWarps], warp_before[kPartWarps];
  __shared__ int sh_bin, sh_want, sh_cnt, sh_few, sh_last;
  __shared__ uint32_t few[32];
  constexpr uint32_t kAll = 0xffffffffu;

  const int NG = p.NG, Mp = p.Mp;
  const int tid = threadIdx.x;
  reinterpret_cast<int4*>(hist)[tid] = make_int4(0, 0, 0, 0);
  if (tid == 0) { sh_bin = 0; sh_want = 1; sh_cnt = 0; sh_few = 0; }
  if ((p.flags & kFlagInputsTwoBack) == 0) pdl_wait();
  pdl_trigger();
  const float* R = scores + int64_t(prob) * p.score_pitch;
  int32_t* out = group_idx + int64_t(prob) * p.M;

  // ---- the scorer's histogram of leading digits: the thread's 4 bins, counted from the top, and all
  // keys of the row (0 = padding, below every real key): every load of the kernel goes out here ----------
  const int base = kBins - 4 * (tid + 1);
  uint2* H = reinterpret_cast<uint2*>(top_hist + int64_t(prob) * (kKeyTopBins / 2) + base / 2);
  uint32_t* ticket = top_hist + int64_t(n_probs) * (kKeyTopBins / 2) + prob;
  // (loads that bypass L1: with kFlagInputsTwoBack the CTA has passed no dependency wait of its own)
  const uint2 h = __ldcg(H);
  uint32_t key[P][4];
  const bool vec = (p.score_pitch & 3) == 0;   // rows start 16-byte aligned and are padded to whole vectors
#pragma unroll
  for (int q = 0; q < P; ++q) {
    const int i = q * kPartKeys + 4 * tid;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (vec) {
      if (i < NG) x = __ldcg(reinterpret_cast<const float4*>(R + i));
    } else {
      if (i < NG) x.x = __ldcg(R + i);
      if (i + 1 < NG) x.y = __ldcg(R + i + 1);
      if (i + 2 < NG) x.z = __ldcg(R + i + 2);
      if (i + 3 < NG) x.w = __ldcg(R + i + 3);
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


// CTAs per problem of this select: parts of 4096 keys; 0 when the row is too long for it.
inline int plan_topk_parts(const Problem& p) {
  if (p.NG < 1 || p.NG > kMaxParts * kPartKeys || int64_t(p.B) * p.S > 65535) return 0;
  const int need = (p.NG + kPartKeys - 1) / kPartKeys;
  return need <= 1 ? 1 : need <= 2 ? 2 : 4;
}

}  // namespace kvswap
