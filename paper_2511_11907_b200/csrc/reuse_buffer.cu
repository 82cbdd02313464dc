// Reuse buffer (Sec. 4.4.2): a fixed set of slots, each holding the K/V rows of one group, in
// front of a slower tier that holds the whole cache; a slot table records which group a slot
// holds; groups the predictor selects are served from their slot when present (hit) and are
// otherwise fetched into the next slot in FIFO order (miss).
//
//   reuse_lookup_kernel   one CTA per (sequence, selection scope).  The sequential rule "in list
//                         order, a miss takes the next slot in FIFO order that does not serve
//                         this step" is evaluated in parallel: hits mark their slots busy; the
//                         misses are ranked in list order and the non-busy slots in FIFO order
//                         (one block scan each); the k-th miss takes the k-th such slot.
//   reuse_fill_kernel     one CTA per missed group: copies its G rows of K and V from the slow
//                         tier (any device-accessible memory, e.g. pinned host memory) into the slot.
//
// State of one buffer set (caller-owned device memory, one per layer), int32 words:
//   head[B*S] | slot_group[B*S*C] | group_slot[B*S*max_groups]
// group_slot is the inverse of the slot table (-1: the group is in no slot), so a lookup is
// one read.
#include <algorithm>

#include "async_copy.cuh"
#include "common.cuh"

namespace kvswap {
namespace {

constexpr int kThreads = 1024;
constexpr int kMaxPerThread = 8;              // selected groups per thread: M <= 8192
constexpr int kMaxSlots = 32768;              // busy flags live in shared memory, one byte each

// Exclusive prefix sum of `v` over the CTA; *total receives the sum.  `warp_tot`: 32 ints.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_tot, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += t;
  }
  __syncthreads();                            // warp_tot may still be read from a previous scan
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = warp_tot[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, w, off);
      if (lane >= off) w += t;
    }
    warp_tot[lane] = w;
  }
  __syncthreads();
  *total = warp_tot[31];
  return incl - v + (warp > 0 ? warp_tot[warp - 1] : 0);
}

__global__ void __launch_bounds__(kThreads)
reuse_lookup_kernel(int M, int NG, int C, int max_groups, const int32_t* __restrict__ group_idx,
                    const int32_t* __restrict__ n_selected, int32_t* __restrict__ head_all,
                    int32_t* __restrict__ slot_group_all, int32_t* __restrict__ group_slot_all,
                    int32_t* __restrict__ slot_idx, int32_t* __restrict__ miss_group, int32_t* __restrict__ miss_slot,
                    int32_t* __restrict__ n_miss_out) {
  extern __shared__ unsigned char smem[];
  unsigned char* busy = smem;                                    // [C]
  int32_t* victim = reinterpret_cast<int32_t*>(smem + ((C + 15) & ~15));   // [M]
  __shared__ int warp_tot[32];

  const int prob = blockIdx.x;
  const int32_t* idx = group_idx + int64_t(prob) * M;
  int32_t* slot_group = slot_group_all + int64_t(prob) * C;
  int32_t* group_slot = group_slot_all + int64_t(prob) * max_groups;
  const int head = head_all[prob];
  const int n_sel = max(0, min(n_selected[prob], M));

  for (int c = threadIdx.x; c < C; c += kThreads) busy[c] = 0;
  __syncthreads();

  // ---- this thread's consecutive list entries: group, slot if present ---------------------------------
  const int per = (M + kThreads - 1) / kThreads;                 // <= kMaxPerThread
  const int i0 = int(threadIdx.x) * per;
  int grp[kMaxPerThread], slot[kMaxPerThread];
  int my_miss = 0;
#pragma unroll
  for (int e = 0; e < kMaxPerThread; ++e) {
    grp[e] = -1; slot[e] = -1;
    const int i = i0 + e;
    if (e < per && i < n_sel) {
      const int j = idx[i];
      if (j >= 0 && j < NG) {
        grp[e] = j;
        slot[e] = group_slot[j];
        if (slot[e] >= 0) busy[slot[e]] = 1;
        else atomicMin(&group_slot[j], -2 - (M - i));          // claim (< -1): of a group listed twice the first entry, with the lowest mark, loads it
      }
    }
  }
  __syncthreads();
  bool loads[kMaxPerThread];
#pragma unroll
  for (int e = 0; e < kMaxPerThread; ++e) {
    loads[e] = false;
    if (grp[e] >= 0 && slot[e] < 0) {
      slot[e] = -1;                                            // a claim read in the first pass is not a slot
      loads[e] = group_slot[grp[e]] == -2 - (M - (i0 + e));
      my_miss += loads[e] ? 1 : 0;
    }
  }
  int n_miss;
  int rank = block_exclusive_scan(my_miss, warp_tot, &n_miss);   // list-order rank of my first miss
  // (the scan's barriers also order the busy[] writes before the reads below)

  // ---- the slots that do not serve this step, in FIFO order from the head ------------------------------
  const int per_c = (C + kThreads - 1) / kThreads;
  const int p0 = int(threadIdx.x) * per_c;
  int my_free = 0;
  for (int e = 0; e < per_c; ++e) {
    const int pos = p0 + e;
    if (pos < C) {
      int c = head + pos; if (c >= C) c -= C;
      my_free += busy[c] ? 0 : 1;
    }
  }
  int n_free;
  int frank = block_exclusive_scan(my_free, warp_tot, &n_free);
  for (int e = 0; e < per_c; ++e) {
    const int pos = p0 + e;
    if (pos < C) {
      int c = head + pos; if (c >= C) c -= C;
      if (!busy[c]) { if (frank < n_miss) victim[frank] = c; ++frank; }
    }
  }
  __syncthreads();
  // n_free >= n_miss because C >= M >= hits + loads (checked on the host).

  // ---- serve the list ---------------------------------------------------------------------------------------
#pragma unroll
  for (int e = 0; e < kMaxPerThread; ++e) {
    const int i = i0 + e;
    if (e < per && i < M) {
      int s = slot[e];
      if (loads[e]) {
        s = victim[rank];
        const int old = slot_group[s];
        if (old >= 0) group_slot[old] = -1;                     // `old` is not selected in this step
        slot_group[s] = grp[e];
        group_slot[grp[e]] = s;
        miss_group[int64_t(prob) * M + rank] = grp[e];
        miss_slot[int64_t(prob) * M + rank] = s;
        ++rank;
      }
      slot[e] = s;
    }
  }
  __syncthreads();                                             // the loaders' table entries are in place
#pragma unroll
  for (int e = 0; e < kMaxPerThread; ++e) {
    const int i = i0 + e;
    if (e < per && i < M) {
      int s = slot[e];
      if (grp[e] >= 0 && s < 0) s = group_slot[grp[e]];        // a repeated entry: the slot its first entry loaded
      slot_idx[int64_t(prob) * M + i] = s;
    }
  }
  for (int k = n_miss + threadIdx.x; k < M; k += kThreads) {
    miss_group[int64_t(prob) * M + k] = -1;
    miss_slot[int64_t(prob) * M + k] = -1;
  }
  if (threadIdx.x == 0) {
    n_miss_out[prob] = n_miss;
    if (n_miss > 0) { int h = victim[n_miss - 1] + 1; head_all[prob] = (h >= C) ? 0 : h; }
  }
}

// One CTA per (miss ordinal, sequence x scope).  Rows are copied in 16-byte pieces.
__global__ void __launch_bounds__(256)
reuse_fill_kernel(Problem p, int M, int C, const unsigned char* __restrict__ K_slow,
                  const unsigned char* __restrict__ V_slow, unsigned char* __restrict__ K_reuse,
                  unsigned char* __restrict__ V_reuse, const int32_t* __restrict__ miss_group,
                  const int32_t* __restrict__ miss_slot, const int32_t* __restrict__ n_miss, int elem_bytes) {
  const int prob = blockIdx.y, k = blockIdx.x;
  if (k >= n_miss[prob]) return;
  const int j = miss_group[int64_t(prob) * M + k], slot = miss_slot[int64_t(prob) * M + k];
  if (j < 0 || slot < 0) return;
  const int b = prob / p.S, s = prob % p.S;
  const int g_first = (p.scope == KVSWAP_SCOPE_KV_HEAD) ? s : 0;
  const int g_count = (p.scope == KVSWAP_SCOPE_KV_HEAD) ? 1 : p.Hkv;
  const int pieces = p.d * elem_bytes / 16;                      // per row
  const int64_t R = int64_t(C + 1) * p.G;                        // rows per head of the reuse store
  const int total = 2 * g_count * p.G * pieces;
  for (int t = threadIdx.x; t < total; t += blockDim.x) {
    const int piece = t % pieces;
    const int row = (t / pieces) % p.G;
    const int gi = (t / (pieces * p.G)) % g_count;
    const bool is_v = t >= g_count * p.G * pieces;
    const int g = g_first + gi;
    const int64_t src = (int64_t(b) * p.kv_sb + int64_t(g) * p.kv_sh + (int64_t(j) * p.G + row) * p.kv_sn) * elem_bytes +
                        piece * 16;
    const int64_t dst = ((int64_t(b) * p.Hkv + g) * R + int64_t(slot) * p.G + row) * p.d * elem_bytes + piece * 16;
    const uint4 v = *reinterpret_cast<const uint4*>((is_v ? V_slow : K_slow) + src);
    *reinterpret_cast<uint4*>((is_v ? V_reuse : K_reuse) + dst) = v;
  }
}

__global__ void reuse_init_kernel(int32_t* state, int64_t n_head, int64_t n_total) {
  for (int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n_total; i += int64_t(gridDim.x) * blockDim.x)
    state[i] = (i < n_head) ? 0 : -1;
}

}  // namespace

bool reuse_supported(const Problem& p, int n_slots, int max_groups) {
  return n_slots >= p.M && n_slots <= kMaxSlots && p.M <= kThreads * kMaxPerThread && max_groups >= 1;
}

size_t reuse_state_words(const Problem& p, int n_slots, int max_groups) {
  const size_t probs = size_t(p.B) * p.S;
  return probs * (size_t(1) + size_t(n_slots) + size_t(max_groups));
}

cudaError_t launch_reuse_init(const Problem& p, int n_slots, int max_groups, int32_t* state, cudaStream_t st) {
  const int64_t n_head = int64_t(p.B) * p.S, n_total = int64_t(reuse_state_words(p, n_slots, max_groups));
  const int blocks = int(std::min<int64_t>(1024, (n_total + 255) / 256));
  reuse_init_kernel<<<blocks, 256, 0, st>>>(state, n_head, n_total);
  return cudaGetLastError();
}

cudaError_t launch_reuse_lookup(const Problem& p, int n_slots, int max_groups, const int32_t* group_idx,
                                const int32_t* n_selected, int32_t* state, int32_t* slot_idx, int32_t* miss_group,
                                int32_t* miss_slot, int32_t* n_miss, cudaStream_t st) {
  const int64_t probs = int64_t(p.B) * p.S;
  int32_t* head = state;
  int32_t* slot_group = head + probs;
  int32_t* group_slot = slot_group + probs * n_slots;
  const size_t smem = size_t((n_slots + 15) & ~15) + sizeof(int32_t) * size_t(p.M);
  if (smem > 40 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(reuse_lookup_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
  }
  reuse_lookup_kernel<<<int(probs), kThreads, smem, st>>>(p.M, std::min(p.NG, max_groups), n_slots, max_groups, group_idx,
                                                          n_selected, head, slot_group, group_slot, slot_idx, miss_group,
                                                          miss_slot, n_miss);
  return cudaGetLastError();
}

cudaError_t launch_reuse_fill(const Problem& p, int n_slots, const void* K_slow, const void* V_slow, void* K_reuse,
                              void* V_reuse, const int32_t* miss_group, const int32_t* miss_slot, const int32_t* n_miss,
                              cudaStream_t st) {
  const int e = (p.kv_dtype == KVSWAP_F32) ? 4 : 2;
  reuse_fill_kernel<<<dim3(p.M, p.B * p.S), 256, 0, st>>>(
      p, p.M, n_slots, static_cast<const unsigned char*>(K_slow), static_cast<const unsigned char*>(V_slow),
      static_cast<unsigned char*>(K_reuse), static_cast<unsigned char*>(V_reuse), miss_group, miss_slot, n_miss, e);
  return cudaGetLastError();
}

}  // namespace kvswap
