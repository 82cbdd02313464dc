// Shared declarations of the kvswap CUDA library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "kvswap.h"

namespace kvswap {

constexpr int kNumSMs = 148;  // B200: 2 dies x 74 SMs; grids are sized in multiples of this.

// Shape with every "0 = dense" stride resolved and the derived sizes filled in.
struct Problem {
  int B, N, Hq, Hkv, d, r, Hm, G, M;
  int kv_dtype, meta_dtype, q_dtype, scope;
  int flags;   // KVSWAP_INPUTS_SETTLED, KVSWAP_SCORE_SOFTMAX, kFlag*
  int meta_exp;   // 8-bit metadata stores K_lr * 2^-meta_exp (0 for the other types)
  int64_t kv_sb, kv_sh, kv_sn;
  int64_t meta_sb, meta_sh, meta_sn;
  int rho;   // H_q / H_kv
  int S;     // selections per sequence
  int NG;    // complete groups
  int Mp;    // min(M, NG)
  int Su;    // rows of the low-rank query buffer per sequence (see score_pool.cu)
  int score_pitch;   // floats between rows of the group-score buffer: NG in a caller's buffer, padded in the workspace
};

// Internal flags (never taken from a caller's shape; a decode step sets them).
// kFlagWaitEarly, on the split-K gather with KVSWAP_INPUTS_SETTLED: the dependency wait comes right after
// the first fills are requested, and only then may the kernel enqueued behind this one start.
// kFlagInputsTwoBack, on the TopK enqueued behind such a gather: its scores and counts were complete
// before the gather's wait returned, i.e. before any of its own CTAs started, and nothing it writes is
// touched by the gather: it does not wait at all.
constexpr int kFlagWaitEarly = 1 << 16;
constexpr int kFlagInputsTwoBack = 1 << 17;

// Partition of the caller's workspace (byte offsets, each 256-byte aligned).
struct Workspace {
  size_t off_uq;       // float [2][B, Su, r]    summed low-rank queries; two buffers of uq_bytes (a decode step alternates)
  size_t uq_bytes;
  size_t off_scores;   // float [B, S, NG]       group scores R (when the caller passes no buffer)
  size_t off_hist;     // uint16 [B, S, 4096] + uint32 [B, S]  leading-digit histograms of the group scores' keys and tickets, zero between calls
  size_t off_partial;  // float [B, Hq, splits, d + 2]  split-K partials (m, l, acc[d])
  size_t off_softmax;  // float [B, Hq, r] per-head low-rank queries + [B, Hq, chunks, 2] softmax statistics (scorer variant)
  size_t off_adapter;  // bf16 [H_kv, 3 r, d]       adapter split into three bf16 pieces (project_keys on tcgen05)
  size_t total;
  int splits;          // split-K factor of sparse_decode for this shape
  int heads_per_cta;   // query heads sharing one K/V pass in sparse_decode
  int depth;           // shared-memory stages per compute warp in sparse_decode
};

int resolve(const kvswap_shape* s, Problem* p);            // validation; returns kvswap_status
void plan_workspace(const Problem& p, Workspace* w);
void plan_sparse_decode(const Problem& p, Workspace* w);   // fills splits, heads_per_cta, depth

// Kernel launchers (each returns a cudaError_t from the launch).
// `scratch` is the workspace region at off_adapter (project_keys_umma_scratch_bytes, may be NULL).
cudaError_t launch_project_keys(const Problem& p, const void* K, const float* proj, void* meta,
                                int n_begin, int n_end, void* scratch, uint32_t* err, cudaStream_t st);
cudaError_t launch_append_rows(const Problem& p, const void* k_new, const void* v_new, void* const* K, void* const* V,
                               int n_layers, int n, cudaStream_t st);
cudaError_t launch_project_keys_layers(const Problem& p, const void* const* K, const float* const* proj,
                                       void* const* meta, int n_layers, int n_begin, int n_end, cudaStream_t st);
cudaError_t launch_flush_rows(const Problem& p, const void* const* K_fast, const void* const* V_fast, void* const* K_slow,
                              void* const* V_slow, int n_layers, int64_t fast_rows, int64_t fast_row0, int64_t slow_row0,
                              cudaStream_t st);
// Softmax variant of the scorer (score_softmax.cu).
int score_softmax_chunks(const Problem& p);
bool score_softmax_supported(const Problem& p);
cudaError_t launch_score_softmax(const Problem& p, const void* q, const float* proj, const void* meta, float* u,
                                 float* stats, float* scores, cudaStream_t st);
// Reuse buffer (reuse_buffer.cu).
bool reuse_supported(const Problem& p, int n_slots, int max_groups);
size_t reuse_state_words(const Problem& p, int n_slots, int max_groups);
cudaError_t launch_reuse_init(const Problem& p, int n_slots, int max_groups, int32_t* state, cudaStream_t st);
cudaError_t launch_reuse_lookup(const Problem& p, int n_slots, int max_groups, const int32_t* group_idx,
                                const int32_t* n_selected, int32_t* state, int32_t* slot_idx, int32_t* miss_group,
                                int32_t* miss_slot, int32_t* n_miss, cudaStream_t st);
cudaError_t launch_reuse_fill(const Problem& p, int n_slots, const void* K_slow, const void* V_slow, void* K_reuse,
                              void* V_reuse, const int32_t* miss_group, const int32_t* miss_slot, const int32_t* n_miss,
                              cudaStream_t st);
size_t project_keys_umma_scratch_bytes(const Problem& p);
bool try_launch_project_keys_umma(const Problem& p, const void* K, const float* proj, void* meta, int n_begin,
                                  int n_end, void* scratch, uint32_t* err, cudaStream_t st, cudaError_t* result);
cudaError_t launch_lowrank_query(const Problem& p, const void* q, const float* proj, float* uq,
                                 cudaStream_t st);
cudaError_t launch_score_pool(const Problem& p, const float* uq, const void* meta, float* scores,
                              uint32_t* err, cudaStream_t st);
// The streaming tensor-core scorer (score_stream.cu) for fp16 metadata rows of 64 bytes.  Where it
// builds the low-rank queries itself it takes q and proj (uq unused), else -- or when q is NULL --
// uq [B, Su, r] from launch_lowrank_query or from the kernel of launch_combine_select.  `top_hist` (may be NULL): per (sequence, scope) a histogram of the leading
// 12 bits of the group scores' keys (4096 16-bit counters, two per word) followed, after all
// histograms, by one ticket word per (sequence, scope).  Everything is zero on entry; the scorer
// counts, and launch_topk_parts, which starts from the counts, leaves everything zero again.
bool score_stream_supported(const Problem& p);
bool score_stream_fuses_query(const Problem& p);
bool score_stream_counts_top_digit(const Problem& p);
cudaError_t launch_score_stream(const Problem& p, const void* q, const float* proj, const float* uq,
                                const void* meta, float* scores, uint32_t* top_hist, uint32_t* err,
                                cudaStream_t st);
cudaError_t launch_topk_select(const Problem& p, const float* scores, int32_t* group_idx,
                               int32_t* n_selected, cudaStream_t st);
bool topk_parts_supported(const Problem& p);   // false: row too long for launch_topk_parts
cudaError_t launch_topk_parts(const Problem& p, const float* scores, uint32_t* top_hist,
                              int32_t* group_idx, int32_t* n_selected, cudaStream_t st);
// `combine` false: only the split-K gather runs; the caller merges the partials (launch_combine_select).
cudaError_t launch_sparse_decode(const Problem& p, const Workspace& w, const void* q, const void* K,
                                 const void* V, const int32_t* group_idx, const int32_t* n_selected,
                                 float* partial, float* out, float* lse, uint32_t* err, cudaStream_t st,
                                 bool combine = true);
cudaError_t launch_combine_only(const Problem& p, const Workspace& w, const float* partial, float* out, float* lse,
                                cudaStream_t st);
// launch_topk_parts for problem `p` and, in the same launch, the merge of `n_rows` rows of split-K
// partials [n_rows, splits, d + 2] (of whatever attention produced them) into out / lse.  With
// q_ahead != NULL the launch also builds the summed low-rank queries of another layer of the same shape
// (its q and proj) into uq_ahead [B, Su, r], for a streaming scorer that is enqueued next: the bits are
// those the scorer would build itself.  Only where score_stream_fuses_query(p).
cudaError_t launch_combine_select(const Problem& p, const float* scores, uint32_t* top_hist, int32_t* group_idx,
                                  int32_t* n_selected, const float* partial, float* out, float* lse, int splits,
                                  int n_rows, int d, const void* q_ahead, const float* proj_ahead, float* uq_ahead,
                                  cudaStream_t st);
// Row sets of the streaming scorer for `p` (0 when it does not take the shape) and scope blocks per
// (sequence, metadata head): the arguments of row_set() in lowrank_query.cuh.
void score_stream_row_sets(const Problem& p, int* n_rests, int* n_sub);

// Launch with programmatic stream serialisation: the kernel may begin (up to its
// griddepcontrol.wait) while the previous kernel in the stream is still draining.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                       Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ------------------------------------------------------------------------------------------
// Device helpers: 16-byte vector loads of storage types, widened to fp32.
// ------------------------------------------------------------------------------------------
template <typename T> struct Elt;
template <> struct Elt<float> { static constexpr int kPer16B = 4; };
template <> struct Elt<__nv_bfloat16> { static constexpr int kPer16B = 8; };
template <> struct Elt<__half> { static constexpr int kPer16B = 8; };

__device__ __forceinline__ void widen16B(const uint4& v, float (&f)[4], float) {
  f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
  f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
__device__ __forceinline__ void widen16B(const uint4& v, float (&f)[8], __nv_bfloat16) {
  // bf16 -> fp32 is a 16-bit shift of the bit pattern.
  f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
  f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
  f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
  f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
}
__device__ __forceinline__ void widen16B(const uint4& v, float (&f)[8], __half) {
  const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 t = __half22float2(h[i]);
    f[2 * i] = t.x; f[2 * i + 1] = t.y;
  }
}

// Storage of one E4M3 value (8-bit metadata): 1 sign, 4 exponent bits with bias 7, 3 mantissa bits.
struct e4m3_t { uint8_t bits; };

// Two fp32 values -> two E4M3 bytes (lo in the low byte): round to nearest even, magnitudes beyond
// 448 saturate.
__device__ __forceinline__ uint16_t to_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}

// 2^-meta_exp, the factor 8-bit metadata is stored with (1 for the other types).
__device__ __forceinline__ float meta_store_scale(const Problem& p) {
  return __uint_as_float(uint32_t(127 - p.meta_exp) << 23);
}

// 16-byte read-only global load that does not allocate in L1 (streamed once).
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

}  // namespace kvswap
