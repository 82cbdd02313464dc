// Host-side helpers shared by the files that implement the C ABI (api.cu, step.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace kvswap {
inline bool misaligned(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) != 0; }
int dtype_bytes(int t);

// Defined in api.cu.
// Argument checks of kvswap_score_select; fills the problem and the workspace plan.
int check_score_select(const kvswap_shape* shape, const void* q, const float* proj, const void* meta,
                       const int32_t* group_idx, const int32_t* n_selected, const float* group_scores_opt,
                       const void* ws, size_t ws_bytes, Problem* p, Workspace* w);
// The predictor of one layer in two halves (arguments already checked): scorer, then TopK.
// uq_ahead = 0 or 1: the summed low-rank queries are already in that one of the workspace's two query
// buffers (select_with_combine_launch put them there), and q is not read; -1: the scorer forms them.
cudaError_t score_launch(const Problem& p_in, const Workspace& w, const void* q, const float* proj, const void* meta,
                         float* group_scores_opt, void* ws, cudaStream_t stream, int uq_ahead = -1);
cudaError_t select_launch(const Problem& p_in, const Workspace& w, int32_t* group_idx, int32_t* n_selected,
                          float* group_scores_opt, void* ws, cudaStream_t stream);
// select_launch merged with the combine pass of a split-K gather enqueued before it (one launch);
// false when this shape's select has no such kernel.  With q_ahead the launch also forms the summed
// low-rank queries of the layer with that q and proj_ahead into query buffer uq_ahead (0 or 1) of the
// workspace, where this shape's scorer can take them from (query_ahead_supported).
bool select_with_combine_launch(const Problem& p_in, const Workspace& w, int32_t* group_idx, int32_t* n_selected,
                                void* ws, const float* partial, float* out, float* lse, int splits, int n_rows, int d,
                                cudaStream_t stream, cudaError_t* result, const void* q_ahead = nullptr,
                                const float* proj_ahead = nullptr, int uq_ahead = -1);
bool query_ahead_supported(const Problem& p);
// True when select_with_combine_launch has a kernel for this shape's select.
bool select_merges_with_combine(const Problem& p);
// Both halves back to back.
cudaError_t score_select_launch(const Problem& p_in, const Workspace& w, const void* q,
                                const float* proj, const void* meta, int32_t* group_idx, int32_t* n_selected,
                                float* group_scores_opt, void* ws, cudaStream_t stream);
// Checks shared by the append calls; on success `p` describes the grown context (N + 1 tokens).
int resolve_grown(const kvswap_shape* shape, Problem* p);
// Checks shared by the reuse-buffer calls.
int resolve_reuse(const kvswap_shape* shape, int32_t n_slots, int32_t max_groups, Problem* p);
}  // namespace kvswap
