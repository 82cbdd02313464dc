// C-ABI entry points of the kvswap library, one layer at a time: host-side validation, workspace
// partition and kernel sequencing.  The calls over all layers of a model are in step.cu.  No entry
// point here allocates or keeps state; only kvswap_read_device_status synchronises.
#include <algorithm>

#include "api_internal.cuh"
#include "async_copy.cuh"
#include "common.cuh"
#include "topk_keys.cuh"

namespace kvswap {

static size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

int dtype_bytes(int t) {
  switch (t) {
    case KVSWAP_F32: return 4;
    case KVSWAP_BF16: case KVSWAP_F16: return 2;
    case KVSWAP_E4M3: return 1;
    default: return 0;
  }
}

int resolve(const kvswap_shape* s, Problem* p) {
  if (s == nullptr) return KVSWAP_ERR_NULL;
  if (s->batch < 1 || s->n_ctx < 1 || s->n_q_heads < 1 || s->n_kv_heads < 1 || s->group_size < 1 ||
      s->top_k < 1 || s->rank < 1)
    return KVSWAP_ERR_SHAPE;
  if (s->n_q_heads % s->n_kv_heads != 0) return KVSWAP_ERR_SHAPE;
  if (s->meta_heads != 1 && s->meta_heads != s->n_kv_heads) return KVSWAP_ERR_SHAPE;
  if (s->scope != KVSWAP_SCOPE_KV_HEAD && s->scope != KVSWAP_SCOPE_ALL_HEADS) return KVSWAP_ERR_SHAPE;
  if ((s->flags & ~int32_t(KVSWAP_INPUTS_SETTLED | KVSWAP_SCORE_SOFTMAX | KVSWAP_CHECK_INDICES | 0xff00)) != 0)
    return KVSWAP_ERR_SHAPE;
  const int meta_exp = int(int8_t((s->flags >> 8) & 0xff));
  if (meta_exp < -64 || meta_exp > 63 || (meta_exp != 0 && s->meta_dtype != KVSWAP_E4M3)) return KVSWAP_ERR_SHAPE;
  if (s->n_ctx > (1 << 30) || s->batch > 65535 || s->n_q_heads > 4096) return KVSWAP_ERR_SHAPE;
  const int ekv = dtype_bytes(s->kv_dtype), em = dtype_bytes(s->meta_dtype), eq = dtype_bytes(s->q_dtype);
  if (ekv == 0 || em == 0 || eq == 0) return KVSWAP_ERR_DTYPE;
  if (s->meta_dtype == KVSWAP_BF16) return KVSWAP_ERR_DTYPE;   // metadata is fp32, fp16 or E4M3
  if (s->kv_dtype == KVSWAP_E4M3 || s->q_dtype == KVSWAP_E4M3) return KVSWAP_ERR_DTYPE;   // a metadata type only
  if (s->q_dtype != KVSWAP_F32 && s->q_dtype != s->kv_dtype) return KVSWAP_ERR_DTYPE;  // q: fp32 or K/V's type
  if (s->head_dim != 64 && s->head_dim != 128) return KVSWAP_ERR_UNSUPPORTED;
  if (s->rank % 4 != 0 || s->rank > 256 || s->group_size > 1024) return KVSWAP_ERR_UNSUPPORTED;
  if (int64_t(s->top_k) * s->group_size > (int64_t(1) << 30)) return KVSWAP_ERR_UNSUPPORTED;
  if ((int64_t(s->rank) * em) % 16 != 0) return KVSWAP_ERR_ALIGN;
  if ((int64_t(s->head_dim) * eq) % 16 != 0) return KVSWAP_ERR_ALIGN;

  p->B = s->batch; p->N = s->n_ctx; p->Hq = s->n_q_heads; p->Hkv = s->n_kv_heads; p->d = s->head_dim;
  p->r = s->rank; p->Hm = s->meta_heads; p->G = s->group_size; p->M = s->top_k;
  p->kv_dtype = s->kv_dtype; p->meta_dtype = s->meta_dtype; p->q_dtype = s->q_dtype; p->scope = s->scope;
  p->flags = s->flags & 0xff;
  p->meta_exp = meta_exp;

  p->kv_sn = s->kv_stride_n ? s->kv_stride_n : p->d;
  p->kv_sh = s->kv_stride_h ? s->kv_stride_h : int64_t(p->N) * p->kv_sn;
  p->kv_sb = s->kv_stride_b ? s->kv_stride_b : int64_t(p->Hkv) * p->kv_sh;
  p->meta_sn = s->meta_stride_n ? s->meta_stride_n : p->r;
  p->meta_sh = s->meta_stride_h ? s->meta_stride_h : int64_t(p->N) * p->meta_sn;
  p->meta_sb = s->meta_stride_b ? s->meta_stride_b : int64_t(p->Hm) * p->meta_sh;
  if (p->kv_sn < p->d || p->kv_sh < 0 || p->kv_sb < 0 || p->meta_sn < p->r || p->meta_sh < 0 || p->meta_sb < 0)
    return KVSWAP_ERR_SHAPE;
  if ((p->kv_sn * ekv) % 16 || (p->kv_sh * ekv) % 16 || (p->kv_sb * ekv) % 16) return KVSWAP_ERR_ALIGN;
  if ((p->meta_sn * em) % 16 || (p->meta_sh * em) % 16 || (p->meta_sb * em) % 16) return KVSWAP_ERR_ALIGN;

  p->rho = p->Hq / p->Hkv;
  p->S = (p->scope == KVSWAP_SCOPE_KV_HEAD) ? p->Hkv : 1;
  p->NG = p->N / p->G;
  p->Mp = std::min(p->M, p->NG);
  p->Su = (p->Hm == 1) ? p->S : p->Hkv;
  p->score_pitch = p->NG;
  if ((p->flags & KVSWAP_SCORE_SOFTMAX) && !score_softmax_supported(*p)) return KVSWAP_ERR_UNSUPPORTED;
  // 8-bit metadata is read by the streaming tensor-core scorer only
  if (p->meta_dtype == KVSWAP_E4M3 && ((p->flags & KVSWAP_SCORE_SOFTMAX) || p->r != 32 || (p->NG > 0 && !score_stream_supported(*p))))
    return KVSWAP_ERR_UNSUPPORTED;
  return KVSWAP_OK;
}

// Rows of the workspace's group-score buffer are padded to whole 16-byte vectors (128 bytes), so
// that the top-k kernel can load them as vectors whatever NG is.
static int workspace_score_pitch(const Problem& p) { return (std::max(p.NG, 1) + 31) / 32 * 32; }

// Room for the leading-digit histograms (score_stream.cu, topk_select.cu) is planned from the
// batch and head counts alone, at a fixed place in front of everything else, so that one workspace
// keeps them zero between calls while the context grows.
static bool hist_capable(const Problem& p) {
  return (p.meta_dtype == KVSWAP_F16 || p.meta_dtype == KVSWAP_E4M3) && p.r == 32 && int64_t(p.B) * p.S <= 1024;
}

// The scorer counts the leading digit of every group score's key and the TopK starts from those
// counts (several CTAs per problem) where both kernels have that path.
static bool counts_top_digit(const Problem& p) {
  return !(p.flags & KVSWAP_SCORE_SOFTMAX) && hist_capable(p) && score_stream_counts_top_digit(p) && topk_parts_supported(p);
}

bool select_merges_with_combine(const Problem& p) {
  return p.NG > 0 && score_stream_supported(p) && counts_top_digit(p);
}

bool query_ahead_supported(const Problem& p) {
  return p.NG > 0 && !(p.flags & KVSWAP_SCORE_SOFTMAX) && score_stream_supported(p) && score_stream_fuses_query(p) &&
         counts_top_digit(p);
}

void plan_workspace(const Problem& p, Workspace* w) {
  plan_sparse_decode(p, w);

  size_t off = 256;  // first 256 bytes reserved
  w->off_hist = off;     off += hist_capable(p) ? align256(size_t(p.B) * p.S * (sizeof(uint16_t) * kKeyTopBins + sizeof(uint32_t))) : 0;
  w->uq_bytes = align256(sizeof(float) * size_t(p.B) * p.Su * p.r);
  w->off_uq = off;       off += 2 * w->uq_bytes;
  w->off_scores = off;   off += align256(sizeof(float) * size_t(p.B) * p.S * workspace_score_pitch(p));
  w->off_partial = off;  off += align256(sizeof(float) * size_t(p.B) * p.Hq * w->splits * (p.d + 2));
  w->off_softmax = off;  off += align256(sizeof(float) * size_t(p.B) * p.Hq * (size_t(p.r) + 2 * size_t(score_softmax_chunks(p))));
  w->off_adapter = off;  off += align256(project_keys_umma_scratch_bytes(p) + 1024);   // 1 KiB: tensor-map base alignment
  w->total = off;
}


// Argument checks of kvswap_score_select; fills the problem and the workspace plan.
int check_score_select(const kvswap_shape* shape, const void* q, const float* proj, const void* meta,
                              const int32_t* group_idx, const int32_t* n_selected, const float* group_scores_opt,
                              const void* ws, size_t ws_bytes, Problem* p, Workspace* w) {
  int st = resolve(shape, p);
  if (st != KVSWAP_OK) return st;
  if (q == nullptr || proj == nullptr || meta == nullptr || group_idx == nullptr || n_selected == nullptr ||
      ws == nullptr)
    return KVSWAP_ERR_NULL;
  if (misaligned(q) || misaligned(proj) || misaligned(meta) || misaligned(ws) ||
      (reinterpret_cast<uintptr_t>(group_idx) & 3u) || (reinterpret_cast<uintptr_t>(n_selected) & 3u) ||
      (group_scores_opt && misaligned(group_scores_opt)))
    return KVSWAP_ERR_ALIGN;
  plan_workspace(*p, w);
  if (ws_bytes < w->total) return KVSWAP_ERR_WORKSPACE;
  return KVSWAP_OK;
}

// The predictor of one layer in two halves (arguments already checked): the scorer, which leaves the
// group scores (and, where that path exists, the leading-digit histograms) in the workspace or the
// caller's buffer, and the TopK over them.  A step may put other work between the two.
cudaError_t score_launch(const Problem& p_in, const Workspace& w, const void* q, const float* proj, const void* meta,
                         float* group_scores_opt, void* ws, cudaStream_t stream, int uq_ahead) {
  char* base = static_cast<char*>(ws);
  float* uq = reinterpret_cast<float*>(base + w.off_uq + (uq_ahead > 0 ? w.uq_bytes : 0));
  float* scores = group_scores_opt ? group_scores_opt : reinterpret_cast<float*>(base + w.off_scores);
  Problem p = p_in;
  p.score_pitch = group_scores_opt ? p.NG : workspace_score_pitch(p);     // a caller's buffer is dense [B, S, NG]
  if (p.flags & KVSWAP_SCORE_SOFTMAX) {
    float* u_heads = reinterpret_cast<float*>(base + w.off_softmax);
    return launch_score_softmax(p, q, proj, meta, u_heads, u_heads + size_t(p.B) * p.Hq * p.r, scores, stream);
  }
  if (p.NG < 1) return cudaSuccess;                                       // nothing to score
  if (score_stream_supported(p)) {
    // fp16 metadata rows of 64 bytes: the tensor-core scorer, which builds the low-rank queries itself
    // where it can and counts the leading digits of its scores for the TopK that follows
    uint32_t* top_hist = counts_top_digit(p) ? reinterpret_cast<uint32_t*>(base + w.off_hist) : nullptr;
    const bool fused = score_stream_fuses_query(p);
    if (uq_ahead >= 0) {                                                  // the queries are in the workspace already
      if (!fused) return cudaErrorInvalidValue;
      return launch_score_stream(p, nullptr, proj, uq, meta, scores, top_hist, static_cast<uint32_t*>(ws), stream);
    }
    cudaError_t e = fused ? cudaSuccess : launch_lowrank_query(p, q, proj, uq, stream);
    if (e != cudaSuccess) return e;
    return launch_score_stream(p, fused ? q : nullptr, proj, uq, meta, scores, top_hist, static_cast<uint32_t*>(ws),
                               stream);
  }
  cudaError_t e = launch_lowrank_query(p, q, proj, uq, stream);
  if (e != cudaSuccess) return e;
  return launch_score_pool(p, uq, meta, scores, static_cast<uint32_t*>(ws), stream);
}

cudaError_t select_launch(const Problem& p_in, const Workspace& w, int32_t* group_idx, int32_t* n_selected,
                          float* group_scores_opt, void* ws, cudaStream_t stream) {
  char* base = static_cast<char*>(ws);
  float* scores = group_scores_opt ? group_scores_opt : reinterpret_cast<float*>(base + w.off_scores);
  Problem p = p_in;
  p.score_pitch = group_scores_opt ? p.NG : workspace_score_pitch(p);
  if (p.NG > 0 && score_stream_supported(p) && counts_top_digit(p))
    return launch_topk_parts(p, scores, reinterpret_cast<uint32_t*>(base + w.off_hist), group_idx, n_selected, stream);
  return launch_topk_select(p, scores, group_idx, n_selected, stream);
}

// select_launch for problem `p_in` merged with the combine pass of a split-K attention whose gather
// (launch_sparse_decode with combine = false, any shape) has been enqueued before: one launch.  False
// when the select of this shape has no such kernel (the caller then launches the two separately).
bool select_with_combine_launch(const Problem& p_in, const Workspace& w, int32_t* group_idx, int32_t* n_selected,
                                void* ws, const float* partial, float* out, float* lse, int splits, int n_rows, int d,
                                cudaStream_t stream, cudaError_t* result, const void* q_ahead,
                                const float* proj_ahead, int uq_ahead) {
  Problem p = p_in;
  p.score_pitch = workspace_score_pitch(p);
  if (!select_merges_with_combine(p)) return false;
  char* base = static_cast<char*>(ws);
  float* uq = reinterpret_cast<float*>(base + w.off_uq + (uq_ahead > 0 ? w.uq_bytes : 0));
  const bool ahead = q_ahead != nullptr && uq_ahead >= 0 && score_stream_fuses_query(p);
  *result = launch_combine_select(p, reinterpret_cast<float*>(base + w.off_scores),
                                  reinterpret_cast<uint32_t*>(base + w.off_hist), group_idx, n_selected, partial, out, lse,
                                  splits, n_rows, d, ahead ? q_ahead : nullptr, proj_ahead, uq, stream);
  return true;
}

cudaError_t score_select_launch(const Problem& p, const Workspace& w, const void* q, const float* proj,
                                const void* meta, int32_t* group_idx, int32_t* n_selected, float* group_scores_opt,
                                void* ws, cudaStream_t stream) {
  cudaError_t e = score_launch(p, w, q, proj, meta, group_scores_opt, ws, stream);
  if (e == cudaSuccess) e = select_launch(p, w, group_idx, n_selected, group_scores_opt, ws, stream);
  return e;
}

// Checks shared by the append calls; on success `p` describes the grown context (N + 1 tokens).
int resolve_grown(const kvswap_shape* shape, Problem* p) {
  if (shape == nullptr) return KVSWAP_ERR_NULL;
  // The store must say how many rows it has room for: dense strides would mean "exactly n_ctx".
  if (shape->kv_stride_h == 0 || shape->meta_stride_h == 0) return KVSWAP_ERR_SHAPE;
  if (shape->n_ctx >= (1 << 30)) return KVSWAP_ERR_SHAPE;
  kvswap_shape grown = *shape;
  grown.n_ctx = shape->n_ctx + 1;
  int st = resolve(&grown, p);
  if (st != KVSWAP_OK) return st;
  if (p->kv_sh < int64_t(p->N) * p->kv_sn || p->meta_sh < int64_t(p->N) * p->meta_sn) return KVSWAP_ERR_SHAPE;  // no room
  return KVSWAP_OK;
}

// Checks shared by the reuse-buffer calls.
int resolve_reuse(const kvswap_shape* shape, int32_t n_slots, int32_t max_groups, Problem* p) {
  int st = resolve(shape, p);
  if (st != KVSWAP_OK) return st;
  // max_groups = 0: a call that does not touch the slot tables (the miss gather, size queries)
  if (n_slots < 1 || max_groups < 0 || n_slots < p->M) return KVSWAP_ERR_SHAPE;
  // The tables have one entry per group id below max_groups: a context with more complete groups
  // than that could select a group the tables cannot record.
  if (max_groups > 0 && p->NG > max_groups) return KVSWAP_ERR_SHAPE;
  if (!reuse_supported(*p, n_slots, std::max(max_groups, 1))) return KVSWAP_ERR_UNSUPPORTED;
  return KVSWAP_OK;
}

}  // namespace kvswap

using namespace kvswap;

extern "C" {

size_t kvswap_workspace_bytes(const kvswap_shape* shape) {
  Problem p;
  if (resolve(shape, &p) != KVSWAP_OK) return 0;
  Workspace w;
  plan_workspace(p, &w);
  return w.total;
}

int kvswap_validate_shape(const kvswap_shape* shape) {
  Problem p;
  return resolve(shape, &p);
}

int kvswap_project_keys(const kvswap_shape* shape, const void* K, const float* proj, void* meta_out,
                        int32_t n_begin, int32_t n_end, void* ws, size_t ws_bytes, void* cuda_stream) {
  Problem p;
  int st = resolve(shape, &p);
  if (st != KVSWAP_OK) return st;
  if (K == nullptr || proj == nullptr || meta_out == nullptr) return KVSWAP_ERR_NULL;
  if (misaligned(K) || misaligned(proj) || misaligned(meta_out)) return KVSWAP_ERR_ALIGN;
  if (n_begin < 0 || n_end < n_begin || n_end > p.N) return KVSWAP_ERR_SHAPE;
  if (n_begin == n_end) return KVSWAP_OK;
  // The workspace is optional here: with one of at least kvswap_workspace_bytes() bf16 K with d in {64, 128}
  // and r in {16, 32, 64} runs on tcgen05 (it needs room for the split adapter), otherwise on the warp-level path.
  void* scratch = nullptr;
  uint32_t* err = nullptr;
  if (ws != nullptr && !misaligned(ws)) {
    Workspace w;
    plan_workspace(p, &w);
    if (ws_bytes >= w.total) {
      char* a = static_cast<char*>(ws) + w.off_adapter;
      scratch = reinterpret_cast<void*>((reinterpret_cast<uintptr_t>(a) + 1023) & ~uintptr_t(1023));
      err = static_cast<uint32_t*>(ws);
    }
  }
  cudaError_t e = launch_project_keys(p, K, proj, meta_out, n_begin, n_end, scratch, err,
                                      static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? KVSWAP_OK : KVSWAP_ERR_CUDA;
}

int kvswap_append_kv(const kvswap_shape* shape, const void* k_new, const void* v_new, void* K, void* V,
                     const float* proj, void* meta, int32_t* flushed_opt, void* cuda_stream) {
  if (flushed_opt != nullptr) *flushed_opt = 0;
  Problem p;
  int st = resolve_grown(shape, &p);
  if (st != KVSWAP_OK) return st;
  if (k_new == nullptr || v_new == nullptr || K == nullptr || V == nullptr || proj == nullptr || meta == nullptr)
    return KVSWAP_ERR_NULL;
  if (misaligned(k_new) || misaligned(v_new) || misaligned(K) || misaligned(V) || misaligned(proj) || misaligned(meta))
    return KVSWAP_ERR_ALIGN;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (launch_append_rows(p, k_new, v_new, &K, &V, 1, p.N - 1, stream) != cudaSuccess) return KVSWAP_ERR_CUDA;
  if (p.N % p.G == 0) {                                        // the new token completes a group: flush it
    if (launch_project_keys(p, K, proj, meta, p.N - p.G, p.N, nullptr, nullptr, stream) != cudaSuccess)
      return KVSWAP_ERR_CUDA;
    if (flushed_opt != nullptr) *flushed_opt = 1;
  }
  return KVSWAP_OK;
}

size_t kvswap_reuse_state_bytes(const kvswap_shape* shape, int32_t n_slots, int32_t max_groups) {
  Problem p;
  if (max_groups < 1 || resolve_reuse(shape, n_slots, max_groups, &p) != KVSWAP_OK) return 0;
  return sizeof(int32_t) * reuse_state_words(p, n_slots, max_groups);
}

int kvswap_reuse_init(const kvswap_shape* shape, int32_t n_slots, int32_t max_groups, void* state, size_t state_bytes,
                      void* cuda_stream) {
  Problem p;
  if (max_groups < 1) return KVSWAP_ERR_SHAPE;
  int st = resolve_reuse(shape, n_slots, max_groups, &p);
  if (st != KVSWAP_OK) return st;
  if (state == nullptr) return KVSWAP_ERR_NULL;
  if (misaligned(state)) return KVSWAP_ERR_ALIGN;
  if (state_bytes < sizeof(int32_t) * reuse_state_words(p, n_slots, max_groups)) return KVSWAP_ERR_WORKSPACE;
  cudaError_t e = launch_reuse_init(p, n_slots, max_groups, static_cast<int32_t*>(state),
                                    static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? KVSWAP_OK : KVSWAP_ERR_CUDA;
}

int kvswap_reuse_lookup(const kvswap_shape* shape, int32_t n_slots, int32_t max_groups, const int32_t* group_idx,
                        const int32_t* n_selected, void* state, size_t state_bytes, int32_t* slot_idx,
                        int32_t* miss_group, int32_t* miss_slot, int32_t* n_miss, void* cuda_stream) {
  Problem p;
  if (max_groups < 1) return KVSWAP_ERR_SHAPE;
  int st = resolve_reuse(shape, n_slots, max_groups, &p);
  if (st != KVSWAP_OK) return st;
  if (group_idx == nullptr || n_selected == nullptr || state == nullptr || slot_idx == nullptr ||
      miss_group == nullptr || miss_slot == nullptr || n_miss == nullptr)
    return KVSWAP_ERR_NULL;
  const void* words[] = {group_idx, n_selected, state, slot_idx, miss_group, miss_slot, n_miss};
  for (const void* w : words)
    if (reinterpret_cast<uintptr_t>(w) & 3u) return KVSWAP_ERR_ALIGN;
  if (state_bytes < sizeof(int32_t) * reuse_state_words(p, n_slots, max_groups)) return KVSWAP_ERR_WORKSPACE;
  cudaError_t e = launch_reuse_lookup(p, n_slots, max_groups, group_idx, n_selected, static_cast<int32_t*>(state),
                                      slot_idx, miss_group, miss_slot, n_miss, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? KVSWAP_OK : KVSWAP_ERR_CUDA;
}

int kvswap_reuse_fill(const kvswap_shape* shape, int32_t n_slots, const void* K_slow, const void* V_slow,
                      void* K_reuse, void* V_reuse, const int32_t* miss_group, const int32_t* miss_slot,
                      const int32_t* n_miss, void* cuda_stream) {
  Problem p;
  int st = resolve_reuse(shape, n_slots, 0, &p);
  if (st != KVSWAP_OK) return st;
  if (K_slow == nullptr || V_slow == nullptr || K_reuse == nullptr || V_reuse == nullptr || miss_group == nullptr ||
      miss_slot == nullptr || n_miss == nullptr)
    return KVSWAP_ERR_NULL;
  if (misaligned(K_slow) || misaligned(V_slow) || misaligned(K_reuse) || misaligned(V_reuse)) return KVSWAP_ERR_ALIGN;
  cudaError_t e = launch_reuse_fill(p, n_slots, K_slow, V_slow, K_reuse, V_reuse, miss_group, miss_slot, n_miss,
                                    static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? KVSWAP_OK : KVSWAP_ERR_CUDA;
}

int kvswap_score_select(const kvswap_shape* shape, const void* q, const float* proj, const void* meta,
                        int32_t* group_idx, int32_t* n_selected, float* group_scores_opt, void* ws,
                        size_t ws_bytes, void* cuda_stream) {
  Problem p;
  Workspace w;
  int st = check_score_select(shape, q, proj, meta, group_idx, n_selected, group_scores_opt, ws, ws_bytes, &p, &w);
  if (st != KVSWAP_OK) return st;
  cudaError_t e = score_select_launch(p, w, q, proj, meta, group_idx, n_selected, group_scores_opt, ws,
                                      static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? KVSWAP_OK : KVSWAP_ERR_CUDA;
}

int kvswap_sparse_decode(const kvswap_shape* shape, const void* q, const void* K, const void* V,
                         const int32_t* group_idx, const int32_t* n_selected, float* out, float* lse_opt,
                         void* ws, size_t ws_bytes, void* cuda_stream) {
  Problem p;
  int st = resolve(shape, &p);
  if (st != KVSWAP_OK) return st;
  if (q == nullptr || K == nullptr || V == nullptr || group_idx == nullptr || n_selected == nullptr ||
      out == nullptr || ws == nullptr)
    return KVSWAP_ERR_NULL;
  if (misaligned(q) || misaligned(K) || misaligned(V) || misaligned(out) || misaligned(ws) ||
      (reinterpret_cast<uintptr_t>(group_idx) & 3u) || (reinterpret_cast<uintptr_t>(n_selected) & 3u) ||
      (lse_opt && (reinterpret_cast<uintptr_t>(lse_opt) & 3u)))
    return KVSWAP_ERR_ALIGN;
  Workspace w;
  plan_workspace(p, &w);
  if (ws_bytes < w.total) return KVSWAP_ERR_WORKSPACE;
  float* partial = reinterpret_cast<float*>(static_cast<char*>(ws) + w.off_partial);
  cudaError_t e = launch_sparse_decode(p, w, q, K, V, group_idx, n_selected, partial, out, lse_opt,
                                       static_cast<uint32_t*>(ws), static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? KVSWAP_OK : KVSWAP_ERR_CUDA;
}

int kvswap_workspace_init(void* ws, size_t ws_bytes, void* cuda_stream) {
  if (ws == nullptr) return KVSWAP_ERR_NULL;
  if (ws_bytes < 256) return KVSWAP_ERR_WORKSPACE;
  // The status word and the predictor's histograms must start at zero; the rest does not care.
  return cudaMemsetAsync(ws, 0, ws_bytes, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? KVSWAP_OK
                                                                                                  : KVSWAP_ERR_CUDA;
}

int kvswap_read_device_status(const void* ws, void* cuda_stream) {
  if (ws == nullptr) return KVSWAP_ERR_NULL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint32_t word = 0;
  if (cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return KVSWAP_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return KVSWAP_ERR_CUDA;
  return word == kDevOk ? KVSWAP_OK : word == kDevBadIndex ? KVSWAP_ERR_INDEX : KVSWAP_ERR_TIMEOUT;
}

const char* kvswap_status_string(int status) {
  switch (status) {
    case KVSWAP_OK: return "ok";
    case KVSWAP_ERR_NULL: return "a required pointer is NULL";
    case KVSWAP_ERR_SHAPE: return "invalid shape, stride, range or enum value";
    case KVSWAP_ERR_DTYPE: return "unknown or unsupported dtype";
    case KVSWAP_ERR_ALIGN: return "pointer or row size is not 16-byte aligned";
    case KVSWAP_ERR_WORKSPACE: return "workspace smaller than kvswap_workspace_bytes()";
    case KVSWAP_ERR_UNSUPPORTED: return "shape outside the implemented range";
    case KVSWAP_ERR_CUDA: return "CUDA runtime or launch error";
    case KVSWAP_ERR_INDEX: return "group index out of range";
    case KVSWAP_ERR_STATIC_SCRATCH: return "problem needs more scratch than the built-in static buffer holds";
    case KVSWAP_ERR_TIMEOUT: return "a kernel gave up a bounded wait (device status word set)";
    default: return "unknown status";
  }
}

int kvswap_version(void) { return 100; }

}  // extern "C"
