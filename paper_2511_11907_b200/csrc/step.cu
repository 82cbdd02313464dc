// C-ABI entry points that serve all layers of a model in one call: the decode step over
// HBM-resident stores (one stream, each layer predicted one layer ahead of its attention), the
// decode step over reuse buffers in front of a slow tier (the predictor on a stream of its own)
// and the append steps.  The tiered step keeps one internal stream and a set of events per device;
// nothing else here keeps state.
#include <algorithm>
#include <mutex>
#include <vector>

#include "api_internal.cuh"
#include "combine.cuh"
#include "common.cuh"

using namespace kvswap;

extern "C" {

int kvswap_append_step(const kvswap_shape* shape, const kvswap_layers* layers, const void* k_new, const void* v_new,
                       int32_t* flushed_opt, void* cuda_stream) {
  if (flushed_opt != nullptr) *flushed_opt = 0;
  Problem p;
  int st = resolve_grown(shape, &p);
  if (st != KVSWAP_OK) return st;
  if (layers == nullptr || layers->K == nullptr || layers->V == nullptr || layers->meta == nullptr ||
      layers->proj == nullptr || k_new == nullptr || v_new == nullptr)
    return KVSWAP_ERR_NULL;
  if (layers->n_layers < 1) return KVSWAP_ERR_SHAPE;
  if (misaligned(k_new) || misaligned(v_new)) return KVSWAP_ERR_ALIGN;
  for (int l = 0; l < layers->n_layers; ++l) {
    if (layers->K[l] == nullptr || layers->V[l] == nullptr || layers->meta[l] == nullptr || layers->proj[l] == nullptr)
      return KVSWAP_ERR_NULL;
    if (misaligned(layers->K[l]) || misaligned(layers->V[l]) || misaligned(layers->meta[l]) ||
        misaligned(layers->proj[l]))
      return KVSWAP_ERR_ALIGN;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  // The tables are declared const for the read-only calls; this one writes the stores.
  void* const* Ks = const_cast<void* const*>(layers->K);
  void* const* Vs = const_cast<void* const*>(layers->V);
  if (launch_append_rows(p, k_new, v_new, Ks, Vs, layers->n_layers, p.N - 1, stream) != cudaSuccess)
    return KVSWAP_ERR_CUDA;
  if (p.N % p.G == 0) {
    if (launch_project_keys_layers(p, layers->K, layers->proj, const_cast<void* const*>(layers->meta),
                                   layers->n_layers, p.N - p.G, p.N, stream) != cudaSuccess)
      return KVSWAP_ERR_CUDA;
    if (flushed_opt != nullptr) *flushed_opt = 1;
  }
  return KVSWAP_OK;
}

static int check_layers(const kvswap_layers* layers, bool need_kv = true) {
  if (layers == nullptr || layers->meta == nullptr || layers->proj == nullptr) return KVSWAP_ERR_NULL;
  if (need_kv && (layers->K == nullptr || layers->V == nullptr)) return KVSWAP_ERR_NULL;
  if (layers->n_layers < 1 || layers->max_lookahead < 0) return KVSWAP_ERR_SHAPE;
  return KVSWAP_OK;
}

// The shape under which kvswap_sparse_decode sees a reuse store: n_slots groups followed by the
// rolling-buffer rows, dense [B, H_kv, (n_slots + 1) G, d].
static kvswap_shape reuse_store_shape(const kvswap_shape& s, int32_t n_slots) {
  kvswap_shape r = s;
  const int64_t R = int64_t(n_slots + 1) * s.group_size;
  r.n_ctx = n_slots * s.group_size + s.n_ctx % s.group_size;
  r.kv_stride_n = s.head_dim;
  r.kv_stride_h = R * s.head_dim;
  r.kv_stride_b = int64_t(s.n_kv_heads) * R * s.head_dim;
  return r;
}

// Per-device resources of kvswap_decode_step's two-stream schedule: a stream for the predictor and
// two events per layer.  Created on first use, kept for the life of the process.
namespace {
struct StepResources {
  cudaStream_t predictor = nullptr;
  cudaEvent_t fork = nullptr;
  std::vector<cudaEvent_t> selected;     // selected[l]: layer l's selection is written
  std::vector<cudaEvent_t> attended;     // attended[l]: layer l's attention output is written
};
constexpr int kMaxDevices = 64;
constexpr int kHostLead = 3;           // layers by which the host enqueues the predictor ahead of the attention
std::mutex g_step_mutex;
StepResources g_step[kMaxDevices];

cudaError_t grow(std::vector<cudaEvent_t>* evs, int n) {
  while (int(evs->size()) < n) {
    cudaEvent_t ev = nullptr;
    cudaError_t e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
    if (e != cudaSuccess) return e;
    evs->push_back(ev);
  }
  return cudaSuccess;
}

// Must be called with g_step_mutex held.
cudaError_t step_resources(int n_layers, StepResources** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  StepResources& r = g_step[dev];
  if (r.predictor == nullptr) {
    e = cudaStreamCreateWithFlags(&r.predictor, cudaStreamNonBlocking);
    if (e != cudaSuccess) { r.predictor = nullptr; return e; }
  }
  if (r.fork == nullptr) {
    e = cudaEventCreateWithFlags(&r.fork, cudaEventDisableTiming);
    if (e != cudaSuccess) { r.fork = nullptr; return e; }
  }
  if ((e = grow(&r.selected, n_layers)) != cudaSuccess) return e;
  if ((e = grow(&r.attended, n_layers)) != cudaSuccess) return e;
  *out = &r;
  return cudaSuccess;
}
}  // namespace

// One decode step over all layers; with `tiers` the attention is served from per-layer reuse buffers
// that the predictor stream keeps filled from the slow tier.
static int decode_step_impl(const kvswap_shape* shape, const kvswap_layers* layers, const kvswap_tiers* tiers,
                            const void* q, float* out, float* lse_opt, int32_t* group_idx, int32_t* n_selected,
                            void* ws, size_t ws_bytes, const kvswap_probe* probe_opt, void* cuda_stream) {
  Problem p;
  int st = resolve(shape, &p);
  if (st != KVSWAP_OK) return st;
  st = check_layers(layers, tiers == nullptr);
  if (st != KVSWAP_OK) return st;
  if (q == nullptr || out == nullptr || group_idx == nullptr || n_selected == nullptr) return KVSWAP_ERR_NULL;
  // Tiered: the predictor uses the head of the workspace, the attention over the reuse stores
  // (another shape, another plan) the part behind it, since the two run on different streams.
  kvswap_shape shape_attn = *shape;
  void* ws_attn = ws;
  size_t ws_attn_bytes = ws_bytes;
  if (tiers != nullptr) {
    Problem pr;
    if (tiers->max_groups < 1) return KVSWAP_ERR_SHAPE;
    st = resolve_reuse(shape, tiers->n_slots, tiers->max_groups, &pr);
    if (st != KVSWAP_OK) return st;
    if (tiers->K_slow == nullptr || tiers->V_slow == nullptr || tiers->K_reuse == nullptr ||
        tiers->V_reuse == nullptr || tiers->state == nullptr || tiers->slot_idx == nullptr ||
        tiers->miss_group == nullptr || tiers->miss_slot == nullptr || tiers->n_miss == nullptr)
      return KVSWAP_ERR_NULL;
    if (tiers->state_bytes < sizeof(int32_t) * reuse_state_words(pr, tiers->n_slots, tiers->max_groups))
      return KVSWAP_ERR_WORKSPACE;
    for (int l = 0; l < layers->n_layers; ++l) {
      if (tiers->K_slow[l] == nullptr || tiers->V_slow[l] == nullptr || tiers->K_reuse[l] == nullptr ||
          tiers->V_reuse[l] == nullptr || tiers->state[l] == nullptr)
        return KVSWAP_ERR_NULL;
      if (misaligned(tiers->K_slow[l]) || misaligned(tiers->V_slow[l]) || misaligned(tiers->K_reuse[l]) ||
          misaligned(tiers->V_reuse[l]) || misaligned(tiers->state[l]))
        return KVSWAP_ERR_ALIGN;
    }
    shape_attn = reuse_store_shape(*shape, tiers->n_slots);
    const size_t head_bytes = (kvswap_workspace_bytes(shape) + 255) & ~size_t(255);
    if (ws == nullptr) return KVSWAP_ERR_NULL;
    if (ws_bytes < head_bytes + kvswap_workspace_bytes(&shape_attn)) return KVSWAP_ERR_WORKSPACE;
    ws_attn = static_cast<char*>(ws) + head_bytes;
    ws_attn_bytes = ws_bytes - head_bytes;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const int L = layers->n_layers;
  const size_t q_bytes = size_t(p.B) * p.Hq * p.d * dtype_bytes(p.q_dtype);
  const size_t out_elems = size_t(p.B) * p.Hq * p.d;
  const size_t idx_elems = size_t(p.B) * p.S * p.M, nsel_elems = size_t(p.B) * p.S;
  Workspace w;
  st = check_score_select(shape, q, layers->proj[0], layers->meta[0], group_idx, n_selected, nullptr, ws, ws_bytes,
                          &p, &w);
  if (st != KVSWAP_OK) return st;
  for (int l = 0; l < L; ++l) {
    if (layers->proj[l] == nullptr || layers->meta[l] == nullptr) return KVSWAP_ERR_NULL;
    if (tiers == nullptr && (layers->K[l] == nullptr || layers->V[l] == nullptr)) return KVSWAP_ERR_NULL;
    if (tiers == nullptr && (misaligned(layers->K[l]) || misaligned(layers->V[l]))) return KVSWAP_ERR_ALIGN;
    if (misaligned(layers->proj[l]) || misaligned(layers->meta[l])) return KVSWAP_ERR_ALIGN;
  }

  if (tiers == nullptr) {
    if (misaligned(out) || (lse_opt && (reinterpret_cast<uintptr_t>(lse_opt) & 3u))) return KVSWAP_ERR_ALIGN;
    // Schedule (Sec. 4.3, online prediction, and Sec. 4.4): layer l + 1 is scored ahead of layer l's
    // attention -- as early as a model allows whose layer-(l+1) prediction is formed from the input of
    // layer l, which exists once layer l - 1 has been attended -- and its TopK follows that attention.
    // All on the caller's stream, every kernel a programmatic dependent launch, so each kernel's
    // set-up and first fetches overlap its predecessor's tail:
    //   score(0) select(0) | score(1) attention(0) select(1) | score(2) attention(1) select(2) | ...
    // The scorer streams the compact cache at HBM rate and the attention gathers at HBM rate; neither
    // leaves the other room on an SM, so they run one after the other, and what the order hides is
    // the latency-bound part: the TopK of layer l + 1 is not needed before attention l + 1, and the
    // gather of layer l starts fetching while the scorer of layer l + 1 drains.
    // Settled inputs: q is an input of the step; a selection is complete before the scorer that
    // precedes its attention passes its own dependency wait.
    Problem p_settled = p;
    p_settled.flags |= KVSWAP_INPUTS_SETTLED;
    kvswap_shape shape_settled = *shape;
    shape_settled.flags |= KVSWAP_INPUTS_SETTLED;
    auto ev = [&](void* e) { if (e != nullptr) cudaEventRecord(static_cast<cudaEvent_t>(e), stream); };
    auto probed = [&](int l) { return probe_opt != nullptr && probe_opt->layer == l; };
    // Where the kernel that merges layer l's partials and selects for layer l + 1 can also form the
    // summed low-rank queries of layer l + 2 (its combine CTAs idle until the gather has finished),
    // that layer's scorer finds them in the workspace and goes straight to its tiles.  The workspace
    // has two query buffers: the scorer of layer l + 1 may still be reading its own.
    const bool ahead = query_ahead_supported(p);
    const bool merges = select_merges_with_combine(p) && (p.d == 64 || p.d == 128) && w.splits <= kMaxSplits;
    int formed_for = -1;                            // the layer whose queries the last merged launch formed
    auto score = [&](int l) -> int {
      if (probed(l)) ev(probe_opt->ev_begin);
      const void* ql = static_cast<const char*>(q) + size_t(l) * q_bytes;
      return score_launch(p_settled, w, ql, layers->proj[l], layers->meta[l], nullptr, ws, stream,
                          formed_for == l ? (l & 1) : -1) == cudaSuccess
                 ? KVSWAP_OK : KVSWAP_ERR_CUDA;
    };
    auto select = [&](int l) -> int {
      const cudaError_t e = select_launch(p_settled, w, group_idx + size_t(l) * idx_elems,
                                          n_selected + size_t(l) * nsel_elems, nullptr, ws, stream);
      if (probed(l)) ev(probe_opt->ev_mid);
      return e == cudaSuccess ? KVSWAP_OK : KVSWAP_ERR_CUDA;
    };
    // The attention of layer l and the TopK of layer l + 1: the split-K gather, then one kernel that
    // merges its partials and selects (where the select has that form), else the two one after the other.
    float* partial = reinterpret_cast<float*>(static_cast<char*>(ws) + w.off_partial);
    auto attend_then_select = [&](int l) -> int {
      const void* ql = static_cast<const char*>(q) + size_t(l) * q_bytes;
      float* out_l = out + size_t(l) * out_elems;
      float* lse_l = lse_opt ? lse_opt + size_t(l) * p.B * p.Hq : nullptr;
      const int32_t* idx_l = group_idx + size_t(l) * idx_elems;
      const int32_t* nsel_l = n_selected + size_t(l) * nsel_elems;
      const bool next = l + 1 < L;
      // (the last layer's attention follows its own TopK directly: that selection is not settled)
      // Where the merged launch follows, the gather waits for the scorer before it as soon as its
      // first fills are out and lets that launch start only then: its TopK, whose inputs that scorer
      // wrote, need not wait for the gather.
      Problem p_early = p_settled;
      p_early.flags |= kFlagWaitEarly;
      const Problem& pa = !next ? p : merges ? p_early : p_settled;
      if (launch_sparse_decode(pa, w, ql, layers->K[l], layers->V[l], idx_l, nsel_l, partial, out_l, lse_l,
                               static_cast<uint32_t*>(ws), stream, /*combine=*/false) != cudaSuccess)
        return KVSWAP_ERR_CUDA;
      cudaError_t e = cudaSuccess;
      const bool form = ahead && l + 2 < L;
      const void* q_ahead = form ? static_cast<const char*>(q) + size_t(l + 2) * q_bytes : nullptr;
      Problem p_two_back = p_settled;
      p_two_back.flags |= kFlagInputsTwoBack;
      const bool merged = next && merges &&
                          select_with_combine_launch(p_two_back, w, group_idx + size_t(l + 1) * idx_elems,
                                                     n_selected + size_t(l + 1) * nsel_elems, ws, partial, out_l, lse_l,
                                                     w.splits, p.B * p.Hq, p.d, stream, &e, q_ahead,
                                                     form ? layers->proj[l + 2] : nullptr, (l + 2) & 1);
      if (merged && form && e == cudaSuccess) formed_for = l + 2;
      if (!merged) {
        e = launch_combine_only(p, w, partial, out_l, lse_l, stream);
      }
      if (probed(l)) ev(probe_opt->ev_end);
      if (e != cudaSuccess) return KVSWAP_ERR_CUDA;
      if (next && !merged) return select(l + 1);
      if (next && probed(l + 1)) ev(probe_opt->ev_mid);
      return KVSWAP_OK;
    };
    int status = score(0);
    if (status == KVSWAP_OK) status = select(0);
    for (int l = 0; l < L && status == KVSWAP_OK; ++l) {
      if (l + 1 < L) status = score(l + 1);
      if (status == KVSWAP_OK) status = attend_then_select(l);
    }
    return status;
  }

  // Tiered schedule: a layer's groups are predicted ahead of
  // its attention, concurrently with the layers before it.  The predictor therefore runs on a
  // stream of its own, ahead of the attention on the caller's stream by at most `look` layers
  // (any number when the caller sets no limit):
  //   predictor stream:  ... wait attended[l-1-look];  score/select(l);  record selected[l]  ...
  //   caller's stream:   ... wait selected[l];         attention(l);     record attended[l]  ...
  // With look = 1, predictor(l) overlaps attention(l-1) only: nothing runs further ahead than a
  // model whose layer-(l-1) input (from which the paper forms the approximate query) exists
  // once layer l-2 is done could run.  With look >= 2 the caller's stream waits for two layers'
  // selections at a time, so that every second attention follows the previous one without a
  // stream-level wait in between and, its inputs being settled, starts fetching while that one
  // is still finishing.  Everything on the predictor stream is ordered after the work already
  // in the caller's stream (fork event) and joins it again through the last selection event.
  const bool bounded = layers->max_lookahead > 0 && layers->max_lookahead < L;
  const int look = bounded ? layers->max_lookahead : L;
  const int join = look >= 2 ? 2 : 1;          // layers of attention per wait on the predictor
  // q is an input of the step (the fork event orders both streams after whatever produced it) and
  // each selection is awaited through its event before the attention that reads it is launched:
  // the inputs of both the predictor and the attention are settled.
  kvswap_shape shape_settled = shape_attn;
  shape_settled.flags |= KVSWAP_INPUTS_SETTLED;
  Problem p_settled = p;
  p_settled.flags |= KVSWAP_INPUTS_SETTLED;
  std::lock_guard<std::mutex> lock(g_step_mutex);
  StepResources* res = nullptr;
  if (step_resources(L, &res) != cudaSuccess) return KVSWAP_ERR_CUDA;
  cudaStream_t pred = res->predictor;
  if (cudaEventRecord(res->fork, stream) != cudaSuccess || cudaStreamWaitEvent(pred, res->fork, 0) != cudaSuccess)
    return KVSWAP_ERR_CUDA;

  auto enqueue_predictor = [&](int l) -> int {
    if (bounded && l > look && cudaStreamWaitEvent(pred, res->attended[l - 1 - look], 0) != cudaSuccess)
      return KVSWAP_ERR_CUDA;
    const bool probed = probe_opt != nullptr && probe_opt->layer == l;
    if (probed && probe_opt->ev_begin) cudaEventRecord(static_cast<cudaEvent_t>(probe_opt->ev_begin), pred);
    const void* ql = static_cast<const char*>(q) + size_t(l) * q_bytes;
    if (score_select_launch(p_settled, w, ql, layers->proj[l], layers->meta[l], group_idx + size_t(l) * idx_elems,
                            n_selected + size_t(l) * nsel_elems, nullptr, ws, pred) != cudaSuccess)
      return KVSWAP_ERR_CUDA;
    if (tiers != nullptr) {
      // Hits keep their slots, misses are fetched from the slow tier -- still on the predictor
      // stream, so the fetch for this layer overlaps the attention of the layers before it.
      int32_t* slot_l = tiers->slot_idx + size_t(l) * idx_elems;
      int32_t* mg_l = tiers->miss_group + size_t(l) * idx_elems;
      int32_t* ms_l = tiers->miss_slot + size_t(l) * idx_elems;
      int32_t* nm_l = tiers->n_miss + size_t(l) * nsel_elems;
      if (launch_reuse_lookup(p, tiers->n_slots, tiers->max_groups, group_idx + size_t(l) * idx_elems,
                              n_selected + size_t(l) * nsel_elems, static_cast<int32_t*>(tiers->state[l]), slot_l, mg_l,
                              ms_l, nm_l, pred) != cudaSuccess ||
          launch_reuse_fill(p, tiers->n_slots, tiers->K_slow[l], tiers->V_slow[l], tiers->K_reuse[l],
                            tiers->V_reuse[l], mg_l, ms_l, nm_l, pred) != cudaSuccess)
        return KVSWAP_ERR_CUDA;
    }
    if (probed && probe_opt->ev_mid) cudaEventRecord(static_cast<cudaEvent_t>(probe_opt->ev_mid), pred);
    if (cudaEventRecord(res->selected[l], pred) != cudaSuccess) return KVSWAP_ERR_CUDA;
    return KVSWAP_OK;
  };
  auto enqueue_attention = [&](int l) -> int {
    if (l % join == 0 &&
        cudaStreamWaitEvent(stream, res->selected[std::min(L - 1, l + join - 1)], 0) != cudaSuccess)
      return KVSWAP_ERR_CUDA;
    const bool probed = probe_opt != nullptr && probe_opt->layer == l;
    const void* ql = static_cast<const char*>(q) + size_t(l) * q_bytes;
    const void* Kl = tiers ? tiers->K_reuse[l] : layers->K[l];
    const void* Vl = tiers ? tiers->V_reuse[l] : layers->V[l];
    const int32_t* list_l = (tiers ? tiers->slot_idx : group_idx) + size_t(l) * idx_elems;
    const int r = kvswap_sparse_decode(&shape_settled, ql, Kl, Vl, list_l, n_selected + size_t(l) * nsel_elems,
                                       out + size_t(l) * out_elems,
                                       lse_opt ? lse_opt + size_t(l) * p.B * p.Hq : nullptr, ws_attn, ws_attn_bytes,
                                       cuda_stream);
    if (probed && probe_opt->ev_end) cudaEventRecord(static_cast<cudaEvent_t>(probe_opt->ev_end), stream);
    if (bounded && r == KVSWAP_OK && cudaEventRecord(res->attended[l], stream) != cudaSuccess)
      return KVSWAP_ERR_CUDA;
    return r;
  };

  // Host order: a predictor is handed to its stream before the wait on its selection is enqueued
  // (join - 1 layers ahead at least), up to kHostLead layers ahead of the attention that consumes
  // it, and never before the attention whose event it waits on (look - join + 1 at most).
  const int lead = std::max(join - 1, std::min(look - join + 1, kHostLead));
  int status = KVSWAP_OK;
  int next_pred = 0;
  for (int l = 0; l < L && status == KVSWAP_OK; ++l) {
    while (status == KVSWAP_OK && next_pred < L && next_pred <= l - l % join + lead)
      status = enqueue_predictor(next_pred++);
    if (status == KVSWAP_OK) status = enqueue_attention(l);
  }
  if (status != KVSWAP_OK) {
    // a launch failed: join whatever the predictor stream was given after its last awaited event
    if (cudaEventRecord(res->fork, pred) != cudaSuccess || cudaStreamWaitEvent(stream, res->fork, 0) != cudaSuccess)
      return KVSWAP_ERR_CUDA;
  }
  return status;
}

int kvswap_decode_step(const kvswap_shape* shape, const kvswap_layers* layers, const void* q, float* out,
                       float* lse_opt, int32_t* group_idx, int32_t* n_selected, void* ws, size_t ws_bytes,
                       const kvswap_probe* probe_opt, void* cuda_stream) {
  return decode_step_impl(shape, layers, nullptr, q, out, lse_opt, group_idx, n_selected, ws, ws_bytes, probe_opt,
                          cuda_stream);
}

size_t kvswap_tiered_workspace_bytes(const kvswap_shape* shape, int32_t n_slots) {
  Problem p;
  if (resolve_reuse(shape, n_slots, 0, &p) != KVSWAP_OK) return 0;
  const kvswap_shape r = reuse_store_shape(*shape, n_slots);
  const size_t tail = kvswap_workspace_bytes(&r);
  if (tail == 0) return 0;
  return ((kvswap_workspace_bytes(shape) + 255) & ~size_t(255)) + tail;
}

int kvswap_decode_step_tiered(const kvswap_shape* shape, const kvswap_layers* layers, const kvswap_tiers* tiers,
                              const void* q, float* out, float* lse_opt, int32_t* group_idx, int32_t* n_selected,
                              void* ws, size_t ws_bytes, void* cuda_stream) {
  if (tiers == nullptr) return KVSWAP_ERR_NULL;
  return decode_step_impl(shape, layers, tiers, q, out, lse_opt, group_idx, n_selected, ws, ws_bytes, nullptr,
                          cuda_stream);
}

int kvswap_append_step_tiered(const kvswap_shape* shape, const kvswap_layers* layers, const kvswap_tiers* tiers,
                              const void* k_new, const void* v_new, int32_t* flushed_opt, void* cuda_stream) {
  if (flushed_opt != nullptr) *flushed_opt = 0;
  Problem p;                                   // the grown context: N + 1 tokens, the slow tier's strides
  int st = resolve_grown(shape, &p);
  if (st != KVSWAP_OK) return st;
  st = check_layers(layers, false);
  if (st != KVSWAP_OK) return st;
  if (tiers == nullptr || tiers->K_slow == nullptr || tiers->V_slow == nullptr || tiers->K_reuse == nullptr ||
      tiers->V_reuse == nullptr || k_new == nullptr || v_new == nullptr)
    return KVSWAP_ERR_NULL;
  if (tiers->n_slots < 1) return KVSWAP_ERR_SHAPE;
  // the grown context must still fit the slot tables the next tiered step will use
  if (tiers->max_groups > 0 && p.NG > tiers->max_groups) return KVSWAP_ERR_SHAPE;
  if (misaligned(k_new) || misaligned(v_new)) return KVSWAP_ERR_ALIGN;
  const int L = layers->n_layers;
  for (int l = 0; l < L; ++l) {
    if (tiers->K_slow[l] == nullptr || tiers->V_slow[l] == nullptr || tiers->K_reuse[l] == nullptr ||
        tiers->V_reuse[l] == nullptr || layers->meta[l] == nullptr || layers->proj[l] == nullptr)
      return KVSWAP_ERR_NULL;
    if (misaligned(tiers->K_slow[l]) || misaligned(tiers->V_slow[l]) || misaligned(tiers->K_reuse[l]) ||
        misaligned(tiers->V_reuse[l]) || misaligned(layers->meta[l]) || misaligned(layers->proj[l]))
      return KVSWAP_ERR_ALIGN;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  // The new token joins the rolling-buffer rows of every layer's reuse store.
  const int64_t fast_rows = int64_t(tiers->n_slots + 1) * p.G;
  const int n = p.N - 1;                       // its position in the context
  Problem fast = p;
  fast.kv_sn = p.d;
  fast.kv_sh = fast_rows * p.d;
  fast.kv_sb = int64_t(p.Hkv) * fast.kv_sh;
  if (launch_append_rows(fast, k_new, v_new, tiers->K_reuse, tiers->V_reuse, L, tiers->n_slots * p.G + n % p.G,
                         stream) != cudaSuccess)
    return KVSWAP_ERR_CUDA;
  if (p.N % p.G == 0) {
    // The group is complete: its rows go to the slow tier, and its compact-cache rows are built
    // from there (the projection reads the rows it was just handed; same stream).
    if (launch_flush_rows(p, tiers->K_reuse, tiers->V_reuse, const_cast<void* const*>(tiers->K_slow),
                          const_cast<void* const*>(tiers->V_slow), L, fast_rows, int64_t(tiers->n_slots) * p.G,
                          p.N - p.G, stream) != cudaSuccess ||
        launch_project_keys_layers(p, tiers->K_slow, layers->proj, const_cast<void* const*>(layers->meta), L,
                                   p.N - p.G, p.N, stream) != cudaSuccess)
      return KVSWAP_ERR_CUDA;
    if (flushed_opt != nullptr) *flushed_opt = 1;
  }
  return KVSWAP_OK;
}

int kvswap_decode_step_host(const kvswap_shape* shape, const kvswap_layers* layers, const void* q_host,
                            float* out_host, void* q_dev, float* out_dev, int32_t* group_idx,
                            int32_t* n_selected, void* ws, size_t ws_bytes, void* cuda_stream) {
  Problem p;
  int st = resolve(shape, &p);
  if (st != KVSWAP_OK) return st;
  st = check_layers(layers);
  if (st != KVSWAP_OK) return st;
  if (q_host == nullptr || out_host == nullptr || q_dev == nullptr || out_dev == nullptr) return KVSWAP_ERR_NULL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const size_t L = size_t(layers->n_layers);
  const size_t q_bytes = L * p.B * p.Hq * p.d * dtype_bytes(p.q_dtype);
  const size_t out_bytes = L * p.B * p.Hq * p.d * sizeof(float);
  if (cudaMemcpyAsync(q_dev, q_host, q_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) return KVSWAP_ERR_CUDA;
  st = kvswap_decode_step(shape, layers, q_dev, out_dev, nullptr, group_idx, n_selected, ws, ws_bytes, nullptr,
                          cuda_stream);
  if (st != KVSWAP_OK) return st;
  if (cudaMemcpyAsync(out_host, out_dev, out_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
    return KVSWAP_ERR_CUDA;
  return KVSWAP_OK;
}

}  // extern "C"
