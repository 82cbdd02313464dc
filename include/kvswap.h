/*
 * kvswap.h -- C ABI of the KVSwap decode hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, on one GPU, the per-decode-step KV-entry predictor of KVSwap and
 * the exact sparse decode attention that consumes its output:
 *
 *   kvswap_project_keys   K_lr = Flatten(K) A                         (Sec. 4.2)
 *   kvswap_score_select   low-rank scores (Eq. 1) -> sum over heads -> ReduceMax over groups of
 *                         G tokens -> TopK M groups                   (Sec. 4.3)
 *   kvswap_sparse_decode  softmax attention over the selected groups plus the rolling-buffer
 *                         tail                                        (Sec. 4.4, 4.4.1, 4.4.4)
 *
 * and around them
 *
 *   kvswap_decode_step / _host        one decode step over all layers of a model, each layer predicted
 *                                     one layer ahead of its attention (Sec. 4.3, 4.4)
 *   kvswap_append_kv / _append_step   a generated token joins the rolling buffer; a completed
 *                                     group is flushed into the compact cache      (Sec. 4.4.1)
 *   kvswap_reuse_* , kvswap_decode_step_tiered, kvswap_append_step_tiered
 *                                     reuse buffer (slots, slot table, FIFO) in front of a slower
 *                                     tier that holds the whole cache              (Sec. 4.4.2)
 *
 * The paper keeps the full KV cache on disk; by default here it is an HBM-resident tensor and
 * "loading a group" is a gather of G consecutive rows; the tiered calls put it in any memory the
 * GPU can read (pinned host memory in the tests) behind reuse buffers in HBM.
 *
 * Notation: B sequences, N cached tokens, H_q query heads, H_kv KV heads, rho = H_q / H_kv,
 * g(h) = floor(h / rho), d head dim, r metadata rank, A_g = proj[g] in R^{d x r} the row block of
 * the adapter A for KV head g, G group size, M groups to select, NG = floor(N / G).
 * H_m ("meta_heads") is 1 for the joint-head adapter the paper adopts (design (b) of Sec. 4.2)
 * or H_kv for one adapter per KV head (design (a)).  S is the number of selections per
 * sequence: H_kv for KVSWAP_SCOPE_KV_HEAD (scores summed over the rho query heads of one KV
 * head), 1 for KVSWAP_SCOPE_ALL_HEADS (scores summed over all query heads, the paper's wording).
 *
 * General conventions
 *  - Every pointer is a DEVICE pointer owned by the caller unless its comment says "host".
 *    The library never allocates, frees or keeps device memory (kvswap_decode_step_tiered creates
 *    one stream and a set of events per device on its first call), and never synchronises: work is
 *    enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL = default stream) and the
 *    returned status covers host-side validation and launch errors only.
 *  - Tensors are row-major with a dense last dimension; K, V and the metadata take explicit
 *    element strides for the leading dimensions.
 *  - Device pointers must be 16-byte aligned, and d*sizeof(kv) and r*sizeof(meta) must be
 *    multiples of 16 bytes (KVSWAP_ERR_ALIGN otherwise).
 *  - Inputs must be finite.  NaN/Inf never fault but give unspecified selections/outputs.
 *  - Errors are returned, never raised: no call aborts or traps.
 *  - `ws` is caller-provided scratch of at least kvswap_workspace_bytes(shape) bytes, cleared once
 *    with kvswap_workspace_init before its first use.  The predictor keeps a region at its head
 *    (sized by B, H_kv, the scope and the metadata type alone) zero from call to call; the rest is
 *    undefined between calls.  One workspace may serve shapes that differ in n_ctx, top_k and
 *    flags; clear it again before using it for another batch size, head count or scope, and after
 *    a call that returned KVSWAP_ERR_CUDA.  Calls that run concurrently on different streams need
 *    different workspaces.
 */
#ifndef KVSWAP_H_
#define KVSWAP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  KVSWAP_OK = 0,
  KVSWAP_ERR_NULL = 1,        /* a required pointer is NULL                                  */
  KVSWAP_ERR_SHAPE = 2,       /* a size/stride/enum combination is invalid                   */
  KVSWAP_ERR_DTYPE = 3,       /* unknown dtype tag or unsupported dtype combination          */
  KVSWAP_ERR_ALIGN = 4,       /* pointer or row size not 16-byte aligned                     */
  KVSWAP_ERR_WORKSPACE = 5,   /* ws_bytes smaller than kvswap_workspace_bytes()              */
  KVSWAP_ERR_UNSUPPORTED = 6, /* valid request outside the implemented range                 */
  KVSWAP_ERR_CUDA = 7,        /* a CUDA runtime call or kernel launch failed                 */
  KVSWAP_ERR_INDEX = 8,       /* device status: a group index or count out of range was seen (KVSWAP_CHECK_INDICES) */
  KVSWAP_ERR_STATIC_SCRATCH = 9, /* problem needs more than KVSWAP_STATIC_SCRATCH_BYTES of scratch */
  KVSWAP_ERR_TIMEOUT = 10     /* a kernel gave up a bounded wait; its outputs are invalid     */
} kvswap_status;

/* KVSWAP_E4M3 is a metadata type only: the 8-bit floating-point format E4M3 (1 sign, 4 exponent bits
 * with bias 7, 3 mantissa bits; no infinities; S.1111.111 = NaN; largest finite value 448). */
typedef enum { KVSWAP_F32 = 0, KVSWAP_BF16 = 1, KVSWAP_F16 = 2, KVSWAP_E4M3 = 3 } kvswap_dtype;
typedef enum { KVSWAP_SCOPE_KV_HEAD = 0, KVSWAP_SCOPE_ALL_HEADS = 1 } kvswap_scope;

/*
 * kvswap_shape.flags (bit set; unknown bits are KVSWAP_ERR_SHAPE).
 *   KVSWAP_INPUTS_SETTLED  a promise by the caller of kvswap_score_select or
 *       kvswap_sparse_decode: the call's inputs (q; for kvswap_sparse_decode also group_idx and
 *       n_selected; K, V, proj and the metadata always) are not outputs of work that may still
 *       be running when the call's kernels start, i.e. nothing enqueued earlier in `cuda_stream`
 *       writes them, or a full dependency (an event wait, a copy, a host synchronisation) lies
 *       in between.  The first kernel of the call then starts while the previous kernel of the
 *       stream is still finishing (programmatic dependent launch) and only waits for it before
 *       writing its own results.  Without the flag it waits first.  Results are the same.
 *   KVSWAP_SCORE_SOFTMAX   a variant of the predictor (kvswap_score_select, and the steps built on
 *       it): each query head's low-rank scores pass through a softmax over the tokens of the
 *       context's complete groups, scaled by 1/sqrt(d), BEFORE the sum over heads -- the scores
 *       of Sec. 4.3 read as attention weights rather than logits (for one head the selection is
 *       the same; across heads a sharply peaked head then outweighs a flat one).  Group scores
 *       lie in [0, heads per scope].  Two passes over the metadata (tensor cores for joint
 *       fp16 metadata with r = 32 and H_q <= 32, general fp32 kernels otherwise).
 *       KVSWAP_ERR_UNSUPPORTED if H_q * (r + 2) floats exceed 160 KB.
 *   KVSWAP_META_EXP(e)     bits 8..15: a power of two for 8-bit metadata (meta_dtype = KVSWAP_E4M3),
 *       -64 <= e <= 63, 0 for every other metadata type.  The paper leaves the precision of the
 *       compact cache open ("can be flexibly traded", Sec. 4.1 / 4.2); with KVSWAP_E4M3 a row of
 *       K_lr takes r bytes: kvswap_project_keys stores round(K_lr * 2^-e) -- one round-to-nearest-
 *       even, magnitudes beyond 448 saturate -- and kvswap_score_select scores the stored values
 *       times 2^e.  The ranking does not depend on e; choose it so that |K_lr| * 2^-e stays below
 *       448 and the bulk of the values above 2^-6 (e = 0 suits keys of unit scale).  Supported for
 *       r = 32, G a power of two <= 32 and dense metadata rows (else KVSWAP_ERR_UNSUPPORTED); not with
 *       KVSWAP_SCORE_SOFTMAX.
 *   KVSWAP_CHECK_INDICES   a debugging aid for callers that build their own index lists: besides
 *       skipping them, kvswap_sparse_decode (and the steps built on it) records in the device
 *       status word of `ws` that it met a group index outside [0, NG) other than the padding
 *       value -1, or an n_selected outside [0, M]; kvswap_read_device_status then returns
 *       KVSWAP_ERR_INDEX.  Results are those without the flag.
 */
enum { KVSWAP_INPUTS_SETTLED = 1, KVSWAP_SCORE_SOFTMAX = 2, KVSWAP_CHECK_INDICES = 4 };
#define KVSWAP_META_EXP(e) ((int32_t)(((uint32_t)(e) & 0xffu) << 8))

/*
 * Problem description shared by all calls.
 *   kv_*   strides (in elements) of K and V, both laid out [B, H_kv, N, d];
 *   meta_* strides (in elements) of the metadata, laid out [B, H_m, N, r].
 * A stride of 0 means "dense": the natural stride of the contiguous tensor.
 * Supported ranges: d in {64, 128}; r a multiple of 4 with 4 <= r <= 256; G >= 1; M >= 1;
 * rho >= 1; G <= 1024; M * G <= 2^30; kv_dtype in {F32, BF16, F16}; q_dtype = kv_dtype or F32; meta_dtype in
 * {F32, F16, E4M3}.
 */
typedef struct {
  int32_t batch, n_ctx, n_q_heads, n_kv_heads, head_dim; /* B, N, H_q, H_kv, d            */
  int32_t rank, meta_heads, group_size, top_k;           /* r, H_m in {1, H_kv}, G, M     */
  int32_t kv_dtype, meta_dtype, q_dtype, scope;          /* enums above                   */
  int32_t flags;                                         /* bit set of the flags above    */
  int64_t kv_stride_b, kv_stride_h, kv_stride_n;
  int64_t meta_stride_b, meta_stride_h, meta_stride_n;
} kvswap_shape;

/* Bytes of scratch any of the calls below may need for `shape`; 0 if the shape is invalid. */
size_t kvswap_workspace_bytes(const kvswap_shape* shape);

/* Validates `shape` exactly as the compute calls do (host only, touches no GPU). */
int kvswap_validate_shape(const kvswap_shape* shape);

/*
 * Workspace set-up and the device status word.  The kernels stage K/V rows through shared memory
 * with asynchronous copies and wait for them with a bounded number of attempts; a wait that runs
 * out (which no valid input can cause) is recorded in the first word of the workspace instead of
 * hanging the GPU.
 *   kvswap_workspace_init     clears the workspace (asynchronously, on `cuda_stream`): the status
 *                             word and the counters kvswap_score_select expects to find zero.
 *                             Required once after allocating a workspace (see the conventions
 *                             above); a workspace that was never cleared selects wrong groups.
 *   kvswap_read_device_status waits for `cuda_stream` to drain (the only call of the library that
 *                             synchronises), then returns KVSWAP_OK, or KVSWAP_ERR_TIMEOUT if a
 *                             kernel using `ws` has given up a wait since the word was cleared,
 *                             or KVSWAP_ERR_INDEX if a call with KVSWAP_CHECK_INDICES has met an
 *                             index out of range since then.
 */
int kvswap_workspace_init(void* ws, size_t ws_bytes, void* cuda_stream);
int kvswap_read_device_status(const void* ws, void* cuda_stream);

/*
 * Metadata build, K_lr = Flatten(K) A (Sec. 4.2), for tokens n_begin <= n < n_end (prefill: the
 * whole context; decode: the rows of a group the rolling buffer has just completed, Sec. 4.4.1).
 *   joint    (H_m = 1):    meta[b, 0, n, :] = sum_g K[b, g, n, :] . proj[g]   (Flatten is head-major)
 *   per-head (H_m = H_kv): meta[b, g, n, :] =       K[b, g, n, :] . proj[g]
 * K: [B, H_kv, N, d] kv_dtype.  proj: [H_kv, d, r] fp32, dense.  meta_out: [B, H_m, N, r]
 * meta_dtype; fp32 accumulation, one round-to-nearest-even into meta_dtype.  Rows outside
 * [n_begin, n_end) are not touched.  Requires 0 <= n_begin <= n_end <= N (empty range: no-op).
 * `ws` may be NULL here.  With a workspace of at least kvswap_workspace_bytes(shape), bf16 K with
 * d in {64, 128} and r in {16, 32, 64} runs on the tcgen05 tensor cores (it keeps a pre-split copy of
 * the adapter in the workspace); without one, and for every other shape, a warp-level kernel computes
 * the same result.
 */
int kvswap_project_keys(const kvswap_shape* shape, const void* K, const float* proj,
                        void* meta_out, int32_t n_begin, int32_t n_end,
                        void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * New KV entries (Sec. 4.4.1, rolling buffer).  shape->n_ctx is the context length N BEFORE the
 * call.  k_new, v_new [B, H_kv, d] kv_dtype (dense, device) are written to token row N of K and
 * V; the rows past the last complete group are the rolling buffer, which kvswap_sparse_decode
 * always attends, so the new token takes part in the next attention at once.  When the N + 1
 * tokens end a group ((N + 1) % G == 0) the group is "flushed": its G rows of the compact cache,
 * meta[.., N+1-G .. N, ..] = K_lr of those tokens (Sec. 4.2), are built, and from then on
 * kvswap_score_select (called with n_ctx = N + 1) ranks the group.  *flushed_opt (host, may be
 * NULL) is set to 1 when that happened, else 0; it depends on N and G only.
 * The store needs room for the row: kv_stride_h and meta_stride_h must be given (not 0) and
 * cover at least N + 1 rows, else KVSWAP_ERR_SHAPE; nothing is reallocated or moved.  After
 * the call the caller describes the context with n_ctx = N + 1 and the same strides.
 * Asynchronous on `cuda_stream`; needs no workspace.
 */
int kvswap_append_kv(const kvswap_shape* shape, const void* k_new, const void* v_new, void* K, void* V,
                     const float* proj, void* meta, int32_t* flushed_opt, void* cuda_stream);

/*
 * Grouped critical-KV prediction (Eq. 1 and "Scoring and selection", Sec. 4.3).
 * For every sequence b and selection scope s:
 *   T[b,s,n] = sum_{h in scope s} (q[b,h,:] . proj[g(h)]) . meta[b, m(g(h)), n, :]   (raw logits:
 *              no softmax, no 1/sqrt(d)),  m(g) = 0 for joint metadata, g for per-head metadata;
 *   R[b,s,j] = max_{0<=t<G} T[b,s,jG+t]   for j < NG  (the N mod G newest tokens form no group);
 *   the M' = min(M, NG) groups with the largest R are selected; of equal scores the lower index
 *   wins; indices are written in ascending order.
 * q: [B, H_q, d] q_dtype, dense (may be an approximate query, Sec. 4.3 "Online prediction").
 * group_idx: [B, S, M] int32; entries [M', M) of each row are set to -1.
 * n_selected: [B, S] int32, receives M'.
 * group_scores_opt: NULL or [B, S, NG] fp32, receives R.
 * Scores are accumulated in fp32.
 */
int kvswap_score_select(const kvswap_shape* shape, const void* q, const float* proj,
                        const void* meta, int32_t* group_idx, int32_t* n_selected,
                        float* group_scores_opt, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Exact decode attention over the selected groups and the rolling-buffer tail (Sec. 4.4,
 * 4.4.1, 4.4.4).  For every (b, h), with g = g(h) and row s = g (KV_HEAD) or 0 (ALL_HEADS) of
 * the index list:
 *   tokens  = U_{i < n_selected[b,s]} [ j_i G, j_i G + G )  U  [ NG*G, N ),  j_i = group_idx[b,s,i]
 *   logit_n = q[b,h,:] . K[b,g,n,:] / sqrt(d)
 *   out[b,h,:] = sum_n softmax(logit)_n V[b,g,n,:],   lse[b,h] = log sum_n exp(logit_n)
 * computed with an fp32 online softmax in split-K partials merged by a combine pass.
 * group_idx: [B, S, M] int32, any duplicate-free list of groups in [0, NG) (ascending order is
 * not required); n_selected: [B, S] with 0 <= n_selected <= M.  Indices outside [0, NG) are
 * skipped, never dereferenced.  If a head attends no token at all (n_selected = 0 and N a
 * multiple of G) its output row is 0 and its lse is -inf.
 * out: [B, H_q, d] fp32.  lse_opt: NULL or [B, H_q] fp32.
 */
int kvswap_sparse_decode(const kvswap_shape* shape, const void* q, const void* K, const void* V,
                         const int32_t* group_idx, const int32_t* n_selected,
                         float* out, float* lse_opt, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * kvswap_sparse_decode without a workspace argument.  (Library convenience: the paper has no
 * counterpart; the computation is exactly that of kvswap_sparse_decode.)
 *
 * For callers that must not allocate device memory where they call the library and therefore
 * have no scratch buffer to pass: e.g. a serving process whose memory manager took the whole GPU
 * at start-up, or code running inside a host framework's enqueue callback where cudaMalloc is
 * off limits because it synchronises the device and may fail late.  The split-K partials live
 * in a buffer of KVSWAP_STATIC_SCRATCH_BYTES that is built into the library; every GPU that
 * loads the library holds that much memory until the process exits.
 *
 *  - Inputs and outputs are the caller's, with the same meaning, layout and checks as in
 *    kvswap_sparse_decode.  The call itself allocates and frees nothing.
 *  - Problems whose partials, 256 + 4 * B * H_q * splits * (d + 2) bytes (splits as chosen by
 *    the library for the shape, at most 256), exceed the buffer are refused with
 *    KVSWAP_ERR_STATIC_SCRATCH before anything is launched.  All five benchmark configurations
 *    fit (the largest needs about 2 MiB).
 *  - The first call on each device looks up the buffer's device address (with that device
 *    current) and caches it for the life of the process; make that first call outside of any
 *    stream capture, and do not call this entry point on a device after the process has reset
 *    it (cudaDeviceReset): the cached address would be stale.
 *  - The size check is the first check after the shape's: KVSWAP_ERR_STATIC_SCRATCH is returned
 *    whatever the pointers are.
 *  - All calls on a device share the one buffer, and it keeps whatever the previous call left
 *    there.  Nothing in it needs clearing (each call overwrites every slot it later reads), but
 *    two calls that overlap on the GPU -- different streams, or threads -- race on it and give
 *    wrong results: serialise them, or use kvswap_sparse_decode with separate workspaces.
 */
#define KVSWAP_STATIC_SCRATCH_BYTES (8u << 20)
int kvswap_sparse_decode_static(const kvswap_shape* shape, const void* q, const void* K,
                                const void* V, const int32_t* group_idx,
                                const int32_t* n_selected, float* out, float* lse_opt,
                                void* cuda_stream);

/*
 * Per-layer tensors of a model with L layers that all share one kvswap_shape.  Each member is a
 * HOST array of L DEVICE pointers: K[l], V[l] are [B, H_kv, N, d]; meta[l] is [B, H_m, N, r];
 * proj[l] is [H_kv, d, r] fp32.  max_lookahead bounds how many layers the predictor stream of
 * kvswap_decode_step_tiered may run ahead of its attention: 1 = layer l is predicted while layer
 * l-1 is attended (what a model allows, whose layer-l prediction needs the input of layer l-1);
 * 0 = no limit.  kvswap_decode_step always predicts exactly one layer ahead and ignores the value.
 * Negative values are KVSWAP_ERR_SHAPE.
 */
typedef struct {
  int32_t n_layers;
  int32_t max_lookahead;
  const void* const* K;
  const void* const* V;
  const void* const* meta;
  const float* const* proj;
} kvswap_layers;

/*
 * Optional timing probe of kvswap_decode_step: for layer `layer`, CUDA events (cudaEvent_t passed
 * as void*, created with timing enabled by the caller) are recorded on the stream before
 * score_select (ev_begin), between score_select and sparse_decode (ev_mid) and after
 * sparse_decode (ev_end).  NULL events are skipped.
 */
typedef struct {
  int32_t layer;
  void* ev_begin;
  void* ev_mid;
  void* ev_end;
} kvswap_probe;

/*
 * Reuse buffer (Sec. 4.4.2): n_slots slots per (sequence, selection scope), each holding the K/V
 * rows of one group, in front of a slower tier that holds the whole cache (any memory the GPU can
 * read: device memory, pinned host memory).  A slot table records the group in each slot; a
 * selected group found there is a hit and is attended from its slot; any other is a miss: it
 * takes the next slot in FIFO order (slots are filled in the order 0, 1, .., n_slots-1, 0, ..),
 * passing over slots that serve the current step, and is fetched from the slow tier.
 *
 *   state       caller-owned device memory, kvswap_reuse_state_bytes(shape, n_slots, max_groups)
 *               bytes, one per layer; kvswap_reuse_init empties every slot.  max_groups bounds
 *               the group ids that will ever be looked up (floor(N_max / G)).
 *   reuse store K_reuse, V_reuse [B, H_kv, (n_slots + 1) * G, d] kv_dtype, dense: slot c is rows
 *               [c G, c G + G); the last G rows are room for the rolling buffer (the caller keeps
 *               the N mod G newest tokens there).  With the per-KV-head scope head g's rows follow
 *               head g's slot table; with the all-heads scope one table serves every head.
 *
 * kvswap_reuse_lookup takes a step's selection (group_idx [B, S, M], n_selected [B, S], as written
 * by kvswap_score_select; a group listed twice is loaded once and both entries get its slot; entries
 * outside [0, floor(n_ctx / G)) are "no group") and writes slot_idx [B, S, M] (the slot serving each entry, -1 for "no group"), the
 * misses in list order as miss_group / miss_slot [B, S, M] (-1 beyond the count) and n_miss
 * [B, S]; the slot table is updated.  kvswap_reuse_fill copies each missed group's G rows of K and
 * V (of the scope's heads) from the slow tier, described by `shape`'s kv strides, into its slot.
 * The step's attention is then kvswap_sparse_decode over the reuse store: K = K_reuse, V = V_reuse,
 * group_idx = slot_idx, a shape with n_ctx = n_slots * G + (N mod G) and the reuse store's strides.
 * Hits / (hits + misses) is the paper's reuse rate.
 *
 * Limits: n_slots >= M (else KVSWAP_ERR_SHAPE: a step's groups must fit); floor(n_ctx / G) <=
 * max_groups in every call that takes max_groups, the tiered steps included (else
 * KVSWAP_ERR_SHAPE: the tables have no entry for a group id beyond max_groups, so a context that
 * has grown past max_groups * G + G - 1 tokens needs a larger state); n_slots <= 32768 and
 * M <= 8192 (else KVSWAP_ERR_UNSUPPORTED).  KVSWAP_ERR_WORKSPACE if state_bytes is too small.
 * All calls are asynchronous on `cuda_stream`.
 */
size_t kvswap_reuse_state_bytes(const kvswap_shape* shape, int32_t n_slots, int32_t max_groups);
int kvswap_reuse_init(const kvswap_shape* shape, int32_t n_slots, int32_t max_groups, void* state,
                      size_t state_bytes, void* cuda_stream);
int kvswap_reuse_lookup(const kvswap_shape* shape, int32_t n_slots, int32_t max_groups,
                        const int32_t* group_idx, const int32_t* n_selected, void* state,
                        size_t state_bytes, int32_t* slot_idx, int32_t* miss_group, int32_t* miss_slot,
                        int32_t* n_miss, void* cuda_stream);
int kvswap_reuse_fill(const kvswap_shape* shape, int32_t n_slots, const void* K_slow, const void* V_slow,
                      void* K_reuse, void* V_reuse, const int32_t* miss_group, const int32_t* miss_slot,
                      const int32_t* n_miss, void* cuda_stream);

/*
 * kvswap_append_kv for every layer of a model at once: k_new, v_new [L, B, H_kv, d] kv_dtype
 * (dense, device) join row N = shape->n_ctx of layers->K[l], layers->V[l] (one launch per 32
 * layers); when that completes a group, each layer's compact-cache rows of the group are built.
 * The tables are const-qualified for the read-only calls; this call WRITES the K, V and meta
 * buffers they point to.  max_lookahead is ignored.  Same errors and capacity rule as
 * kvswap_append_kv.
 */
int kvswap_append_step(const kvswap_shape* shape, const kvswap_layers* layers, const void* k_new,
                       const void* v_new, int32_t* flushed_opt, void* cuda_stream);

/*
 * One decode step of the predictor + sparse attention (Sec. 4.4, decoding): for l = 0..L-1, in
 * order on `cuda_stream`, kvswap_score_select then kvswap_sparse_decode on layer l, with
 *   q          [L, B, H_q, d] q_dtype  (the same query scores and attends; device)
 *   out        [L, B, H_q, d] fp32     (device)
 *   lse_opt    NULL or [L, B, H_q] fp32
 *   group_idx  [L, B, S, M] int32, n_selected [L, B, S] int32: the selections of this step, kept
 *              per layer so that the caller can compare consecutive steps (Sec. 4.4.2).
 * `ws` is shared by all layers (size: kvswap_workspace_bytes).  probe_opt may be NULL.
 * The call orders prediction and attention as the paper's runtime does (Sec. 4.3 "Online
 * prediction", Sec. 4.4): layer l + 1 is scored before layer l is attended and its TopK follows
 * that attention, i.e. the predictor is exactly one layer ahead -- what a model allows whose
 * layer-(l+1) prediction is formed from the input of layer l.  Everything is enqueued on
 * `cuda_stream` as programmatic dependent launches (a kernel's set-up and first fetches overlap
 * the tail of the kernel before it); the call keeps no state, creates nothing and takes no lock.
 * Results are identical to calling kvswap_score_select and kvswap_sparse_decode layer by layer.
 * A probe's events are recorded on `cuda_stream`: ev_begin before the layer's scorer, ev_mid
 * after its TopK, ev_end after its attention (the attention of the layer before lies between
 * ev_begin and ev_mid).
 */
int kvswap_decode_step(const kvswap_shape* shape, const kvswap_layers* layers, const void* q,
                       float* out, float* lse_opt, int32_t* group_idx, int32_t* n_selected,
                       void* ws, size_t ws_bytes, const kvswap_probe* probe_opt, void* cuda_stream);

/*
 * The decode step over a tiered cache (Sec. 4.4.2, Sec. 4.4.3): the full K/V of every layer lives
 * in a slow tier, each layer has a reuse buffer (kvswap_reuse_* above) in device memory, and the
 * step's attention reads only reuse stores.  Per layer the internal predictor stream runs
 * score/select, kvswap_reuse_lookup and kvswap_reuse_fill, so a layer's misses are fetched while
 * the layers before it are attended on `cuda_stream`; the attention is kvswap_sparse_decode over
 * the layer's reuse store with the slot list.  Arrays of L per-layer pointers are HOST arrays.
 *   K_slow, V_slow    [L] slow-tier stores, laid out by shape's kv strides (GPU-readable memory)
 *   K_reuse, V_reuse  [L] reuse stores [B, H_kv, (n_slots + 1) G, d]; the caller keeps the
 *                     N mod G newest tokens in rows [n_slots G, n_slots G + N mod G)
 *   state             [L] reuse-buffer states of state_bytes each (kvswap_reuse_init)
 *   slot_idx, miss_group, miss_slot [L, B, S, M], n_miss [L, B, S]: device, written by the step
 * layers->K and layers->V are not used (may be NULL).  `ws` needs
 * kvswap_tiered_workspace_bytes(shape, n_slots) bytes.  group_idx / n_selected receive the
 * selections as in kvswap_decode_step.  Errors as for the calls it is made of.
 */
typedef struct {
  int32_t n_slots, max_groups;
  const void* const* K_slow;
  const void* const* V_slow;
  void* const* K_reuse;
  void* const* V_reuse;
  void* const* state;
  size_t state_bytes;
  int32_t* slot_idx;
  int32_t* miss_group;
  int32_t* miss_slot;
  int32_t* n_miss;
} kvswap_tiers;

size_t kvswap_tiered_workspace_bytes(const kvswap_shape* shape, int32_t n_slots);
int kvswap_decode_step_tiered(const kvswap_shape* shape, const kvswap_layers* layers,
                              const kvswap_tiers* tiers, const void* q, float* out, float* lse_opt,
                              int32_t* group_idx, int32_t* n_selected, void* ws, size_t ws_bytes,
                              void* cuda_stream);

/*
 * kvswap_append_step for the tiered cache (Sec. 4.4.1 over Sec. 4.4.2).  shape->n_ctx is N before
 * the call and shape's kv strides describe the slow-tier stores, which need room for row N (as
 * in kvswap_append_kv).  k_new, v_new [L, B, H_kv, d] join the rolling-buffer rows of each
 * layer's reuse store (row n_slots G + N mod G).  When the token completes a group, the group's
 * G rows are written from there to rows [N+1-G, N] of the slow tier (this call WRITES K_slow and
 * V_slow) and its compact-cache rows are built.  Of `tiers` only n_slots, max_groups, K_slow,
 * V_slow, K_reuse and V_reuse are used; KVSWAP_ERR_SHAPE if the grown context has more complete
 * groups than a non-zero max_groups.  Asynchronous on `cuda_stream`.
 */
int kvswap_append_step_tiered(const kvswap_shape* shape, const kvswap_layers* layers,
                              const kvswap_tiers* tiers, const void* k_new, const void* v_new,
                              int32_t* flushed_opt, void* cuda_stream);

/*
 * The same step for callers whose queries and outputs live in HOST memory: q_host
 * [L, B, H_q, d] q_dtype is copied to the device buffer q_dev, the step runs, and out_dev is
 * copied to out_host [L, B, H_q, d] fp32, all asynchronously on `cuda_stream` (use pinned host
 * memory for the copies to overlap; the call returns before they complete).  q_dev, out_dev,
 * group_idx, n_selected and ws are caller-provided device buffers as in kvswap_decode_step.
 */
int kvswap_decode_step_host(const kvswap_shape* shape, const kvswap_layers* layers,
                            const void* q_host, float* out_host, void* q_dev, float* out_dev,
                            int32_t* group_idx, int32_t* n_selected, void* ws, size_t ws_bytes,
                            void* cuda_stream);

/*
 * Calibration helper of the benchmark (the paper has no counterpart): one kernel that does nothing
 * but read `bytes` bytes at `buf` (device; both multiples of 16) with 16-byte loads, on
 * `cuda_stream`.  Timed over buffers of the sizes the predictor and the attention stream, it gives
 * the rate a read-only pass reaches on this GPU and, with bytes = 0, the cost of an empty launch.
 * `sink` (device, 4 bytes, may be NULL) exists only to keep the loads alive.
 */
int kvswap_read_probe(const void* buf, size_t bytes, void* sink, void* cuda_stream);

/* Static, NUL-terminated description of a kvswap_status value. */
const char* kvswap_status_string(int status);

/* Library version as major*10000 + minor*100 + patch. */
int kvswap_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KVSWAP_H_ */
