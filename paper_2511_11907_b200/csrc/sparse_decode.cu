// K4 + K5: exact decode attention over the selected groups and the rolling-buffer tail
// (Sec. 4.4, 4.4.1, 4.4.4): gather + split-K flash-decode with an fp32 online softmax, then a
// log-sum-exp merge of the split partials.
//
// The attended tokens of one (sequence, selection row) form a virtual list
//     v in [0, n_sel*G):  token  group_idx[v / G] * G + v % G
//     v in [n_sel*G, n_sel*G + tail):  token  NG*G + (v - n_sel*G)
// which is cut into `splits` contiguous ranges, one CTA each.  A CTA serves RH query heads that
// share the KV head, so every K/V row is read once per CTA.  Within a warp, a lane-group of
// LPR = d*sizeof(kv)/16 lanes owns one token row; each lane owns 16 bytes of channels.
#include "common.cuh"

namespace kvswap {
namespace {

constexpr int kThreads = 256;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

template <typename Q_T>
__device__ __forceinline__ float q_to_float(Q_T v) { return float(v); }

template <typename KV_T, typename Q_T, int D, int RH>
__global__ void __launch_bounds__(kThreads)
sparse_decode_splitk_kernel(Problem p, const Q_T* __restrict__ q, const KV_T* __restrict__ K,
                            const KV_T* __restrict__ V, const int32_t* __restrict__ group_idx,
                            const int32_t* __restrict__ n_selected, float* __restrict__ partial,
                            int splits) {
  constexpr int EPL = Elt<KV_T>::kPer16B;        // channels per lane
  constexpr int LPR = D / EPL;                   // lanes per token row
  constexpr int NLG = kThreads / LPR;            // lane-groups per CTA
  static_assert(LPR <= 32 && (LPR & (LPR - 1)) == 0, "row must fit a warp");

  const int split = blockIdx.x;
  const int chunks = p.rho / RH;
  const int g = blockIdx.y / chunks, hc = blockIdx.y % chunks;
  const int b = blockIdx.z;
  const int h0 = g * p.rho + hc * RH;            // first query head of this CTA
  const int srow = (p.scope == KVSWAP_SCOPE_KV_HEAD) ? g : 0;
  const int lg = threadIdx.x / LPR, lig = threadIdx.x % LPR;

  const int32_t* idx = group_idx + (int64_t(b) * p.S + srow) * p.M;
  int n_sel = n_selected[int64_t(b) * p.S + srow];
  n_sel = max(0, min(n_sel, p.M));
  const int tail0 = p.NG * p.G;
  const int64_t total = int64_t(n_sel) * p.G + (p.N - tail0);
  const int64_t per_split = (total + splits - 1) / splits;
  const int64_t v_begin = per_split * split, v_end = min(total, v_begin + per_split);

  // q slice of this lane, pre-scaled by log2(e)/sqrt(d): logits live in the log2 domain.
  const float scale = kLog2e * rsqrtf(float(D));
  float qr[RH][EPL];
#pragma unroll
  for (int hh = 0; hh < RH; ++hh)
#pragma unroll
    for (int e = 0; e < EPL; ++e)
      qr[hh][e] = q_to_float(q[(int64_t(b) * p.Hq + h0 + hh) * D + lig * EPL + e]) * scale;

  float m[RH], l[RH], acc[RH][EPL];
#pragma unroll
  for (int hh = 0; hh < RH; ++hh) {
    m[hh] = -INFINITY; l[hh] = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[hh][e] = 0.f;
  }

  const KV_T* Kg = K + int64_t(b) * p.kv_sb + int64_t(g) * p.kv_sh;
  const KV_T* Vg = V + int64_t(b) * p.kv_sb + int64_t(g) * p.kv_sh;
  const int64_t sel_tokens = int64_t(n_sel) * p.G;

  // All lane-groups of a warp run the same number of iterations.
  for (int64_t vb = v_begin; vb < v_end; vb += NLG) {
    const int64_t v = vb + lg;
    int64_t n = -1;
    if (v < v_end) {
      if (v < sel_tokens) {
        const int j = idx[v / p.G];
        if (j >= 0 && j < p.NG) n = int64_t(j) * p.G + (v % p.G);
      } else {
        n = tail0 + (v - sel_tokens);
      }
    }
    float kf[EPL], vf[EPL];
    if (n >= 0) {
      widen16B(ld_stream16(Kg + n * p.kv_sn + lig * EPL), kf, KV_T());
      widen16B(ld_stream16(Vg + n * p.kv_sn + lig * EPL), vf, KV_T());
    } else {
#pragma unroll
      for (int e = 0; e < EPL; ++e) { kf[e] = 0.f; vf[e] = 0.f; }
    }
    float s[RH];
#pragma unroll
    for (int hh = 0; hh < RH; ++hh) {
      float a = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) a = fmaf(qr[hh][e], kf[e], a);
      s[hh] = a;
    }
#pragma unroll
    for (int off = LPR / 2; off > 0; off >>= 1)
#pragma unroll
      for (int hh = 0; hh < RH; ++hh) s[hh] += __shfl_xor_sync(0xffffffffu, s[hh], off);
    if (n >= 0) {
#pragma unroll
      for (int hh = 0; hh < RH; ++hh) {
        const float mn = fmaxf(m[hh], s[hh]);
        const float corr = exp2f(m[hh] - mn);     // exp2(-inf) = 0 on the first token
        const float pw = exp2f(s[hh] - mn);
        l[hh] = fmaf(l[hh], corr, pw);
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[hh][e] = fmaf(acc[hh][e], corr, pw * vf[e]);
        m[hh] = mn;
      }
    }
  }

  // Merge the lane-groups of the CTA: lane-group states to shared memory, then one thread per
  // (head, channel) folds them.
  __shared__ float sm_m[NLG][RH], sm_l[NLG][RH];
  __shared__ float sm_acc[NLG][RH][D + 4];
  if (lig == 0) {
#pragma unroll
    for (int hh = 0; hh < RH; ++hh) { sm_m[lg][hh] = m[hh]; sm_l[lg][hh] = l[hh]; }
  }
#pragma unroll
  for (int hh = 0; hh < RH; ++hh)
#pragma unroll
    for (int e = 0; e < EPL; ++e) sm_acc[lg][hh][lig * EPL + e] = acc[hh][e];
  __syncthreads();
  for (int i = threadIdx.x; i < RH * D; i += kThreads) {
    const int hh = i / D, c = i % D;
    float mx = -INFINITY;
    for (int k = 0; k < NLG; ++k) mx = fmaxf(mx, sm_m[k][hh]);
    float lsum = 0.f, a = 0.f;
    if (mx > -INFINITY) {
      for (int k = 0; k < NLG; ++k) {
        const float w = exp2f(sm_m[k][hh] - mx);
        lsum = fmaf(sm_l[k][hh], w, lsum);
        a = fmaf(sm_acc[k][hh][c], w, a);
      }
    }
    float* dst = partial + ((int64_t(b) * p.Hq + h0 + hh) * splits + split) * (D + 2);
    if (c == 0) { dst[0] = mx; dst[1] = lsum; }
    dst[2 + c] = a;
  }
}

// K5: merge the split partials of one (sequence, head).
template <int D>
__global__ void __launch_bounds__(D)
combine_kernel(const float* __restrict__ partial, float* __restrict__ out, float* __restrict__ lse, int splits) {
  const int64_t bh = blockIdx.x;
  const float* src = partial + bh * splits * (D + 2);
  const int c = threadIdx.x;
  float mx = -INFINITY;
  for (int s = 0; s < splits; ++s) mx = fmaxf(mx, src[s * (D + 2)]);
  float lsum = 0.f, a = 0.f;
  if (mx > -INFINITY) {
    for (int s = 0; s < splits; ++s) {
      const float w = exp2f(src[s * (D + 2)] - mx);
      lsum = fmaf(src[s * (D + 2) + 1], w, lsum);
      a = fmaf(src[s * (D + 2) + 2 + c], w, a);
    }
  }
  out[bh * D + c] = (lsum > 0.f) ? a / lsum : 0.f;
  if (lse != nullptr && c == 0) lse[bh] = (lsum > 0.f) ? (mx + log2f(lsum)) * kLn2 : -INFINITY;
}

template <typename KV_T, typename Q_T, int D, int RH>
cudaError_t launch_one(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                       const int32_t* group_idx, const int32_t* n_selected, float* partial, float* out, float* lse,
                       cudaStream_t st) {
  dim3 grid(w.splits, p.Hkv * (p.rho / RH), p.B);
  sparse_decode_splitk_kernel<KV_T, Q_T, D, RH><<<grid, kThreads, 0, st>>>(
      p, static_cast<const Q_T*>(q), static_cast<const KV_T*>(K), static_cast<const KV_T*>(V), group_idx,
      n_selected, partial, w.splits);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  combine_kernel<D><<<p.B * p.Hq, D, 0, st>>>(partial, out, lse, w.splits);
  return cudaGetLastError();
}

template <typename KV_T, typename Q_T, int D>
cudaError_t launch_rh(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                      const int32_t* gi, const int32_t* ns, float* partial, float* out, float* lse, cudaStream_t st) {
  switch (w.heads_per_cta) {
    case 4: return launch_one<KV_T, Q_T, D, 4>(p, w, q, K, V, gi, ns, partial, out, lse, st);
    case 3: return launch_one<KV_T, Q_T, D, 3>(p, w, q, K, V, gi, ns, partial, out, lse, st);
    case 2: return launch_one<KV_T, Q_T, D, 2>(p, w, q, K, V, gi, ns, partial, out, lse, st);
    default: return launch_one<KV_T, Q_T, D, 1>(p, w, q, K, V, gi, ns, partial, out, lse, st);
  }
}

template <typename KV_T, typename Q_T>
cudaError_t launch_d(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                     const int32_t* gi, const int32_t* ns, float* partial, float* out, float* lse, cudaStream_t st) {
  if (p.d == 128) return launch_rh<KV_T, Q_T, 128>(p, w, q, K, V, gi, ns, partial, out, lse, st);
  return launch_rh<KV_T, Q_T, 64>(p, w, q, K, V, gi, ns, partial, out, lse, st);
}

template <typename KV_T>
cudaError_t launch_q(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                     const int32_t* gi, const int32_t* ns, float* partial, float* out, float* lse, cudaStream_t st) {
  // q is stored as fp32 or in the K/V type (checked at validation).
  if (p.q_dtype == KVSWAP_F32) return launch_d<KV_T, float>(p, w, q, K, V, gi, ns, partial, out, lse, st);
  return launch_d<KV_T, KV_T>(p, w, q, K, V, gi, ns, partial, out, lse, st);
}

}  // namespace

cudaError_t launch_sparse_decode(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                                 const int32_t* group_idx, const int32_t* n_selected, float* partial, float* out,
                                 float* lse, cudaStream_t st) {
  switch (p.kv_dtype) {
    case KVSWAP_F32: return launch_q<float>(p, w, q, K, V, group_idx, n_selected, partial, out, lse, st);
    case KVSWAP_BF16: return launch_q<__nv_bfloat16>(p, w, q, K, V, group_idx, n_selected, partial, out, lse, st);
    default: return launch_q<__half>(p, w, q, K, V, group_idx, n_selected, partial, out, lse, st);
  }
}

}  // namespace kvswap
