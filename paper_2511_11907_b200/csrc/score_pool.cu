// K2: low-rank query (Eq. 1), token scoring, head aggregation and group ReduceMax (Sec. 4.3).
//
// The per-head score (Q_h A_g(h)) K_lr^T is linear in the low-rank query, so the sum over the
// heads of a scope is taken on the low-rank queries first:
//     T[b,s,n] = sum_t  uq[b, row(s,t), :] . meta[b, head(t), n, :]
// with, per KV head g,  u_g = (sum_{h: g(h)=g} q_h) A_g  and
//   joint metadata   (H_m = 1):    one term, head 0, uq row s = sum of u_g over the scope;
//   per-head metadata, KV_HEAD:    one term, head g = s, uq row g = u_g;
//   per-head metadata, ALL_HEADS:  H_kv terms, term t reads head t with uq row t = u_t.
#include "common.cuh"

namespace kvswap {
namespace {

constexpr int kThreads = 256;

// ------------------------------------------------------------------------------------------
// K2a: uq rows.  grid (B, rows-or-1): a CTA produces one uq row, looping over the KV heads that
// feed it.
// ------------------------------------------------------------------------------------------
template <typename Q_T>
__global__ void __launch_bounds__(kThreads)
lowrank_query_kernel(Problem p, const Q_T* __restrict__ q, const float* __restrict__ proj,
                     float* __restrict__ uq) {
  __shared__ float qsum[128];
  __shared__ float red[kThreads];
  const int b = blockIdx.x, row = blockIdx.y;
  // KV heads summed into this row
  const bool joint_all = (p.Hm == 1 && p.scope == KVSWAP_SCOPE_ALL_HEADS);
  const int g0 = joint_all ? 0 : row;
  const int g1 = joint_all ? p.Hkv : row + 1;
  const int parts = kThreads / p.r;               // r <= 256
  const int j = threadIdx.x % p.r, part = threadIdx.x / p.r;
  float acc = 0.f;
  for (int g = g0; g < g1; ++g) {
    __syncthreads();
    for (int c = threadIdx.x; c < p.d; c += kThreads) {
      float s = 0.f;
      for (int hh = 0; hh < p.rho; ++hh) {
        const Q_T v = q[(int64_t(b) * p.Hq + g * p.rho + hh) * p.d + c];
        if constexpr (sizeof(Q_T) == 4) s += v; else s += float(v);
      }
      qsum[c] = s;
    }
    __syncthreads();
    if (part < parts) {
      const float* Pg = proj + int64_t(g) * p.d * p.r;
      for (int c = part; c < p.d; c += parts) acc = fmaf(qsum[c], Pg[int64_t(c) * p.r + j], acc);
    }
  }
  red[threadIdx.x] = (part < parts) ? acc : 0.f;
  __syncthreads();
  if (threadIdx.x < p.r) {
    float s = 0.f;
    for (int k = 0; k < parts; ++k) s += red[k * p.r + threadIdx.x];
    uq[(int64_t(b) * p.Su + row) * p.r + threadIdx.x] = s;
  }
}

// ------------------------------------------------------------------------------------------
// K2: generic fp32 scorer.  A CTA owns a tile of whole groups of one sequence and up to NS
// scores per token that share the same metadata row.
// ------------------------------------------------------------------------------------------
template <typename META_T, int NS>
__global__ void __launch_bounds__(kThreads)
score_pool_kernel(Problem p, const float* __restrict__ uq, const META_T* __restrict__ meta,
                  float* __restrict__ scores, int groups_per_tile, int lanes_per_row) {
  extern __shared__ float smem[];
  constexpr int kPer = Elt<META_T>::kPer16B;
  const int b = blockIdx.z, sub = blockIdx.y;
  int ns, n_terms, head0, urow0, out0;
  if (p.Hm == 1) { out0 = urow0 = sub * NS; ns = min(NS, p.S - out0); n_terms = 1; head0 = 0; }
  else if (p.scope == KVSWAP_SCOPE_KV_HEAD) { out0 = urow0 = head0 = sub; ns = 1; n_terms = 1; }
  else { out0 = urow0 = head0 = 0; ns = 1; n_terms = p.Hkv; }

  const int u_rows = max(ns, n_terms);
  float* u_s = smem;                       // [u_rows][r]
  float* sc = smem + u_rows * p.r;         // [NS][tile tokens]
  const int tile_tok = groups_per_tile * p.G;
  for (int i = threadIdx.x; i < u_rows * p.r; i += kThreads)
    u_s[i] = uq[(int64_t(b) * p.Su + urow0) * p.r + i];
  __syncthreads();

  const int grp0 = blockIdx.x * groups_per_tile;
  const int n_grp = min(groups_per_tile, p.NG - grp0);
  const int rows = n_grp * p.G;
  const int64_t tok0 = int64_t(grp0) * p.G;
  const int chunks = p.r / kPer;           // 16-byte chunks per metadata row
  const int lg = threadIdx.x / lanes_per_row, lig = threadIdx.x % lanes_per_row;
  const int n_lg = kThreads / lanes_per_row;
  const META_T* Mb = meta + int64_t(b) * p.meta_sb + int64_t(head0) * p.meta_sh;

  // Every lane-group of a warp runs the same number of iterations (the shuffles need them all).
  for (int rb = 0; rb < rows; rb += n_lg) {
    const int row = rb + lg;
    const bool act = row < rows;
    float part[NS];
#pragma unroll
    for (int k = 0; k < NS; ++k) part[k] = 0.f;
    if (act) {
      for (int t = 0; t < n_terms; ++t) {
        const META_T* Mrow = Mb + int64_t(t) * p.meta_sh + (tok0 + row) * p.meta_sn;
        for (int ch = lig; ch < chunks; ch += lanes_per_row) {
          float f[kPer];
          widen16B(ld_stream16(Mrow + ch * kPer), f, META_T());
#pragma unroll
          for (int k = 0; k < NS; ++k) {
            if (k < ns) {
              const float* u = u_s + (k + t) * p.r + ch * kPer;
#pragma unroll
              for (int e = 0; e < kPer; ++e) part[k] = fmaf(f[e], u[e], part[k]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int k = 0; k < NS; ++k) {
      float v = part[k];
      for (int off = lanes_per_row >> 1; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
      if (act && lig == 0 && k < ns) sc[k * tile_tok + row] = v;
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < ns * n_grp; i += kThreads) {
    const int k = i / n_grp, gi = i % n_grp;
    const float* s = sc + k * tile_tok + gi * p.G;
    float m = s[0];
    for (int t = 1; t < p.G; ++t) m = fmaxf(m, s[t]);
    scores[(int64_t(b) * p.S + out0 + k) * p.NG + grp0 + gi] = m;
  }
}

template <typename META_T, int NS>
cudaError_t launch_ns(const Problem& p, const float* uq, const void* meta, float* scores, int subs_per_b,
                      cudaStream_t st) {
  constexpr int kPer = Elt<META_T>::kPer16B;
  const int chunks = p.r / kPer;
  int lpr = 1;
  while (lpr < chunks && lpr < 32) lpr <<= 1;
  const int gpt = std::max(1, 512 / p.G);
  const int u_rows = std::max(NS, (p.Hm != 1 && p.scope == KVSWAP_SCOPE_ALL_HEADS) ? p.Hkv : 1);
  const size_t smem = sizeof(float) * (size_t(u_rows) * p.r + size_t(NS) * gpt * p.G);
  auto kern = score_pool_kernel<META_T, NS>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
  }
  dim3 grid((p.NG + gpt - 1) / gpt, subs_per_b, p.B);
  kern<<<grid, kThreads, smem, st>>>(p, uq, static_cast<const META_T*>(meta), scores, gpt, lpr);
  return cudaGetLastError();
}

template <typename META_T>
cudaError_t launch_meta(const Problem& p, const float* uq, const void* meta, float* scores, cudaStream_t st) {
  if (p.Hm == 1) {
    if (p.S == 1) return launch_ns<META_T, 1>(p, uq, meta, scores, 1, st);
    if (p.S == 2) return launch_ns<META_T, 2>(p, uq, meta, scores, 1, st);
    if (p.S <= 4) return launch_ns<META_T, 4>(p, uq, meta, scores, 1, st);
    return launch_ns<META_T, 8>(p, uq, meta, scores, (p.S + 7) / 8, st);
  }
  const int subs = (p.scope == KVSWAP_SCOPE_KV_HEAD) ? p.Hkv : 1;
  return launch_ns<META_T, 1>(p, uq, meta, scores, subs, st);
}

}  // namespace

cudaError_t launch_lowrank_query(const Problem& p, const void* q, const float* proj, float* uq, cudaStream_t st) {
  dim3 grid(p.B, p.Su);
  switch (p.q_dtype) {
    case KVSWAP_F32:
      lowrank_query_kernel<float><<<grid, kThreads, 0, st>>>(p, static_cast<const float*>(q), proj, uq); break;
    case KVSWAP_BF16:
      lowrank_query_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>(p, static_cast<const __nv_bfloat16*>(q), proj, uq);
      break;
    default:
      lowrank_query_kernel<__half><<<grid, kThreads, 0, st>>>(p, static_cast<const __half*>(q), proj, uq); break;
  }
  return cudaGetLastError();
}

cudaError_t launch_score_pool(const Problem& p, const float* uq, const void* meta, float* scores, cudaStream_t st) {
  if (p.meta_dtype == KVSWAP_F16) return launch_meta<__half>(p, uq, meta, scores, st);
  return launch_meta<float>(p, uq, meta, scores, st);
}

}  // namespace kvswap
