// Predictor variant (KVSWAP_SCORE_SOFTMAX): every head's low-rank logits pass through a softmax over
// the tokens of the context's complete groups, scaled by 1/sqrt(d) as attention scales them, before
// the head sum -- approximate attention weights instead of approximate logits (the other reading
// of "attention scores" in Sec. 4.3).  The sum over heads no longer commutes with the dot product,
// so each head is scored on its own, and the normaliser needs a pass of its own:
//   lowrank_query_heads_kernel  u[b,h,:] = q[b,h,:] A_g(h) * log2(e) / sqrt(d)      (logits in base 2)
//   softmax_stats_kernel        per (sequence, head, chunk of 1024 tokens): running max and sum of
//                               2^(logit - max); also clears the group-score buffer
//   softmax_pool_kernel         combines the chunks' statistics, recomputes the logits, sums the
//                               heads' weights per selection scope and takes the group maximum
//                               (weights are non-negative, so an integer atomicMax on the float's
//                               bits orders them)
// Plain fp32-pipe kernels: metadata rows are re-read once per block of eight heads (from L2).
#include <algorithm>

#include "common.cuh"

namespace kvswap {
namespace {

constexpr int kThreads = 256;
constexpr int kTokensPerThread = 4;
constexpr int kChunkTokens = kThreads * kTokensPerThread;     // tokens per CTA
constexpr int kHeadBlock = 8;                                 // heads scored per pass over a row
constexpr float kLog2e = 1.4426950408889634f;

template <typename Q_T>
__global__ void __launch_bounds__(kThreads)
lowrank_query_heads_kernel(Problem p, const Q_T* __restrict__ q, const float* __restrict__ proj, float* __restrict__ u) {
  const int b = blockIdx.x, h = blockIdx.y, g = h / p.rho;
  const Q_T* qh = q + (int64_t(b) * p.Hq + h) * p.d;
  const float* A = proj + int64_t(g) * p.d * p.r;
  const float scale = kLog2e * rsqrtf(float(p.d));
  for (int j = threadIdx.x; j < p.r; j += kThreads) {
    float acc = 0.f;
    for (int c = 0; c < p.d; ++c) acc = fmaf(float(qh[c]), A[int64_t(c) * p.r + j], acc);
    u[(int64_t(b) * p.Hq + h) * p.r + j] = acc * scale;
  }
}

__device__ __forceinline__ void load4(const float* row, int k, float (&m)[4]) {
  const float4 v = *reinterpret_cast<const float4*>(row + k);
  m[0] = v.x; m[1] = v.y; m[2] = v.z; m[3] = v.w;
}
__device__ __forceinline__ void load4(const __half* row, int k, float (&m)[4]) {
  const uint2 v = *reinterpret_cast<const uint2*>(row + k);
  const __half2 a = *reinterpret_cast<const __half2*>(&v.x), c = *reinterpret_cast<const __half2*>(&v.y);
  m[0] = __low2float(a); m[1] = __high2float(a); m[2] = __low2float(c); m[3] = __high2float(c);
}

// Base-2 logits of heads h0 .. h0 + nh - 1 (all on metadata head hm) for one token row.
template <typename META_T>
__device__ __forceinline__ void head_logits(const Problem& p, const META_T* row, const float* u_s, int h0, int nh,
                                            float (&s)[kHeadBlock]) {
#pragma unroll
  for (int i = 0; i < kHeadBlock; ++i) s[i] = 0.f;
  for (int k = 0; k < p.r; k += 4) {
    float m[4];
    load4(row, k, m);
#pragma unroll
    for (int i = 0; i < kHeadBlock; ++i) {
      if (i < nh) {
        // shared memory, same address across the warp: one 16-byte broadcast read per four products
        const float4 uh = *reinterpret_cast<const float4*>(u_s + (h0 + i) * p.r + k);
        s[i] = fmaf(uh.x, m[0], fmaf(uh.y, m[1], fmaf(uh.z, m[2], fmaf(uh.w, m[3], s[i]))));
      }
    }
  }
}

// Heads are visited in blocks of at most kHeadBlock that share a metadata head: with joint metadata
// any eight consecutive heads, with per-head metadata the heads of one KV head.
__device__ __forceinline__ int block_heads(const Problem& p, int h0) {
  const int limit = (p.Hm == 1) ? p.Hq : (h0 / p.rho + 1) * p.rho;
  return min(kHeadBlock, limit - h0);
}

template <typename META_T>
__global__ void __launch_bounds__(kThreads)
softmax_stats_kernel(Problem p, const float* __restrict__ u, const META_T* __restrict__ meta, float* __restrict__ stats,
                     float* __restrict__ scores, int chunks, int n_scored) {
  extern __shared__ __align__(16) float u_s[];                 // [Hq][r]
  __shared__ float red_m[kThreads / 32][kHeadBlock], red_l[kThreads / 32][kHeadBlock];
  const int chunk = blockIdx.x, b = blockIdx.y;
  for (int i = threadIdx.x; i < p.Hq * p.r; i += kThreads) u_s[i] = u[int64_t(b) * p.Hq * p.r + i];
  // the group-score buffer of this sequence is cleared here, before the pooling kernel runs
  {
    const int64_t row_elems = int64_t(p.S) * p.score_pitch;
    for (int64_t i = int64_t(chunk) * kThreads + threadIdx.x; i < row_elems; i += int64_t(chunks) * kThreads)
      scores[int64_t(b) * row_elems + i] = 0.f;
  }
  __syncthreads();
  const int n0 = chunk * kChunkTokens;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int h0 = 0; h0 < p.Hq;) {
    const int nh = block_heads(p, h0);
    const int hm = (p.Hm == 1) ? 0 : h0 / p.rho;
    const META_T* base = meta + int64_t(b) * p.meta_sb + int64_t(hm) * p.meta_sh;
    float mx[kHeadBlock], l[kHeadBlock];
#pragma unroll
    for (int i = 0; i < kHeadBlock; ++i) { mx[i] = -INFINITY; l[i] = 0.f; }
    for (int t = 0; t < kTokensPerThread; ++t) {
      const int n = n0 + t * kThreads + threadIdx.x;
      if (n < n_scored) {
        float s[kHeadBlock];
        head_logits(p, base + int64_t(n) * p.meta_sn, u_s, h0, nh, s);
#pragma unroll
        for (int i = 0; i < kHeadBlock; ++i) {
          if (i < nh) {
            const float m_new = fmaxf(mx[i], s[i]);
            l[i] = l[i] * exp2f(mx[i] - m_new) + exp2f(s[i] - m_new);     // exp2f(-inf) = 0 on the first token
            mx[i] = m_new;
          }
        }
      }
    }
    // reduce over the CTA: lanes, then warps
#pragma unroll
    for (int i = 0; i < kHeadBlock; ++i) {
      float m_w = mx[i];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) m_w = fmaxf(m_w, __shfl_xor_sync(0xffffffffu, m_w, off));
      float l_w = (mx[i] > -INFINITY) ? l[i] * exp2f(mx[i] - m_w) : 0.f;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) l_w += __shfl_xor_sync(0xffffffffu, l_w, off);
      if (lane == 0) { red_m[warp][i] = m_w; red_l[warp][i] = l_w; }
    }
    __syncthreads();
    if (threadIdx.x < nh) {
      const int i = threadIdx.x;
      float m_c = -INFINITY;
      for (int w = 0; w < kThreads / 32; ++w) m_c = fmaxf(m_c, red_m[w][i]);
      float l_c = 0.f;
      for (int w = 0; w < kThreads / 32; ++w)
        if (red_m[w][i] > -INFINITY) l_c += red_l[w][i] * exp2f(red_m[w][i] - m_c);
      float* dst = stats + ((int64_t(b) * p.Hq + h0 + i) * chunks + chunk) * 2;
      dst[0] = m_c; dst[1] = l_c;
    }
    __syncthreads();
    h0 += nh;
  }
}

template <typename META_T>
__global__ void __launch_bounds__(kThreads)
softmax_pool_kernel(Problem p, const float* __restrict__ u, const META_T* __restrict__ meta,
                    const float* __restrict__ stats, float* __restrict__ scores, int chunks, int n_scored) {
  extern __shared__ __align__(16) float smem[];
  float* u_s = smem;                                           // [Hq][r]
  float* m_s = u_s + p.Hq * p.r;                               // [Hq] maximum of the head's logits
  float* z_s = m_s + p.Hq;                                     // [Hq] 1 / sum of 2^(logit - max)
  const int chunk = blockIdx.x, b = blockIdx.y;
  for (int i = threadIdx.x; i < p.Hq * p.r; i += kThreads) u_s[i] = u[int64_t(b) * p.Hq * p.r + i];
  for (int h = threadIdx.x; h < p.Hq; h += kThreads) {
    const float* src = stats + (int64_t(b) * p.Hq + h) * chunks * 2;
    float m = -INFINITY;
    for (int c = 0; c < chunks; ++c) m = fmaxf(m, src[2 * c]);
    float l = 0.f;
    for (int c = 0; c < chunks; ++c)
      if (src[2 * c] > -INFINITY) l += src[2 * c + 1] * exp2f(src[2 * c] - m);
    m_s[h] = m;
    z_s[h] = 1.f / l;                                          // l >= 1: the maximum itself contributes 1
  }
  __syncthreads();
  const int n0 = chunk * kChunkTokens;
  const bool per_kv = (p.scope == KVSWAP_SCOPE_KV_HEAD);
  for (int t = 0; t < kTokensPerThread; ++t) {
    const int n = n0 + t * kThreads + threadIdx.x;
    if (n >= n_scored) continue;
    const int grp = n / p.G;
    float total = 0.f;                                         // all-heads scope
    for (int g = 0; g < p.Hkv; ++g) {
      float t_g = 0.f;
      const int hm = (p.Hm == 1) ? 0 : g;
      const META_T* row = meta + int64_t(b) * p.meta_sb + int64_t(hm) * p.meta_sh + int64_t(n) * p.meta_sn;
      for (int h0 = g * p.rho; h0 < (g + 1) * p.rho; h0 += kHeadBlock) {
        const int nh = min(kHeadBlock, (g + 1) * p.rho - h0);
        float s[kHeadBlock];
        head_logits(p, row, u_s, h0, nh, s);
#pragma unroll
        for (int i = 0; i < kHeadBlock; ++i)
          if (i < nh) t_g = fmaf(exp2f(s[i] - m_s[h0 + i]), z_s[h0 + i], t_g);
      }
      if (per_kv)
        atomicMax(reinterpret_cast<int*>(scores + (int64_t(b) * p.S + g) * p.score_pitch + grp), __float_as_int(t_g));
      else
        total += t_g;
    }
    if (!per_kv) atomicMax(reinterpret_cast<int*>(scores + int64_t(b) * p.S * p.score_pitch + grp), __float_as_int(total));
  }
}

template <typename META_T>
cudaError_t launch_stats_and_pool(const Problem& p, const float* u, const void* meta, float* stats, float* scores,
                                  int chunks, int n_scored, cudaStream_t st) {
  const size_t smem1 = sizeof(float) * size_t(p.Hq) * p.r;
  const size_t smem2 = smem1 + sizeof(float) * 2 * size_t(p.Hq);
  cudaError_t e = cudaFuncSetAttribute(softmax_stats_kernel<META_T>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem1));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(softmax_pool_kernel<META_T>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem2));
  if (e != cudaSuccess) return e;
  const META_T* m = static_cast<const META_T*>(meta);
  softmax_stats_kernel<META_T><<<dim3(chunks, p.B), kThreads, smem1, st>>>(p, u, m, stats, scores, chunks, n_scored);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  softmax_pool_kernel<META_T><<<dim3(chunks, p.B), kThreads, smem2, st>>>(p, u, m, stats, scores, chunks, n_scored);
  return cudaGetLastError();
}

}  // namespace

int score_softmax_chunks(const Problem& p) { return std::max(1, (p.NG * p.G + kChunkTokens - 1) / kChunkTokens); }

bool score_softmax_supported(const Problem& p) {
  return (size_t(p.Hq) * p.r + 2 * size_t(p.Hq)) * sizeof(float) <= 160 * 1024;
}

// Group scores R[b, s, j] (row pitch p.score_pitch) of the softmax variant.  u: [B, H_q, r] floats,
// stats: [B, H_q, chunks, 2] floats, both scratch.
cudaError_t launch_score_softmax(const Problem& p, const void* q, const float* proj, const void* meta, float* u,
                                 float* stats, float* scores, cudaStream_t st) {
  const dim3 grid(p.B, p.Hq);
  switch (p.q_dtype) {
    case KVSWAP_F32:
      lowrank_query_heads_kernel<float><<<grid, kThreads, 0, st>>>(p, static_cast<const float*>(q), proj, u);
      break;
    case KVSWAP_BF16:
      lowrank_query_heads_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>(p, static_cast<const __nv_bfloat16*>(q), proj, u);
      break;
    default:
      lowrank_query_heads_kernel<__half><<<grid, kThreads, 0, st>>>(p, static_cast<const __half*>(q), proj, u);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess || p.NG == 0) return e;
  const int chunks = score_softmax_chunks(p), n_scored = p.NG * p.G;
  if (p.meta_dtype == KVSWAP_F16) return launch_stats_and_pool<__half>(p, u, meta, stats, scores, chunks, n_scored, st);
  return launch_stats_and_pool<float>(p, u, meta, stats, scores, chunks, n_scored, st);
}

}  // namespace kvswap
