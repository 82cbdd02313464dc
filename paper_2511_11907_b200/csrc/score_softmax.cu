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
  // eight slices of the contraction index x 32 output columns; columns beyond 32 in further rounds
  __shared__ float part_sum[8][32];
  const int b = blockIdx.x, h = blockIdx.y, g = h / p.rho;
  const Q_T* qh = q + (int64_t(b) * p.Hq + h) * p.d;
  const float* A = proj + int64_t(g) * p.d * p.r;
  const float scale = kLog2e * rsqrtf(float(p.d));
  const int lane = threadIdx.x & 31, part = threadIdx.x >> 5, per_part = p.d / 8;
  for (int j0 = 0; j0 < p.r; j0 += 32) {
    const int j = j0 + lane;
    float acc = 0.f;
    if (j < p.r)
      for (int c = part * per_part; c < (part + 1) * per_part; ++c) acc = fmaf(float(qh[c]), A[int64_t(c) * p.r + j], acc);
    part_sum[part][lane] = acc;
    __syncthreads();
    if (part == 0 && j < p.r) {
      float sum = 0.f;
#pragma unroll
      for (int k = 0; k < 8; ++k) sum += part_sum[k][lane];
      u[(int64_t(b) * p.Hq + h) * p.r + j] = sum * scale;
    }
    __syncthreads();
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


// (max, 1 / normaliser) of one head from its per-chunk statistics; the eight lanes of an aligned
// group of eight call together (lane index `part`), each takes every eighth chunk.
__device__ __forceinline__ void combine_stats(const float* __restrict__ src, int chunks, int part, float* m_out,
                                              float* z_out) {
  float m = -INFINITY, l = 0.f;
  for (int c = part; c < chunks; c += 8) {
    const float mc = src[2 * c], lc = src[2 * c + 1];
    const float m_new = fmaxf(m, mc);
    if (m_new > -INFINITY) { l = l * exp2f(m - m_new) + lc * exp2f(mc - m_new); m = m_new; }
  }
#pragma unroll
  for (int off = 1; off <= 4; off <<= 1) {
    const float m_o = __shfl_xor_sync(0xffffffffu, m, off), l_o = __shfl_xor_sync(0xffffffffu, l, off);
    const float m_new = fmaxf(m, m_o);
    if (m_new > -INFINITY) { l = l * exp2f(m - m_new) + l_o * exp2f(m_o - m_new); m = m_new; }
  }
  *m_out = m;
  *z_out = 1.f / l;                                            // l >= 1: the maximum itself contributes 1
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
  for (int h0 = 0; h0 < p.Hq; h0 += kThreads / 8) {           // eight lanes per head
    const int h = min(h0 + int(threadIdx.x) / 8, p.Hq - 1);
    float m, z;
    combine_stats(stats + (int64_t(b) * p.Hq + h) * chunks * 2, chunks, threadIdx.x & 7, &m, &z);
    if ((threadIdx.x & 7) == 0) { m_s[h] = m; z_s[h] = z; }
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


// ------------------------------------------------------------------------------------------
// Tensor-core path: joint fp16 metadata with 64-byte rows (r = 32), at most 32 query heads.
//
// The logits of a row for all heads are a [H_q x r] . [r x 1] product; for eight consecutive
// tokens that is two mma.sync m16n8k16 row tiles (heads 0..15, 16..31) x two k-steps.  The row
// operand holds the per-head low-rank queries, each head scaled by a power of two so that its
// largest entry lies in [1024, 2048) and split into an fp16 head and remainder (both products are
// exact in the fp32 accumulator; the scale is undone exactly afterwards).  The column operand is
// read straight from global memory: lane (g, t) needs halves 2t, 2t+1, 2t+8, 2t+9 of the k-step's
// 16 entries of token g -- two 4-byte loads, and a warp covers 8 rows x 64 bytes = 512 contiguous
// bytes.  The accumulator leaves lane (g, t) with heads g and g + 8 of each row tile for tokens 2t
// and 2t + 1.  One template serves both passes.
// ------------------------------------------------------------------------------------------
constexpr int kTcWarps = 8;
constexpr int kTcChunkTokens = 1024;                          // per CTA: 16 tiles of 8 tokens per warp
constexpr int kTcHeads = 32;
constexpr int kTcRank = 32;

__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  return uint32_t(__half_as_ushort(__float2half_rn(lo))) | (uint32_t(__half_as_ushort(__float2half_rn(hi))) << 16);
}

// HS: heads per scope when it is a power of two (the head sum then runs over the accumulator
// fragments with shuffles), 0 otherwise (through shared memory).  Ignored by the statistics pass.
template <bool POOL, int HS>
__global__ void __launch_bounds__(kTcWarps * 32)
softmax_tc_kernel(Problem p, const float* __restrict__ u, const __half* __restrict__ meta, float* __restrict__ stats,
                  float* __restrict__ scores, int chunks, int n_scored) {
  __shared__ float u_s[kTcHeads][kTcRank + 1];                 // zero rows beyond H_q
  __shared__ float unscale_s[kTcHeads];                        // 2^-k of the head's scale
  __shared__ float m_s[kTcHeads], z_s[kTcHeads];               // POOL: the head's maximum and 1 / normaliser
  __shared__ float red[kTcWarps][kTcHeads][2];                 // !POOL: per-warp (max, sum)
  __shared__ float ps[kTcWarps][kTcHeads][9];                  // POOL: a warp's weights of one tile, [head][token]
  const int chunk = blockIdx.x, b = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;

  for (int i = threadIdx.x; i < kTcHeads * kTcRank; i += blockDim.x) {
    const int h = i / kTcRank, k = i % kTcRank;
    u_s[h][k] = (h < p.Hq) ? u[(int64_t(b) * p.Hq + h) * kTcRank + k] : 0.f;
  }
  if (!POOL) {                                                  // clear this sequence's group scores for the second pass
    const int64_t row_elems = int64_t(p.S) * p.score_pitch;
    for (int64_t i = int64_t(chunk) * blockDim.x + threadIdx.x; i < row_elems; i += int64_t(chunks) * blockDim.x)
      scores[int64_t(b) * row_elems + i] = 0.f;
  }
  __syncthreads();
  if (threadIdx.x < kTcHeads) {
    const int h = threadIdx.x;
    float mx = 0.f;
    for (int k = 0; k < kTcRank; ++k) mx = fmaxf(mx, fabsf(u_s[h][k]));
    int e = 0;
    if (mx > 0.f) { frexpf(mx, &e); }                          // mx = f 2^e, f in [0.5, 1)
    const int shift = 11 - e;                                  // mx 2^shift in [1024, 2048)
    unscale_s[h] = ldexpf(1.f, -shift);
    const float up = ldexpf(1.f, shift);
    for (int k = 0; k < kTcRank; ++k) u_s[h][k] *= up;        // exact
  }
  if (POOL) {                                                  // 32 heads x eight lanes
    const int h = min(int(threadIdx.x) / 8, p.Hq - 1);
    float m, z;
    combine_stats(stats + (int64_t(b) * p.Hq + h) * chunks * 2, chunks, threadIdx.x & 7, &m, &z);
    if ((threadIdx.x & 7) == 0 && int(threadIdx.x) / 8 < p.Hq) { m_s[h] = m; z_s[h] = z; }
  }
  __syncthreads();

  // Row-operand fragments: [row tile][k-step] x (head part, remainder).
  uint32_t a_hi[2][2][4], a_lo[2][2][4];
  float unscale[4];                                            // rows g, g+8, g+16, g+24
#pragma unroll
  for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {                            // a0: (g, k), a1: (g+8, k), a2: (g, k+8), a3: (g+8, k+8)
        const int row = mt * 16 + g + (q & 1) * 8, k = ks * 16 + 2 * t + (q >> 1) * 8;
        const float x0 = u_s[row][k], x1 = u_s[row][k + 1];
        const float h0 = __half2float(__float2half_rn(x0)), h1 = __half2float(__float2half_rn(x1));
        a_hi[mt][ks][q] = pack2(h0, h1);
        a_lo[mt][ks][q] = pack2(x0 - h0, x1 - h1);
      }
    }
    unscale[2 * mt] = unscale_s[mt * 16 + g];
    unscale[2 * mt + 1] = unscale_s[mt * 16 + g + 8];
  }
  float row_m[4], row_z[4];
  if (POOL) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = (i >> 1) * 16 + g + (i & 1) * 8;
      row_m[i] = (row < p.Hq) ? m_s[row] : 0.f;
      row_z[i] = (row < p.Hq) ? z_s[row] : 0.f;
    }
  }
  float mx[4], l[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) { mx[i] = -INFINITY; l[i] = 0.f; }

  const __half* base = meta + int64_t(b) * p.meta_sb;
  const int tiles = kTcChunkTokens / 8 / kTcWarps;            // per warp
  const bool per_kv = (p.scope == KVSWAP_SCOPE_KV_HEAD);
  // Heads summed into one scope: rho, or every (padded) row for the all-heads scope.  A power of two
  // lets the sum run over the accumulator fragments with shuffles; otherwise through shared memory.
  constexpr int hs = HS;
  constexpr bool shuffle_sum = HS > 0;
  float w_tok[4][2];
  float* const scores_b = scores + int64_t(b) * p.S * p.score_pitch;
  const bool tile_in_group = (p.G & 7) == 0;
  // column operand of tile `it`: token n0 + g (clamped into the scored range; masked below)
  auto load_tile = [&](int it, uint32_t (&frag)[2][2]) {
    const int n_ld = min(chunk * kTcChunkTokens + (warp * tiles + it) * 8 + g, n_scored - 1);
    const uint32_t* row = reinterpret_cast<const uint32_t*>(base + int64_t(n_ld) * p.meta_sn);
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) { frag[ks][0] = row[ks * 8 + t]; frag[ks][1] = row[ks * 8 + 4 + t]; }
  };
  constexpr int kAhead = 4;                                    // tiles whose rows are in flight
  uint32_t ring[kAhead][2][2];
#pragma unroll
  for (int i = 0; i < kAhead; ++i) load_tile(i, ring[i]);
#pragma unroll 4
  for (int it = 0; it < tiles; ++it) {
    const int n0 = chunk * kTcChunkTokens + (warp * tiles + it) * 8;
    if (n0 >= n_scored) break;                                 // warp-uniform
    uint32_t bfrag[2][2];
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) { bfrag[ks][0] = ring[it % kAhead][ks][0]; bfrag[ks][1] = ring[it % kAhead][ks][1]; }
    if (it + kAhead < tiles) load_tile(it + kAhead, ring[it % kAhead]);
    float acc[2][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[mt][q] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 2; ++ks) {
        mma16816(acc[mt], a_lo[mt][ks], bfrag[ks][0], bfrag[ks][1]);
        mma16816(acc[mt], a_hi[mt][ks], bfrag[ks][0], bfrag[ks][1]);
      }
    }
    // acc[mt][0], [1]: head mt*16+g, tokens n0+2t, +1;  acc[mt][2], [3]: head mt*16+g+8
    const bool v0 = n0 + 2 * t < n_scored, v1 = n0 + 2 * t + 1 < n_scored;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int mt = i >> 1, half = i & 1;
      const float s0 = acc[mt][2 * half] * unscale[i], s1 = acc[mt][2 * half + 1] * unscale[i];
      if (!POOL) {
        const float c0 = v0 ? s0 : -INFINITY, c1 = v1 ? s1 : -INFINITY;
        const float m_new = fmaxf(mx[i], fmaxf(c0, c1));
        if (m_new > -INFINITY) {
          l[i] = l[i] * exp2f(mx[i] - m_new) + exp2f(c0 - m_new) + exp2f(c1 - m_new);
          mx[i] = m_new;
        }
      } else {
        w_tok[i][0] = v0 ? exp2f(s0 - row_m[i]) * row_z[i] : 0.f;
        w_tok[i][1] = v1 ? exp2f(s1 - row_m[i]) * row_z[i] : 0.f;
        if (!shuffle_sum) {
          const int head = mt * 16 + g + half * 8;
          ps[warp][head][2 * t] = w_tok[i][0];
          ps[warp][head][2 * t + 1] = w_tok[i][1];
        }
      }
    }
    if (POOL && shuffle_sum) {
      // Rows 8i .. 8i+7 are value i of the eight lane groups g.  hs < 8: sum over the low bits of g
      // (lanes 4 apart, 8 apart); the scope of value i in lane group g is (8i + g) / hs.  hs >= 8: sum
      // over all of g, then over hs / 8 consecutive values.
#pragma unroll
      for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          float w = w_tok[i][c];
          if (hs >= 2) w += __shfl_xor_sync(0xffffffffu, w, 4);
          if (hs >= 4) w += __shfl_xor_sync(0xffffffffu, w, 8);
          if (hs >= 8) w += __shfl_xor_sync(0xffffffffu, w, 16);
          w_tok[i][c] = w;
        }
      }
      constexpr int vals_per_scope = (hs >= 8) ? hs / 8 : 1;
      const int grp0 = n0 / p.G;
#pragma unroll
      for (int i = 0; i < 4; i += vals_per_scope) {
        float w0 = w_tok[i][0], w1 = w_tok[i][1];
#pragma unroll
        for (int k = 1; k < vals_per_scope; ++k) { w0 += w_tok[i + k][0]; w1 += w_tok[i + k][1]; }
        const int sc = (hs < 8) ? (8 * i + g) / hs : (8 * i) / hs;
        const bool owner = ((hs < 8) ? ((g & (hs - 1)) == 0) : (g == 0)) && sc < p.S;
        float* dst = scores_b + int64_t(sc) * p.score_pitch;
        if (tile_in_group) {
          float w = fmaxf(w0, w1);
          w = fmaxf(w, __shfl_xor_sync(0xffffffffu, w, 1));
          w = fmaxf(w, __shfl_xor_sync(0xffffffffu, w, 2));
          if (owner && t == 0) atomicMax(reinterpret_cast<int*>(dst + grp0), __float_as_int(w));
        } else if (owner) {
          if (v0) atomicMax(reinterpret_cast<int*>(dst + (n0 + 2 * t) / p.G), __float_as_int(w0));
          if (v1) atomicMax(reinterpret_cast<int*>(dst + (n0 + 2 * t + 1) / p.G), __float_as_int(w1));
        }
      }
    }
    if (POOL && !shuffle_sum) {
      __syncwarp();
      // entries (scope, token): lane e and e + 32, ... ; a scope's eight tokens sit in eight consecutive lanes
      const int n_entries = p.S * 8;
      for (int e = lane; e < ((n_entries + 31) & ~31); e += 32) {
        float w = 0.f;
        int sc = e >> 3;
        const int tok = e & 7;
        if (e < n_entries) {
          const int h_begin = per_kv ? sc * p.rho : 0, h_end = per_kv ? h_begin + p.rho : p.Hq;
          for (int h = h_begin; h < h_end; ++h) w += ps[warp][h][tok];
        }
        const int n = n0 + tok;
        if (tile_in_group) {                                   // the tile lies inside one group: reduce it first
          w = fmaxf(w, __shfl_xor_sync(0xffffffffu, w, 1));
          w = fmaxf(w, __shfl_xor_sync(0xffffffffu, w, 2));
          w = fmaxf(w, __shfl_xor_sync(0xffffffffu, w, 4));
          if (tok == 0 && e < n_entries)
            atomicMax(reinterpret_cast<int*>(scores + (int64_t(b) * p.S + sc) * p.score_pitch + n0 / p.G),
                      __float_as_int(w));
        } else if (e < n_entries && n < n_scored) {
          atomicMax(reinterpret_cast<int*>(scores + (int64_t(b) * p.S + sc) * p.score_pitch + n / p.G),
                    __float_as_int(w));
        }
      }
      __syncwarp();
    }
  }

  if (!POOL) {
    // the four lanes of a row, then the warps, then one (max, sum) per head and chunk
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
      for (int off = 1; off <= 2; off <<= 1) {
        const float m_o = __shfl_xor_sync(0xffffffffu, mx[i], off), l_o = __shfl_xor_sync(0xffffffffu, l[i], off);
        const float m_new = fmaxf(mx[i], m_o);
        if (m_new > -INFINITY) {
          l[i] = l[i] * exp2f(mx[i] - m_new) + l_o * exp2f(m_o - m_new);
          mx[i] = m_new;
        }
      }
      if (t == 0) {
        const int head = (i >> 1) * 16 + g + (i & 1) * 8;
        red[warp][head][0] = mx[i];
        red[warp][head][1] = l[i];
      }
    }
    __syncthreads();
    if (threadIdx.x < p.Hq) {
      const int h = threadIdx.x;
      float m_c = -INFINITY;
      for (int w = 0; w < kTcWarps; ++w) m_c = fmaxf(m_c, red[w][h][0]);
      float l_c = 0.f;
      for (int w = 0; w < kTcWarps; ++w)
        if (red[w][h][0] > -INFINITY) l_c += red[w][h][1] * exp2f(red[w][h][0] - m_c);
      float* dst = stats + ((int64_t(b) * p.Hq + h) * chunks + chunk) * 2;
      dst[0] = m_c; dst[1] = l_c;
    }
  }
}

bool tensor_core_case(const Problem& p) {
  return p.Hm == 1 && p.meta_dtype == KVSWAP_F16 && p.r == kTcRank && p.meta_sn == kTcRank && p.Hq <= kTcHeads;
}

}  // namespace

// Chunks per sequence: the tensor-core path's chunks are never longer than the general path's, so
// its count bounds both (the statistics buffer is sized from it).
int score_softmax_chunks(const Problem& p) { return std::max(1, (p.NG * p.G + kTcChunkTokens - 1) / kTcChunkTokens); }

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
  const int n_scored = p.NG * p.G;
  if (tensor_core_case(p)) {
    const int chunks = (n_scored + kTcChunkTokens - 1) / kTcChunkTokens;
    const __half* m = static_cast<const __half*>(meta);
    const dim3 grid(chunks, p.B), block(kTcWarps * 32);
    softmax_tc_kernel<false, 0><<<grid, block, 0, st>>>(p, u, m, stats, scores, chunks, n_scored);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    const int hs = (p.scope == KVSWAP_SCOPE_KV_HEAD) ? p.rho : kTcHeads;      // padded rows carry no weight
    switch (hs) {
      case 1: softmax_tc_kernel<true, 1><<<grid, block, 0, st>>>(p, u, m, stats, scores, chunks, n_scored); break;
      case 2: softmax_tc_kernel<true, 2><<<grid, block, 0, st>>>(p, u, m, stats, scores, chunks, n_scored); break;
      case 4: softmax_tc_kernel<true, 4><<<grid, block, 0, st>>>(p, u, m, stats, scores, chunks, n_scored); break;
      case 8: softmax_tc_kernel<true, 8><<<grid, block, 0, st>>>(p, u, m, stats, scores, chunks, n_scored); break;
      case 16: softmax_tc_kernel<true, 16><<<grid, block, 0, st>>>(p, u, m, stats, scores, chunks, n_scored); break;
      case 32: softmax_tc_kernel<true, 32><<<grid, block, 0, st>>>(p, u, m, stats, scores, chunks, n_scored); break;
      default: softmax_tc_kernel<true, 0><<<grid, block, 0, st>>>(p, u, m, stats, scores, chunks, n_scored);
    }
    return cudaGetLastError();
  }
  const int chunks = (n_scored + kChunkTokens - 1) / kChunkTokens;
  if (p.meta_dtype == KVSWAP_F16) return launch_stats_and_pool<__half>(p, u, meta, stats, scores, chunks, n_scored, st);
  return launch_stats_and_pool<float>(p, u, meta, stats, scores, chunks, n_scored, st);
}

}  // namespace kvswap
