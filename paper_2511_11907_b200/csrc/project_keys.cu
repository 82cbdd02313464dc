// K1: metadata build K_lr = Flatten(K) A (Sec. 4.2).
//
// Generic shared-memory tiled contraction on the fp32 pipes: every (kv, meta) dtype pair, any
// supported d and r.  A CTA owns 64 tokens x r outputs and walks the contraction index
// (g, c) in chunks of 32 channels.
#include "common.cuh"

namespace kvswap {
namespace {

constexpr int kTok = 64;      // tokens per CTA
constexpr int kChunk = 32;    // contraction chunk
constexpr int kThreads = 256;

template <typename KV_T, typename META_T, int RC>   // RC = ceil(r / 32) output columns per lane
__global__ void __launch_bounds__(kThreads)
project_keys_kernel(Problem p, const KV_T* __restrict__ K, const float* __restrict__ proj,
                    META_T* __restrict__ meta, int n_begin, int n_end) {
  __shared__ float Ks[kTok][kChunk + 1];
  __shared__ float Ps[kChunk][32 * RC];

  const int b = blockIdx.y;
  const int head_out = blockIdx.z;                 // per-head layout: the KV head; joint: 0
  const int g_first = (p.Hm == 1) ? 0 : head_out;
  const int g_count = (p.Hm == 1) ? p.Hkv : 1;
  const int n0 = n_begin + blockIdx.x * kTok;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  float acc[8][RC];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < RC; ++j) acc[i][j] = 0.f;

  constexpr int kPer = Elt<KV_T>::kPer16B;
  for (int gi = 0; gi < g_count; ++gi) {
    const int g = g_first + gi;
    const KV_T* Kg = K + int64_t(b) * p.kv_sb + int64_t(g) * p.kv_sh;
    const float* Pg = proj + int64_t(g) * p.d * p.r;
    for (int c0 = 0; c0 < p.d; c0 += kChunk) {
      // K tile: 64 x 32 elements, 16-byte vector loads.
      for (int v = threadIdx.x; v < kTok * kChunk / kPer; v += kThreads) {
        const int row = v / (kChunk / kPer), part = v % (kChunk / kPer);
        const int n = n0 + row;
        float f[kPer];
        if (n < n_end) {
          uint4 raw = ld_stream16(Kg + int64_t(n) * p.kv_sn + c0 + part * kPer);
          widen16B(raw, f, KV_T());
        } else {
#pragma unroll
          for (int e = 0; e < kPer; ++e) f[e] = 0.f;
        }
#pragma unroll
        for (int e = 0; e < kPer; ++e) Ks[row][part * kPer + e] = f[e];
      }
      // proj tile: 32 x r (zero padded to 32*RC columns).
      for (int v = threadIdx.x; v < kChunk * 32 * RC; v += kThreads) {
        const int c = v / (32 * RC), j = v % (32 * RC);
        Ps[c][j] = (j < p.r) ? Pg[int64_t(c0 + c) * p.r + j] : 0.f;
      }
      __syncthreads();
#pragma unroll 8
      for (int c = 0; c < kChunk; ++c) {
        float bcol[RC];
#pragma unroll
        for (int j = 0; j < RC; ++j) bcol[j] = Ps[c][lane + 32 * j];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float a = Ks[warp * 8 + i][c];
#pragma unroll
          for (int j = 0; j < RC; ++j) acc[i][j] = fmaf(a, bcol[j], acc[i][j]);
        }
      }
      __syncthreads();
    }
  }

  META_T* Mo = meta + int64_t(b) * p.meta_sb + int64_t(head_out) * p.meta_sh;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int n = n0 + warp * 8 + i;
    if (n >= n_end) continue;
#pragma unroll
    for (int j = 0; j < RC; ++j) {
      const int col = lane + 32 * j;
      if (col < p.r) {
        if constexpr (sizeof(META_T) == 2) Mo[int64_t(n) * p.meta_sn + col] = __float2half_rn(acc[i][j]);
        else Mo[int64_t(n) * p.meta_sn + col] = acc[i][j];
      }
    }
  }
}

template <typename KV_T, typename META_T>
cudaError_t dispatch_rc(const Problem& p, const void* K, const float* proj, void* meta, int n_begin, int n_end,
                        cudaStream_t st) {
  dim3 grid((n_end - n_begin + kTok - 1) / kTok, p.B, p.Hm);
  const KV_T* Kt = static_cast<const KV_T*>(K);
  META_T* Mt = static_cast<META_T*>(meta);
  const int rc = (p.r + 31) / 32;
  if (rc <= 1) project_keys_kernel<KV_T, META_T, 1><<<grid, kThreads, 0, st>>>(p, Kt, proj, Mt, n_begin, n_end);
  else if (rc <= 2) project_keys_kernel<KV_T, META_T, 2><<<grid, kThreads, 0, st>>>(p, Kt, proj, Mt, n_begin, n_end);
  else if (rc <= 4) project_keys_kernel<KV_T, META_T, 4><<<grid, kThreads, 0, st>>>(p, Kt, proj, Mt, n_begin, n_end);
  else project_keys_kernel<KV_T, META_T, 8><<<grid, kThreads, 0, st>>>(p, Kt, proj, Mt, n_begin, n_end);
  return cudaGetLastError();
}

template <typename KV_T>
cudaError_t dispatch_meta(const Problem& p, const void* K, const float* proj, void* meta, int n_begin, int n_end,
                          cudaStream_t st) {
  if (p.meta_dtype == KVSWAP_F16) return dispatch_rc<KV_T, __half>(p, K, proj, meta, n_begin, n_end, st);
  return dispatch_rc<KV_T, float>(p, K, proj, meta, n_begin, n_end, st);
}

}  // namespace

cudaError_t launch_project_keys(const Problem& p, const void* K, const float* proj, void* meta, int n_begin,
                                int n_end, cudaStream_t st) {
  switch (p.kv_dtype) {
    case KVSWAP_F32: return dispatch_meta<float>(p, K, proj, meta, n_begin, n_end, st);
    case KVSWAP_BF16: return dispatch_meta<__nv_bfloat16>(p, K, proj, meta, n_begin, n_end, st);
    default: return dispatch_meta<__half>(p, K, proj, meta, n_begin, n_end, st);
  }
}

}  // namespace kvswap
