// K1: metadata build K_lr = Flatten(K) A (Sec. 4.2) -- the dense contraction of the path.
//
//   project_keys_mma_kernel  bf16 K, r in {16, 32, 64}: tensor cores (mma.sync m16n8k16, fp32
//                            accumulation).  The adapter stays fp32-exact: every entry is split
//                            into three bf16 pieces (8 + 8 + 8 mantissa bits) and each k-step is
//                            issued once per piece, so the products are exact and the only
//                            rounding is the accumulator's and the final one into the metadata
//                            type.  K rows go from global memory straight into A fragments; the
//                            pre-split adapter of every KV head lives in shared memory as ready
//                            B fragments for the whole kernel (persistent CTAs, one per SM).
//   project_keys_kernel      every other case: shared-memory tiled contraction on the fp32
//                            pipes (a CTA owns 64 tokens x r outputs, chunks of 32 channels).
#include <algorithm>

#include "common.cuh"

namespace kvswap {
namespace {

constexpr int kTok = 64;      // tokens per CTA
constexpr int kChunk = 32;    // contraction chunk
constexpr int kThreads = 256;

// Buffers of the layers one launch serves (a flushed group is projected for all layers at once).
constexpr int kMaxProjectLayers = 32;
struct ProjectTable {
  const void* K[kMaxProjectLayers];
  const float* proj[kMaxProjectLayers];
  void* meta[kMaxProjectLayers];
};

template <typename KV_T, typename META_T, int RC>   // RC = ceil(r / 32) output columns per lane
__global__ void __launch_bounds__(kThreads)
project_keys_kernel(Problem p, const ProjectTable tab, int tiles, int n_begin, int n_end) {
  __shared__ float Ks[kTok][kChunk + 1];
  __shared__ float Ps[kChunk][32 * RC];

  const int layer = blockIdx.x / tiles;            // blockIdx.x = layer * tiles + token tile
  const KV_T* __restrict__ K = static_cast<const KV_T*>(tab.K[layer]);
  const float* __restrict__ proj = tab.proj[layer];
  META_T* __restrict__ meta = static_cast<META_T*>(tab.meta[layer]);
  const int b = blockIdx.y;
  const int head_out = blockIdx.z;                 // per-head layout: the KV head; joint: 0
  const int g_first = (p.Hm == 1) ? 0 : head_out;
  const int g_count = (p.Hm == 1) ? p.Hkv : 1;
  const int n0 = n_begin + (blockIdx.x % tiles) * kTok;
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
        if constexpr (sizeof(META_T) == 1)
          Mo[int64_t(n) * p.meta_sn + col].bits = uint8_t(to_e4m3x2(acc[i][j] * meta_store_scale(p), 0.f) & 0xffu);
        else if constexpr (sizeof(META_T) == 2) Mo[int64_t(n) * p.meta_sn + col] = __float2half_rn(acc[i][j]);
        else Mo[int64_t(n) * p.meta_sn + col] = acc[i][j];
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Tensor-core path.
//
// Work item = (sequence b, metadata head hm, tile of 32 tokens); every warp of the grid takes an
// equal contiguous share.  For an item a warp holds two 16-token accumulator tiles [16 x r] and
// walks the contraction index head by head, 32 channels at a time: lane (g = lane / 4,
// t = lane % 4) reads the 16 bytes of channels 32kk + 8t .. +7 of rows g and g + 8 of each tile.
// The contraction index may be permuted as long as both operands agree, so those eight channels
// serve as the lane's A values of two consecutive k-steps, and the B fragments in shared memory
// are built with the same permutation.  The reads of the next half head are in flight while the
// current one is multiplied.
// ------------------------------------------------------------------------------------------
constexpr int kMmaWarps = 12;

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

template <typename META_T, int D, int NT>            // NT = r / 8 output tiles of 8 columns
__global__ void __launch_bounds__(kMmaWarps * 32, 1)
project_keys_mma_kernel(Problem p, const __nv_bfloat16* __restrict__ K, const float* __restrict__ proj,
                        META_T* __restrict__ meta, int n_begin, int n_end, int tiles_per_row) {
  constexpr int KS = D / 16;                         // k-steps per head
  constexpr int KK = D / 32;                         // 32-channel blocks per head
  constexpr int HALF = (KK >= 2) ? 2 : 1;            // blocks multiplied per pipeline step
  constexpr int STEPS_PER_HEAD = KK / HALF;
  extern __shared__ __align__(16) unsigned char dyn[];
  uint2* bfrag = reinterpret_cast<uint2*>(dyn);      // [H_kv][KS][NT][3 pieces][32 lanes]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g8 = lane >> 2, t4 = lane & 3;
  const int r = NT * 8;

  // ---- adapter -> B fragments, three bf16 pieces per entry ------------------------------------------
  for (int i = threadIdx.x; i < p.Hkv * KS * NT * 32; i += kMmaWarps * 32) {
    const int ln = i & 31, nt = (i >> 5) % NT, ks = ((i >> 5) / NT) % KS, g = (i >> 5) / (NT * KS);
    const int t = ln & 3, col = nt * 8 + (ln >> 2);
    const int c0 = 32 * (ks >> 1) + 8 * t + 4 * (ks & 1);      // channels c0 .. c0+3 feed this lane's k slots
    const float* src = proj + (int64_t(g) * D + c0) * r + col;
    float v[4], hi[4], mid[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      v[e] = src[int64_t(e) * r];
      hi[e] = __bfloat162float(__float2bfloat16_rn(v[e]));
      mid[e] = __bfloat162float(__float2bfloat16_rn(v[e] - hi[e]));
      lo[e] = v[e] - hi[e] - mid[e];                 // exact; rounds to bf16 below
    }
    uint2* dst = bfrag + (int64_t(i >> 5) * 3) * 32 + ln;
    dst[0] = make_uint2(pack_bf16(hi[0], hi[1]), pack_bf16(hi[2], hi[3]));
    dst[32] = make_uint2(pack_bf16(mid[0], mid[1]), pack_bf16(mid[2], mid[3]));
    dst[64] = make_uint2(pack_bf16(lo[0], lo[1]), pack_bf16(lo[2], lo[3]));
  }
  __syncthreads();

  const int g_count = (p.Hm == 1) ? p.Hkv : 1;
  const int64_t items = int64_t(p.B) * p.Hm * tiles_per_row;
  const int64_t gw = int64_t(blockIdx.x) * kMmaWarps + warp, n_gw = int64_t(gridDim.x) * kMmaWarps;
  const int64_t first = items * gw / n_gw, last = items * (gw + 1) / n_gw;

  for (int64_t item = first; item < last; ++item) {
    const int tile = int(item % tiles_per_row);
    const int bh = int(item / tiles_per_row);
    const int hm = bh % p.Hm, b = bh / p.Hm;
    const int g_first = (p.Hm == 1) ? 0 : hm;
    const int n0 = n_begin + tile * 32;
    // rows of this lane: tile m, half h -> token n0 + 16 m + 8 h + g8
    const __nv_bfloat16* rowp[2][2];
    bool rowok[2][2];
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int n = n0 + 16 * m + 8 * h + g8;
        rowok[m][h] = n < n_end;
        rowp[m][h] = K + int64_t(b) * p.kv_sb + int64_t(rowok[m][h] ? n : n_begin) * p.kv_sn + 8 * t4;
      }
    float acc[2][NT][4];
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[m][nt][e] = 0.f;

    auto load_step = [&](int step, uint4 (&a)[2][2][HALF]) {   // step = head-in-item * STEPS_PER_HEAD + half
      const int g = g_first + step / STEPS_PER_HEAD;
      const int kk0 = (step % STEPS_PER_HEAD) * HALF;
#pragma unroll
      for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int q = 0; q < HALF; ++q) {
            if (rowok[m][h]) a[m][h][q] = ld_stream16(rowp[m][h] + int64_t(g) * p.kv_sh + 32 * (kk0 + q));
            else a[m][h][q] = make_uint4(0u, 0u, 0u, 0u);
          }
    };
    const int n_steps = g_count * STEPS_PER_HEAD;
    uint4 cur[2][2][HALF], nxt[2][2][HALF];
    load_step(0, cur);
    for (int step = 0; step < n_steps; ++step) {
      if (step + 1 < n_steps) load_step(step + 1, nxt);
      const int g = g_first + step / STEPS_PER_HEAD;
      const int kk0 = (step % STEPS_PER_HEAD) * HALF;
      // The tensor core adds into its accumulator with truncation, which over the ~1500 chained
      // products of a joint row would bias the sum by a visible fraction of an fp16 ulp.  So a
      // chain inside the tensor core covers only one 32-channel block (6 products); the running
      // sums are kept outside, in round-to-nearest fp32 adds.
#pragma unroll
      for (int q = 0; q < HALF; ++q) {
        const uint2* bf = bfrag + (int64_t(g * KS + 2 * (kk0 + q)) * NT * 3) * 32 + lane;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          float tmp[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
          for (int sub = 0; sub < 2; ++sub)
#pragma unroll
            for (int pc = 0; pc < 3; ++pc) {
              const uint2 bb = bf[((sub * NT + nt) * 3 + pc) * 32];
#pragma unroll
              for (int m = 0; m < 2; ++m) {
                const uint4 lo = cur[m][0][q], hi = cur[m][1][q];   // rows g8 and g8 + 8
                mma_bf16_16816(tmp[m], sub ? lo.z : lo.x, sub ? hi.z : hi.x, sub ? lo.w : lo.y, sub ? hi.w : hi.y,
                               bb.x, bb.y);
              }
            }
#pragma unroll
          for (int m = 0; m < 2; ++m)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[m][nt][e] += tmp[m][e];
        }
      }
#pragma unroll
      for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int q = 0; q < HALF; ++q) cur[m][h][q] = nxt[m][h][q];
    }
    // ---- one rounding into the metadata type -------------------------------------------------------
    META_T* Mo = meta + int64_t(b) * p.meta_sb + int64_t(hm) * p.meta_sh;
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (!rowok[m][h]) continue;
        const int n = n0 + 16 * m + 8 * h + g8;
        META_T* row = Mo + int64_t(n) * p.meta_sn + 2 * t4;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const float x = acc[m][nt][2 * h], y = acc[m][nt][2 * h + 1];
          if constexpr (sizeof(META_T) == 2) *reinterpret_cast<__half2*>(row + nt * 8) = __floats2half2_rn(x, y);
          else *reinterpret_cast<float2*>(row + nt * 8) = make_float2(x, y);
        }
      }
  }
}

template <typename META_T, int D, int NT>
cudaError_t launch_mma_one(const Problem& p, const void* K, const float* proj, void* meta, int n_begin, int n_end,
                           cudaStream_t st) {
  const size_t smem = size_t(p.Hkv) * (D / 16) * NT * 3 * 32 * sizeof(uint2);
  auto kern = project_keys_mma_kernel<META_T, D, NT>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
  if (e != cudaSuccess) return e;
  const int tiles_per_row = (n_end - n_begin + 31) / 32;
  const int64_t items = int64_t(p.B) * p.Hm * tiles_per_row;
  const int ctas = int(std::max<int64_t>(1, std::min<int64_t>(kNumSMs, (items + kMmaWarps - 1) / kMmaWarps)));
  kern<<<ctas, kMmaWarps * 32, smem, st>>>(p, static_cast<const __nv_bfloat16*>(K), proj, static_cast<META_T*>(meta),
                                           n_begin, n_end, tiles_per_row);
  return cudaGetLastError();
}

// True (and launched) when the tensor-core path covers the problem.
template <typename META_T>
bool try_launch_mma(const Problem& p, const void* K, const float* proj, void* meta, int n_begin, int n_end,
                    cudaStream_t st, cudaError_t* err) {
  if (p.kv_dtype != KVSWAP_BF16 || (p.r != 16 && p.r != 32 && p.r != 64)) return false;
  const size_t smem = size_t(p.Hkv) * (p.d / 16) * (p.r / 8) * 3 * 32 * sizeof(uint2);
  if (smem > 200 * 1024) return false;
  if (p.d == 128) {
    if (p.r == 16) *err = launch_mma_one<META_T, 128, 2>(p, K, proj, meta, n_begin, n_end, st);
    else if (p.r == 32) *err = launch_mma_one<META_T, 128, 4>(p, K, proj, meta, n_begin, n_end, st);
    else *err = launch_mma_one<META_T, 128, 8>(p, K, proj, meta, n_begin, n_end, st);
  } else {
    if (p.r == 16) *err = launch_mma_one<META_T, 64, 2>(p, K, proj, meta, n_begin, n_end, st);
    else if (p.r == 32) *err = launch_mma_one<META_T, 64, 4>(p, K, proj, meta, n_begin, n_end, st);
    else *err = launch_mma_one<META_T, 64, 8>(p, K, proj, meta, n_begin, n_end, st);
  }
  return true;
}

// A handful of tokens (one flushed group, for every layer): one CTA per (token, sequence, metadata
// head, layer).  Eight slices of the contraction index x 32 output columns; every thread keeps up
// to eight columns (r <= 256); the slices are summed through shared memory in a fixed order.
constexpr int kGroupTokens = 64;              // token ranges up to this length take this kernel

template <typename KV_T, typename META_T>
__global__ void __launch_bounds__(256)
project_group_kernel(Problem p, const ProjectTable tab, int n_begin, int n_tokens) {
  __shared__ float part_sum[8][256];
  const int layer = blockIdx.x / n_tokens, n = n_begin + blockIdx.x % n_tokens;
  const int b = blockIdx.y, head_out = blockIdx.z;
  const KV_T* __restrict__ K = static_cast<const KV_T*>(tab.K[layer]);
  const float* __restrict__ proj = tab.proj[layer];
  META_T* __restrict__ meta = static_cast<META_T*>(tab.meta[layer]);
  const int g_first = (p.Hm == 1) ? 0 : head_out;
  const int g_count = (p.Hm == 1) ? p.Hkv : 1;
  const int lane = threadIdx.x & 31, part = threadIdx.x >> 5;
  float acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.f;
  const int per_part = p.d / 8;                                  // d is 64 or 128
  for (int gi = 0; gi < g_count; ++gi) {
    const int g = g_first + gi;
    const KV_T* row = K + int64_t(b) * p.kv_sb + int64_t(g) * p.kv_sh + int64_t(n) * p.kv_sn;
    const float* Pg = proj + int64_t(g) * p.d * p.r;
    for (int c = part * per_part; c < (part + 1) * per_part; ++c) {
      const float k = float(row[c]);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int col = lane + 32 * j;
        if (col < p.r) acc[j] = fmaf(k, Pg[int64_t(c) * p.r + col], acc[j]);
      }
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) part_sum[part][lane + 32 * j] = acc[j];
  __syncthreads();
  for (int col = threadIdx.x; col < p.r; col += blockDim.x) {
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) s += part_sum[k][col];
    META_T* out = meta + int64_t(b) * p.meta_sb + int64_t(head_out) * p.meta_sh + int64_t(n) * p.meta_sn + col;
    if constexpr (sizeof(META_T) == 1) out->bits = uint8_t(to_e4m3x2(s * meta_store_scale(p), 0.f) & 0xffu);
    else if constexpr (sizeof(META_T) == 2) *out = __float2half_rn(s);
    else *out = s;
  }
}

template <typename KV_T, typename META_T>
cudaError_t dispatch_rc(const Problem& p, const ProjectTable& tab, int n_layers, int n_begin, int n_end,
                        cudaStream_t st) {
  if (n_end - n_begin <= kGroupTokens) {
    const int n_tokens = n_end - n_begin;
    project_group_kernel<KV_T, META_T><<<dim3(n_tokens * n_layers, p.B, p.Hm), 256, 0, st>>>(p, tab, n_begin, n_tokens);
    return cudaGetLastError();
  }
  const int tiles = (n_end - n_begin + kTok - 1) / kTok;
  dim3 grid(tiles * n_layers, p.B, p.Hm);
  const int rc = (p.r + 31) / 32;
  if (rc <= 1) project_keys_kernel<KV_T, META_T, 1><<<grid, kThreads, 0, st>>>(p, tab, tiles, n_begin, n_end);
  else if (rc <= 2) project_keys_kernel<KV_T, META_T, 2><<<grid, kThreads, 0, st>>>(p, tab, tiles, n_begin, n_end);
  else if (rc <= 4) project_keys_kernel<KV_T, META_T, 4><<<grid, kThreads, 0, st>>>(p, tab, tiles, n_begin, n_end);
  else project_keys_kernel<KV_T, META_T, 8><<<grid, kThreads, 0, st>>>(p, tab, tiles, n_begin, n_end);
  return cudaGetLastError();
}

template <typename KV_T>
cudaError_t dispatch_rc_meta(const Problem& p, const ProjectTable& tab, int n_layers, int n_begin, int n_end,
                             cudaStream_t st) {
  if (p.meta_dtype == KVSWAP_F16) return dispatch_rc<KV_T, __half>(p, tab, n_layers, n_begin, n_end, st);
  if (p.meta_dtype == KVSWAP_E4M3) return dispatch_rc<KV_T, e4m3_t>(p, tab, n_layers, n_begin, n_end, st);
  return dispatch_rc<KV_T, float>(p, tab, n_layers, n_begin, n_end, st);
}

cudaError_t dispatch_table(const Problem& p, const ProjectTable& tab, int n_layers, int n_begin, int n_end,
                           cudaStream_t st) {
  switch (p.kv_dtype) {
    case KVSWAP_F32: return dispatch_rc_meta<float>(p, tab, n_layers, n_begin, n_end, st);
    case KVSWAP_BF16: return dispatch_rc_meta<__nv_bfloat16>(p, tab, n_layers, n_begin, n_end, st);
    default: return dispatch_rc_meta<__half>(p, tab, n_layers, n_begin, n_end, st);
  }
}

constexpr int kMinTensorCoreTokens = 256;

template <typename KV_T>
cudaError_t dispatch_meta(const Problem& p, const void* K, const float* proj, void* meta, int n_begin, int n_end,
                          bool tensor_cores, cudaStream_t st) {
  cudaError_t e = cudaSuccess;
  if (tensor_cores && p.meta_dtype != KVSWAP_E4M3) {      // (8-bit metadata: tcgen05 path or the fp32 kernel)
    if (p.meta_dtype == KVSWAP_F16) {
      if (try_launch_mma<__half>(p, K, proj, meta, n_begin, n_end, st, &e)) return e;
    } else if (try_launch_mma<float>(p, K, proj, meta, n_begin, n_end, st, &e)) {
      return e;
    }
  }
  ProjectTable tab = {};
  tab.K[0] = K; tab.proj[0] = proj; tab.meta[0] = meta;
  return dispatch_rc_meta<KV_T>(p, tab, 1, n_begin, n_end, st);
}

}  // namespace

cudaError_t launch_project_keys(const Problem& p, const void* K, const float* proj, void* meta, int n_begin,
                                int n_end, void* scratch, uint32_t* err, cudaStream_t st) {
  cudaError_t e = cudaSuccess;
  // A short token range (a flushed group during decoding) is not worth the tensor-core paths'
  // set-up (adapter split, tensor maps, shared-memory-resident operand fragments).
  const bool tensor_cores = n_end - n_begin >= kMinTensorCoreTokens;
  if (tensor_cores && try_launch_project_keys_umma(p, K, proj, meta, n_begin, n_end, scratch, err, st, &e)) return e;
  switch (p.kv_dtype) {
    case KVSWAP_F32: return dispatch_meta<float>(p, K, proj, meta, n_begin, n_end, tensor_cores, st);
    case KVSWAP_BF16: return dispatch_meta<__nv_bfloat16>(p, K, proj, meta, n_begin, n_end, tensor_cores, st);
    default: return dispatch_meta<__half>(p, K, proj, meta, n_begin, n_end, tensor_cores, st);
  }
}

// The same token range of several layers (a group flushed during decoding) on the fp32 path, up
// to kMaxProjectLayers layers per launch.
cudaError_t launch_project_keys_layers(const Problem& p, const void* const* K, const float* const* proj,
                                       void* const* meta, int n_layers, int n_begin, int n_end, cudaStream_t st) {
  for (int l0 = 0; l0 < n_layers; l0 += kMaxProjectLayers) {
    const int count = std::min(kMaxProjectLayers, n_layers - l0);
    ProjectTable tab = {};
    for (int l = 0; l < count; ++l) { tab.K[l] = K[l0 + l]; tab.proj[l] = proj[l0 + l]; tab.meta[l] = meta[l0 + l]; }
    cudaError_t e = dispatch_table(p, tab, count, n_begin, n_end, st);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace kvswap
