// K1 on the 5th-generation tensor cores: metadata build K_lr = Flatten(K) A (Sec. 4.2) with
// tcgen05.mma, accumulators in tensor memory and operands staged by TMA.
//
// Covers bf16 K with d in {64, 128} and r in {16, 32, 64} (r = 32, d = 128 are the benchmark
// shapes); project_keys.cu keeps the warp-level path for everything else.
//
// The adapter stays fp32-exact: every entry is split into three bf16 pieces, laid out by a small
// preparation kernel as a K-major [3r x d] operand per KV head, so one instruction shape
// M = 128 tokens, N = 3r (48, 96 or 192) columns, K = 16 channels yields the three partial products
// side by side; the epilogue adds them in fp32.  The tensor core adds into its accumulator with
// truncation, so a chain inside tensor memory covers one KV head (d / 16 instructions); the sum
// over the heads of a joint row is kept in registers with round-to-nearest adds.
//
// CTA = 6 warps, persistent (one per SM):
//   warp 0   producer: per (token tile, KV head) d / 64 TMA boxes of K (128 rows x 64 channels,
//            128-byte swizzle) and as many of the split adapter into a ring of stages;
//   warp 1   issues the MMAs (one thread), owns the tensor-memory allocation (two accumulators);
//   warps 2-5 epilogue: tcgen05.ld of the finished accumulator (one token row per thread), sum of
//            the three pieces, running sum over heads, one rounding into the metadata type.
// Stages and accumulators are handed over through mbarriers; every wait is bounded.
#include <algorithm>
#include <type_traits>

#include "async_copy.cuh"
#include "common.cuh"
#include "tensor_map.cuh"

namespace kvswap {
namespace {

constexpr int kTileM = 128;                                // tokens per tile
constexpr uint32_t kAHalf = kTileM * 128;                  // 128 rows x 128 bytes (64 bf16 channels)
constexpr int kThreadsUmma = 6 * 32;
constexpr size_t kMaxDynamicSmem = 227 * 1024;
constexpr int kMaxStages = 6;

// Sizes for head dimension D and rank R.
template <int D, int R>
struct Cfg {
  static constexpr int kD = D, kR = R;
  static constexpr int kNcols = 3 * R;                                   // accumulator columns: the three pieces side by side
  static constexpr int kHalves = D / 64;                                 // 128-byte-wide boxes per operand row
  static constexpr uint32_t kBHalf = uint32_t(kNcols) * 128;
  static constexpr uint32_t kStageBytes = kHalves * (kAHalf + kBHalf);   // d = 128, r = 32: 57344
  // as many stages as fit beside the 1 KB of alignment slack, six at most (d = 128: 4 at r = 32, 5 at r = 16, 2 at r = 64)
  static constexpr int kFit = int((kMaxDynamicSmem - 1024) / kStageBytes);
  static constexpr int kStages = kFit > kMaxStages ? kMaxStages : kFit;
  static_assert(kStages >= 2, "at least two stages");
  static constexpr uint32_t kAccStride = (kNcols <= 128) ? 128 : 256;    // tensor-memory columns between the two accumulators
  static constexpr uint32_t kTmemCols = 2 * kAccStride;
  static_assert((D == 64 || D == 128) && (R == 16 || R == 32 || R == 64), "shapes of the tcgen05 projection");
  static_assert(kNcols % 16 == 0 && kNcols <= 256, "N of a 128-row tcgen05.mma");
};

// ---- the adapter as three bf16 pieces, [g][piece * r + j][c] (K-major rows of d channels) ----------
__global__ void split_adapter_kernel(const float* __restrict__ proj, __nv_bfloat16* __restrict__ bsplit, int n, int kD,
                                     int kR) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;     // over [g][c][j]
  if (i >= n) return;
  const int kNcols = 3 * kR;
  const int j = i % kR, c = (i / kR) % kD, g = i / (kR * kD);
  const float v = proj[i];
  const __nv_bfloat16 hi = __float2bfloat16_rn(v);
  const float r1 = v - __bfloat162float(hi);
  const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
  const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
  __nv_bfloat16* dst = bsplit + (int64_t(g) * kNcols + j) * kD + c;
  dst[0] = hi; dst[int64_t(kR) * kD] = mid; dst[int64_t(2 * kR) * kD] = lo;
}

// ---- PTX wrappers ------------------------------------------------------------------------------
// K-major operand tile with 128-byte swizzle: rows of 128 bytes, groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_byte_addr) {
  return uint64_t((smem_byte_addr >> 4) & 0x3fffu) | (uint64_t(1) << 16) | (uint64_t(1024 >> 4) << 32) |
         (uint64_t(1) << 46) | (uint64_t(2) << 61);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, float (&v)[32]) { tmem_ld32(taddr, v); }
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, float (&v)[16]) { tmem_ld16(taddr, v); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

struct UmmaShared {
  unsigned long long full[kMaxStages];     // stage loaded (TMA bytes)
  unsigned long long empty[kMaxStages];    // stage consumed (MMA commit)
  unsigned long long acc_full[2];          // accumulator finished (MMA commit)
  unsigned long long acc_empty[2];         // accumulator read out (4 epilogue warps)
  uint32_t tmem_base;
  uint32_t abort;
};

// D = channels multiplied per stage.  PAIR (D = 128 with heads of 64 channels, joint metadata): a stage
// holds two KV heads, one per 64-channel half, so the chain inside tensor memory sums a pair of heads
// and there are half as many stages to hand over.
template <int D, int R, typename META_T, bool PAIR>
__global__ void __launch_bounds__(kThreadsUmma, 1)
project_keys_umma_kernel(Problem p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_b,
                         META_T* __restrict__ meta, int n_begin, int n_end, int tiles_per_row,
                         uint32_t* __restrict__ err) {
  using C = Cfg<D, R>;
  constexpr int kD = D, kR = R, kNcols = C::kNcols, kStages = C::kStages, kHalves = C::kHalves;
  constexpr uint32_t kBHalf = C::kBHalf, kStageBytes = C::kStageBytes, kTmemCols = C::kTmemCols, kAccStride = C::kAccStride;
  constexpr int kChunk = (R < 32) ? R : 32;                // accumulator columns per tensor-memory load
  extern __shared__ unsigned char dyn_raw[];
  const uint32_t stage0 = (smem_addr(dyn_raw) + 1023u) & ~1023u;          // swizzled tiles need 1024-byte alignment
  __shared__ UmmaShared sh;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_addr(&sh.full[s]), 1); mbar_init(smem_addr(&sh.empty[s]), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(smem_addr(&sh.acc_full[a]), 1); mbar_init(smem_addr(&sh.acc_empty[a]), 4); }
    sh.abort = 0;
    mbar_init_fence();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&sh.tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;

  // Work: contiguous range of (sequence, metadata head, token tile) items; a step = (item, KV head).
  const int g_count = PAIR ? p.Hkv / 2 : (p.Hm == 1) ? p.Hkv : 1;      // stages per (token tile) item
  const int64_t items = int64_t(p.B) * p.Hm * tiles_per_row;
  const int64_t first = items * blockIdx.x / gridDim.x, last = items * (blockIdx.x + 1) / gridDim.x;
  const int n_steps = int(last - first) * g_count;

  if (warp == 0) {
    // ================================ producer ==============================================
    if (lane == 0) {
      for (int s = 0; s < n_steps; ++s) {
        const int stage = s % kStages, use = s / kStages;
        if (use > 0 && !mbar_wait(smem_addr(&sh.empty[stage]), uint32_t(use - 1) & 1u)) { sh.abort = 1; if (err) atomicExch(err, kDevTimeoutEmpty); break; }
        const int64_t item = first + s / g_count;
        const int tile = int(item % tiles_per_row), bh = int(item / tiles_per_row);
        const int hm = bh % p.Hm, b = bh / p.Hm;
        const int g = ((p.Hm == 1) ? 0 : hm) + (s % g_count) * (PAIR ? 2 : 1);
        const uint32_t dst = stage0 + uint32_t(stage) * kStageBytes, bar = smem_addr(&sh.full[stage]);
        mbar_arrive_expect_tx(bar, kStageBytes);
        const int n0 = n_begin + tile * kTileM;
#pragma unroll
        for (int h = 0; h < kHalves; ++h) {
          const int c0 = PAIR ? 0 : 64 * h, gh = PAIR ? g + h : g;       // channels and head of this half
          tma_load_4d(dst + uint32_t(h) * kAHalf, &map_k, bar, c0, n0, gh, b);
          tma_load_2d(dst + kHalves * kAHalf + uint32_t(h) * kBHalf, &map_b, bar, c0, gh * kNcols);
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ================================ MMA issuer ============================================
    if (lane == 0) {
      // M = 128, N = 3r, fp32 accumulate, bf16 x bf16, both operands K-major
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(kNcols >> 3) << 17) | (uint32_t(kTileM >> 4) << 24);
      for (int s = 0; s < n_steps; ++s) {
        const int stage = s % kStages, use = s / kStages, buf = s & 1, acc_use = s >> 1;
        if (acc_use > 0 && !mbar_wait(smem_addr(&sh.acc_empty[buf]), uint32_t(acc_use - 1) & 1u)) { sh.abort = 1; if (err) atomicExch(err, kDevTimeoutEmpty); break; }
        if (!mbar_wait(smem_addr(&sh.full[stage]), uint32_t(use) & 1u)) { sh.abort = 1; if (err) atomicExch(err, kDevTimeoutFull); break; }
        tc_fence_after();
        const uint32_t a0 = stage0 + uint32_t(stage) * kStageBytes, b0 = a0 + kHalves * kAHalf;
#pragma unroll
        for (int k = 0; k < kD / 16; ++k) {
          const uint32_t half = k >> 2, koff = uint32_t(k & 3) * 32u;     // 16 channels = 32 bytes inside the swizzle row
          umma_bf16(tmem + uint32_t(buf) * kAccStride, umma_desc(a0 + half * kAHalf + koff), umma_desc(b0 + half * kBHalf + koff),
                    idesc, k > 0 ? 1u : 0u);
        }
        umma_commit(smem_addr(&sh.empty[stage]));         // the stage may be refilled once these MMAs have read it
        umma_commit(smem_addr(&sh.acc_full[buf]));        // ... and the accumulator is complete
      }
    }
    __syncwarp();
  } else {
    // ================================ epilogue ==============================================
    const int quarter = warp & 3;                          // tensor-memory lanes 32 * quarter .. + 31
    const int row = quarter * 32 + lane;                   // token row of the tile owned by this thread
    float acc[kR];
#pragma unroll
    for (int j = 0; j < kR; ++j) acc[j] = 0.f;
    bool ok = true;
    for (int s = 0; s < n_steps && ok; ++s) {
      const int buf = s & 1, acc_use = s >> 1;
      ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.acc_full[buf]), uint32_t(acc_use) & 1u));
      if (!ok) { if (lane == 0) { sh.abort = 1; if (err) atomicExch(err, kDevTimeoutFull); } break; }
      tc_fence_after();
      const uint32_t taddr = tmem + (uint32_t(quarter * 32) << 16) + uint32_t(buf) * kAccStride;
#pragma unroll
      for (int c0 = 0; c0 < kR; c0 += kChunk) {            // the pieces of columns c0 .. c0 + kChunk - 1 sit kR columns apart
        float hi[kChunk], mid[kChunk], lo[kChunk];
        tmem_ld_cols(taddr + c0, hi);
        tmem_ld_cols(taddr + kR + c0, mid);
        tmem_ld_cols(taddr + 2 * kR + c0, lo);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < kChunk; ++j) acc[c0 + j] += (lo[j] + mid[j]) + hi[j];
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_addr(&sh.acc_empty[buf]));
      if ((s + 1) % g_count == 0) {                        // last head of the item: one rounding, one row out
        const int64_t item = first + s / g_count;
        const int tile = int(item % tiles_per_row), bh = int(item / tiles_per_row);
        const int hm = bh % p.Hm, b = bh / p.Hm;
        const int n = n_begin + tile * kTileM + row;
        if (n < n_end) {
          META_T* dst = meta + int64_t(b) * p.meta_sb + int64_t(hm) * p.meta_sh + int64_t(n) * p.meta_sn;
          if constexpr (sizeof(META_T) == 1) {             // E4M3: the row is kR bytes
            const float sc = meta_store_scale(p);
            uint32_t w[kR / 4];
#pragma unroll
            for (int j = 0; j < kR / 4; ++j)
              w[j] = uint32_t(to_e4m3x2(acc[4 * j] * sc, acc[4 * j + 1] * sc)) |
                     (uint32_t(to_e4m3x2(acc[4 * j + 2] * sc, acc[4 * j + 3] * sc)) << 16);
#pragma unroll
            for (int j = 0; j < kR / 16; ++j)
              reinterpret_cast<uint4*>(dst)[j] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            static_assert(kR % 16 == 0, "whole 16-byte vectors per row");
          } else if constexpr (sizeof(META_T) == 2) {
            uint32_t w[kR / 2];
#pragma unroll
            for (int j = 0; j < kR / 2; ++j) {
              const __half2 h = __floats2half2_rn(acc[2 * j], acc[2 * j + 1]);
              w[j] = *reinterpret_cast<const uint32_t*>(&h);
            }
#pragma unroll
            for (int j = 0; j < kR / 8; ++j)
              reinterpret_cast<uint4*>(dst)[j] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
          } else {
#pragma unroll
            for (int j = 0; j < kR / 4; ++j)
              reinterpret_cast<float4*>(dst)[j] = make_float4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
          }
        }
#pragma unroll
        for (int j = 0; j < kR; ++j) acc[j] = 0.f;
      }
    }
  }

  // ---- teardown: every loop above is bounded, so every warp arrives ------------------------------------
  tc_fence_before();
  __syncthreads();
  if (sh.abort && threadIdx.x == 0) {
    // a wait gave up: give copies that may still be in flight a bounded chance to land
    for (int s = 0; s < kStages; ++s) { mbar_wait(smem_addr(&sh.full[s]), 0); mbar_wait(smem_addr(&sh.full[s]), 1); }
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

}  // namespace

static bool umma_shape(const Problem& p) {
  return p.kv_dtype == KVSWAP_BF16 && (p.d == 64 || p.d == 128) && (p.r == 16 || p.r == 32 || p.r == 64);
}

size_t project_keys_umma_scratch_bytes(const Problem& p) {
  if (!umma_shape(p)) return 0;
  return size_t(p.Hkv) * 3 * p.r * p.d * sizeof(__nv_bfloat16);
}

namespace {

template <int D, int R, bool PAIR>
cudaError_t launch_umma(const Problem& p, const CUtensorMap& map_k, const CUtensorMap& map_b, void* meta, int n_begin,
                        int n_end, uint32_t* err, cudaStream_t st) {
  using C = Cfg<D, R>;
  const int tiles_per_row = (n_end - n_begin + kTileM - 1) / kTileM;
  const int64_t items = int64_t(p.B) * p.Hm * tiles_per_row;
  const int ctas = int(std::max<int64_t>(1, std::min<int64_t>(kNumSMs, items)));
  const size_t smem = size_t(C::kStages) * C::kStageBytes + 1024;
  auto go = [&](auto kern, auto* meta_t) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
    kern<<<ctas, kThreadsUmma, smem, st>>>(p, map_k, map_b, meta_t, n_begin, n_end, tiles_per_row, err);
    return cudaGetLastError();
  };
  if constexpr (R == 32) {                                 // 8-bit metadata exists for r = 32 only
    if (p.meta_dtype == KVSWAP_E4M3) return go(project_keys_umma_kernel<D, R, e4m3_t, PAIR>, static_cast<e4m3_t*>(meta));
  }
  if (p.meta_dtype == KVSWAP_E4M3) return cudaErrorInvalidValue;
  if (p.meta_dtype == KVSWAP_F16) return go(project_keys_umma_kernel<D, R, __half, PAIR>, static_cast<__half*>(meta));
  return go(project_keys_umma_kernel<D, R, float, PAIR>, static_cast<float*>(meta));
}

}  // namespace

// Returns true (and sets *result) when this path took the problem.
bool try_launch_project_keys_umma(const Problem& p, const void* K, const float* proj, void* meta, int n_begin,
                                  int n_end, void* scratch, uint32_t* err, cudaStream_t st, cudaError_t* result) {
  if (scratch == nullptr || project_keys_umma_scratch_bytes(p) == 0) return false;
  if (p.meta_dtype == KVSWAP_E4M3 && p.r != 32) return false;
  // Heads of 64 channels are multiplied in pairs where one metadata row sums all heads; alone they
  // leave each stage half as much to do, and at r = 16 the warp-level kernel is the faster one.
  const bool pair = p.d == 64 && p.Hm == 1 && p.Hkv % 2 == 0;
  if (p.d == 64 && !pair && p.r == 16) return false;
  if (p.kv_sn != p.d && (p.kv_sn * 2) % 16 != 0) return false;
  EncodeTiledFn enc = tensor_map_encoder();
  if (enc == nullptr) return false;
  const int ncols = 3 * p.r;
  CUtensorMap map_k, map_b;
  if (!make_rows_tensor_map(&map_k, K, 2, true, p.d, p.N, p.Hkv, p.B, p.kv_sn, p.kv_sh, p.kv_sb, kTileM)) return false;
  {
    const cuuint64_t dims[2] = {cuuint64_t(p.d), cuuint64_t(p.Hkv) * ncols};
    const cuuint64_t strides[1] = {cuuint64_t(p.d) * 2};
    const cuuint32_t box[2] = {64, cuuint32_t(ncols)}, estr[2] = {1, 1};
    if (enc(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, scratch, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  const int n_proj = p.Hkv * p.d * p.r;
  split_adapter_kernel<<<(n_proj + 255) / 256, 256, 0, st>>>(proj, static_cast<__nv_bfloat16*>(scratch), n_proj, p.d, p.r);
  *result = cudaGetLastError();
  if (*result != cudaSuccess) return true;
  auto by_rank = [&](auto d_tag, auto pair_tag) {
    constexpr int D = decltype(d_tag)::value;
    constexpr bool P = decltype(pair_tag)::value;
    return p.r == 16   ? launch_umma<D, 16, P>(p, map_k, map_b, meta, n_begin, n_end, err, st)
           : p.r == 32 ? launch_umma<D, 32, P>(p, map_k, map_b, meta, n_begin, n_end, err, st)
                       : launch_umma<D, 64, P>(p, map_k, map_b, meta, n_begin, n_end, err, st);
  };
  using D128 = std::integral_constant<int, 128>;
  using D64 = std::integral_constant<int, 64>;
  *result = pair         ? by_rank(D128(), std::true_type())
            : p.d == 128 ? by_rank(D128(), std::false_type())
                         : by_rank(D64(), std::false_type());
  return true;
}

}  // namespace kvswap
