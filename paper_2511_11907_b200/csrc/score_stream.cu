// K2, streaming tensor-core scorer: low-rank query (Eq. 1), token scoring, head aggregation and
// group ReduceMax (Sec. 4.3) for metadata rows of rank 32 that are dense in memory -- fp16 rows of
// 64 bytes, or 8-bit E4M3 rows of 32 bytes whose values convert to fp16 exactly and whose common
// power-of-two scale is applied to the finished score -- G a power of two <= 32 and one metadata
// term per score.
//
// One persistent CTA per SM, 16 warps.  Work item = (sequence b, metadata head hm, block of 8
// scopes, 4 KB tile of 64 fp16 or 128 E4M3 rows); items are numbered with the tile fastest, a "row set" is the items of
// one (b, hm, scope block).  Every warp takes an equal contiguous share of tiles and pulls them
// into its own ring of shared-memory stages with bulk asynchronous copies (cp.async.bulk +
// mbarrier, bounded waits), kDepth tiles in flight per warp; the first tiles are requested before
// the dependency wait, since nothing the library runs during decoding writes metadata.
//
// With joint metadata one row feeds up to 8 scores (the per-KV-head scopes): an [rows x 32].[32 x 8]
// contraction at 8 FLOP per byte, which the fp32 pipes cannot sustain at HBM rate; it runs on the
// tensor cores (mma.sync m16n8k16, fp16 inputs, fp32 accumulation).  The summed low-rank queries
// stay fp32-exact: each is scaled by a power of two and split into an fp16 head and an fp16
// remainder, the head in rows 0..7 and the remainder in rows 8..15 of the row operand, so one
// instruction per k-step yields both partial products and the only rounding is the accumulator's.
//
// Operand layout.  A 16-byte shared-memory read gives lane (g = lane / 4, t = lane % 4) the rank
// entries 8t..8t+7 of row g of an 8-row block.  The contraction index may be permuted freely as
// long as both operands agree, so k-step j takes entries 8t+4j..8t+4j+3 as the four values the
// lane owes for token g (the column operand, 8 tokens wide), and the row operand holds the same
// entries of the query of scope g.  The accumulator then holds, in lane (g, t), the scores of
// scope g for tokens 2t and 2t+1: a group's maximum is a max over two registers and at most two
// shuffles, and a finished group score leaves the registers at once.
//
// The CTA computes the summed low-rank queries of its row sets itself where it can (`fused`):
//     u[b, row, :] = sum over the KV heads g of the row's scope of (sum_{h: g(h) = g} q[b, h, :]) A_g
// which removes the separate low-rank query kernel and its launch dependency from the call.
//
// While it scores, the CTA counts the leading 12 bits of every group score's key in a
// shared-memory histogram (16-bit counters, 8 columns = the scopes of its first row set) and adds
// the non-zero counters to the global histograms at the end, four counters per 64-bit atomic (the
// global histograms have the same packed layout; a row has at most 65535 groups on this path).
// Scores of row sets that do not fit the 8 columns are counted in global memory directly.  The
// global histograms are zero on entry and left zero by the TopK kernel that starts from them
// (topk_select.cu; kvswap_workspace_init clears them once).
#include <algorithm>
#include <cmath>
#include <type_traits>

#include "async_copy.cuh"
#include "common.cuh"
#include "lowrank_query.cuh"
#include "topk_keys.cuh"

namespace kvswap {
namespace {

constexpr uint32_t kFull = 0xffffffffu;
constexpr int kTileBytes = 4096;                          // one stage: 64 fp16 rows of 64 bytes, or 128 E4M3 rows of 32 bytes
                                                          // (the hand-over of a stage costs the same whatever its size: 4 KB x 2
                                                          // stages measured 1.3 us per layer faster than 2 KB x 4 at config 5)
template <bool FP8> struct Tile {
  static constexpr int kRowBytes = FP8 ? 32 : 64;
  static constexpr int kRows = kTileBytes / kRowBytes;
};
constexpr int kWarps = kQueryWarps;                       // 16
constexpr int kThreads = kWarps * 32;
constexpr int kDepth = 2;
constexpr int kCols = kQueryCols;                         // scores per metadata row and instruction
constexpr int kHistWords = kCols * kKeyTopBins / 2;       // two 16-bit counters per word
constexpr int kMaxSets = 4;                               // row sets one CTA may touch when it builds the queries itself
constexpr int kMaxTilesPerCta = 65535 / 128;               // bound that keeps a 16-bit counter from overflowing (128 rows, G = 1)

struct Smem {
  unsigned char tiles[kWarps * kDepth * kTileBytes];      // 128 KB of stages
  uint32_t hist[kHistWords];                              // 64 KB
  unsigned long long full[kWarps * kDepth];
  float qsum[kQuerySumFloats];                            // scratch of build_queries
  float upart[kQueryPartFloats];
  float urow[kMaxSets][kCols * 32];                       // summed low-rank queries per row set of the CTA
};

struct StreamArgs {
  const void* q;            // fused: [B, H_q, d] q_dtype
  const float* proj;        // fused: [H_kv, d, r]
  const float* uq;          // not fused: [B, Su, r] from the low-rank query kernel
  const unsigned char* meta;
  float* scores;
  uint32_t* top_hist;       // NULL, or [B * S, 4096] 16-bit counters, two per word
  int tiles_per_row, n_sub, n_rests;
  int vset_items, ctas_per_vset;   // work split: virtual sets of vset_items items, each shared by ctas_per_vset CTAs
  int base, rem;            // tiles per warp within a virtual set: base, +1 for the first rem warps
  float meta_scale;         // 2^meta_exp (1 unless the metadata is 8-bit)
  uint32_t* err;
};

__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_half2(__half lo, __half hi) {
  return uint32_t(__half_as_ushort(lo)) | (uint32_t(__half_as_ushort(hi)) << 16);
}

// FP8: the metadata is E4M3 (rows of 32 bytes, 64 per tile); every value converts to fp16 exactly, so
// the product below is the same with twice the rows per byte.
template <int GS, bool FUSED, bool FP8>              // GS = log2(G), 0..5
__global__ void __launch_bounds__(kThreads, 1)
score_stream_kernel(Problem p, StreamArgs a) {
  constexpr int g_shift = GS;
  constexpr int kTileRows = Tile<FP8>::kRows;
  constexpr int kRowBytes = Tile<FP8>::kRowBytes;
  extern __shared__ __align__(128) unsigned char dyn[];
  Smem* sm = reinterpret_cast<Smem*>(dyn);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rq = lane >> 2, qt = lane & 3;
  if (lane == 0) {                                  // every warp sets up its own stages
    for (int s = 0; s < kDepth; ++s) mbar_init(smem_addr(&sm->full[warp * kDepth + s]), 1);
    mbar_init_fence();
  }
  if (a.top_hist != nullptr) {
    uint4* H = reinterpret_cast<uint4*>(sm->hist);
    for (int i = threadIdx.x; i < kHistWords / 4; i += kThreads) H[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  __syncwarp();

  // ---- this warp's contiguous share of the work items -----------------------------------------------------
  const int rows_total = p.NG * p.G;
  const int hm_count = (p.Hm == 1) ? 1 : p.Hkv;
  const int vset = blockIdx.x / a.ctas_per_vset, cta_in = blockIdx.x - vset * a.ctas_per_vset;
  auto share_first = [&](int w) { return vset * a.vset_items + w * a.base + min(w, a.rem); };
  const int wi = cta_in * kWarps + warp;
  const int first = share_first(wi);
  const int my_tiles = a.base + (wi < a.rem ? 1 : 0);
  const int cta_first = share_first(cta_in * kWarps), cta_last = share_first((cta_in + 1) * kWarps);   // [first, last) of the CTA
  const int rest0 = cta_first / a.tiles_per_row;                                  // the CTA's first row set
  const int n_sets = (cta_last > cta_first) ? (cta_last - 1) / a.tiles_per_row - rest0 + 1 : 0;
  const int ns_cols = (p.Hm == 1) ? min(kCols, p.S) : 1;                          // histogram columns per row set
  int f_tile = first % a.tiles_per_row, f_rest = first / a.tiles_per_row;         // next item to request
  int c_tile = f_tile, c_rest = f_rest;                                           // next item to consume

  const uint32_t ring = smem_addr(sm->tiles) + uint32_t(warp) * kDepth * kTileBytes;
  const unsigned char* f_base = nullptr;            // metadata of the fill cursor's (sequence, head)
  int f_base_rest = -1;
  auto fill = [&](int stage) {
    if (lane == 0) {
      if (f_rest != f_base_rest) {                  // divisions only when the cursor enters a new row set
        f_base_rest = f_rest;
        const int bh = f_rest / a.n_sub;
        f_base = a.meta + (int64_t(bh / hm_count) * p.meta_sb + int64_t(bh % hm_count) * p.meta_sh) * (FP8 ? 1 : 2);
      }
      const int rows = min(kTileRows, rows_total - f_tile * kTileRows);
      const uint32_t bar = smem_addr(&sm->full[warp * kDepth + stage]);
      mbar_arrive_expect_tx(bar, uint32_t(rows) * kRowBytes);
      bulk_g2s(ring + uint32_t(stage) * kTileBytes, f_base + int64_t(f_tile) * kTileRows * kRowBytes,
               uint32_t(rows) * kRowBytes, bar);
    }
    if (++f_tile == a.tiles_per_row) { f_tile = 0; ++f_rest; }
  };
  // The metadata is never written by a kernel that runs during decoding: request the first tiles now.
  for (int k = 0; k < kDepth && k < my_tiles; ++k) fill(k);

  // ---- dependency wait and the summed low-rank queries ---------------------------------------------------
  // Without KVSWAP_INPUTS_SETTLED the query may be the previous kernel's output: wait first.  With it,
  // only this kernel's writes (scores and histograms, which the previous call's TopK may still read)
  // have to wait, so the queries are built while that kernel finishes.
  const bool settled = FUSED && (p.flags & KVSWAP_INPUTS_SETTLED) != 0;
  if (!settled) pdl_wait();
  if constexpr (FUSED) {
    for (int s = 0; s < n_sets; ++s) build_queries<0>(p, a.q, a.proj, row_set(p, rest0 + s, a.n_sub), sm->qsum, sm->upart, sm->urow[s]);
  }
  if (settled) pdl_wait();
  pdl_trigger();
  if constexpr (!FUSED) __syncthreads();             // the histogram is cleared (the fused path has synchronised)

  uint32_t ahl[2][2], alh[2][2];                    // row-operand fragments: [k-step][entry pair], head (rows 0..7) / remainder (rows 8..15)
  float inv = 1.f;                                  // undoes the scaling of this lane's scope
  int cur_rest = -1;
  float* my_row = a.scores;                         // scores row of this lane's scope (scope rq of the current block)
  uint32_t* my_hist = nullptr;                      // its global histogram
  int my_col = -1;                                  // its column of the shared-memory histogram, or -1
  bool scope_ok = false;                            // the lane's scope exists
  float run = -INFINITY;                            // running maximum of a 16- or 32-row group
  int stage = 0;
  uint32_t phase = 0;
  bool timed_out = false;
  // A finished group score leaves the registers at once: to the score row and, as one count, to the
  // histogram of its key's leading digit.
  auto publish = [&](float* dst, float x) {
    x += 0.f;                                       // -0 becomes +0: the TopK that follows relies on it
    *dst = x;
    if (a.top_hist != nullptr) {
      const uint32_t bin = score_key_top(x);
      if (my_col >= 0) {
        atomicAdd(&sm->hist[(my_col * kKeyTopBins + int(bin)) >> 1], 1u << ((bin & 1u) << 4));
      } else {
        atomicAdd(my_hist + (bin >> 1), 1u << ((bin & 1u) << 4));
      }
    }
  };
  for (int k = 0; k < my_tiles; ++k) {
    const int tile = c_tile;
    if (c_rest != cur_rest) {                       // new row set: rebuild the row operand
      cur_rest = c_rest;
      const RowSet rs = row_set(p, c_rest, a.n_sub);
      float u[8];
      if constexpr (FUSED) {
        const float4* ur = reinterpret_cast<const float4*>(sm->urow[c_rest - rest0] + rq * 32 + qt * 8);
        const float4 x = ur[0], y = ur[1];
        u[0] = x.x; u[1] = x.y; u[2] = x.z; u[3] = x.w; u[4] = y.x; u[5] = y.y; u[6] = y.z; u[7] = y.w;
      } else {
        // this lane supplies the query of column rq: scope sub * 8 + rq (joint) or head hm (column 0 only)
        const int urow = (p.Hm == 1) ? rs.sub * kCols + rq : rs.hm;
        const bool have = (p.Hm == 1) ? (urow < p.S) : (rq == 0);
        if (have) {
          const float4* ur = reinterpret_cast<const float4*>(a.uq + (int64_t(rs.b) * p.Su + urow) * p.r + qt * 8);
          const float4 x = ur[0], y = ur[1];
          u[0] = x.x; u[1] = x.y; u[2] = x.z; u[3] = x.w; u[4] = y.x; u[5] = y.y; u[6] = y.z; u[7] = y.w;
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) u[i] = 0.f;
        }
      }
      float mx = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) mx = fmaxf(mx, fabsf(u[i]));
      mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 2));
      // power of two that brings the largest entry into [2^14, 2^15)
      int sh = 0;
      if (mx > 0.f && mx < INFINITY) sh = min(120, max(-113, 14 - (int((__float_as_uint(mx) >> 23) & 0xffu) - 127)));
      const float scale = __uint_as_float(uint32_t(sh + 127) << 23);
      inv = __uint_as_float(uint32_t(127 - sh) << 23) * a.meta_scale;     // also undoes the 8-bit cache's power of two
      __half hi[8], lo[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float us = u[i] * scale;
        hi[i] = __float2half_rn(us);
        lo[i] = __float2half_rn(us - __half2float(hi[i]));
      }
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        ahl[j][0] = pack_half2(hi[4 * j], hi[4 * j + 1]); ahl[j][1] = pack_half2(hi[4 * j + 2], hi[4 * j + 3]);
        alh[j][0] = pack_half2(lo[4 * j], lo[4 * j + 1]); alh[j][1] = pack_half2(lo[4 * j + 2], lo[4 * j + 3]);
      }
      const int s0 = (p.Hm == 1) ? rs.sub * kCols : rs.hm;
      const int ns_cur = (p.Hm == 1) ? min(kCols, p.S - s0) : 1;
      scope_ok = rq < ns_cur;
      const int64_t prob = int64_t(rs.b) * p.S + s0 + (scope_ok ? rq : 0);
      my_row = a.scores + prob * p.score_pitch;
      if (a.top_hist != nullptr) {
        my_hist = a.top_hist + prob * (kKeyTopBins / 2);
        const int col = (c_rest - rest0) * ns_cols + rq;
        my_col = (scope_ok && col < kCols) ? col : -1;
      }
    }
    if (++c_tile == a.tiles_per_row) { c_tile = 0; ++c_rest; }
    if (!__all_sync(kFull, mbar_wait(smem_addr(&sm->full[warp * kDepth + stage]), phase))) { timed_out = true; break; }
    const int rows = min(kTileRows, rows_total - tile * kTileRows);   // a multiple of G: groups never straddle tiles
    const int ngt = rows >> g_shift;                // groups in this tile
    const uint32_t base = ring + uint32_t(stage) * kTileBytes + uint32_t(lane) * (kRowBytes / 4);
    float* dst = my_row + ((tile * kTileRows) >> g_shift);           // first group of the tile in this lane's row
    float mine[kTileRows / 32] = {};                // G = 8: the groups of reads qt, qt + 4, .. are this lane's to publish
#pragma unroll
    for (int it = 0; it < kTileRows / 8; ++it) {
      if (it * 8 < rows) {
        uint32_t w[4];                              // entries 8t .. 8t+7 of row g as fp16 pairs
        if constexpr (FP8) {
          uint32_t b8[2];
          asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(b8[0]), "=r"(b8[1]) : "r"(base + uint32_t(it) * 8u * kRowBytes));
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint16_t pair = uint16_t(b8[i >> 1] >> ((i & 1) * 16));
            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(w[i]) : "h"(pair));
          }
        } else {
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3])
                       : "r"(base + uint32_t(it) * 8u * kRowBytes));
        }
        float d[4] = {0.f, 0.f, 0.f, 0.f};          // d[0], d[1]: head products of tokens 2t, 2t+1; d[2], d[3]: remainder products
#pragma unroll
        for (int j = 0; j < 2; ++j) mma16816(d, ahl[j][0], alh[j][0], ahl[j][1], alh[j][1], w[2 * j], w[2 * j + 1]);
        const float x0 = d[0] + d[2], x1 = d[1] + d[3];
        if constexpr (GS == 0) {                                   // tokens 2t and 2t+1 of this read are groups
          if (scope_ok && it * 8 + 2 * qt < rows) publish(dst + it * 8 + 2 * qt, x0 * inv);
          if (scope_ok && it * 8 + 2 * qt + 1 < rows) publish(dst + it * 8 + 2 * qt + 1, x1 * inv);
        } else {
          float m = fmaxf(x0, x1);
          if constexpr (GS >= 2) m = fmaxf(m, __shfl_xor_sync(kFull, m, 1));
          if constexpr (GS >= 3) m = fmaxf(m, __shfl_xor_sync(kFull, m, 2));
          // (a ragged last tile holds a whole number of groups, but not of 8-row reads when G < 8)
          if constexpr (GS == 1) { if (scope_ok && it * 4 + qt < ngt) publish(dst + it * 4 + qt, m * inv); }
          else if constexpr (GS == 2) {
            if (scope_ok && (qt & 1) == 0 && it * 2 + (qt >> 1) < ngt) publish(dst + it * 2 + (qt >> 1), m * inv);
          }
          else if constexpr (GS == 3) { if (qt == (it & 3)) mine[it >> 2] = m; }
          else {                                                 // G = 16 or 32: 2 or 4 reads per group
            run = fmaxf(run, m);
            if (((it + 1) & ((1 << (GS - 3)) - 1)) == 0) {
              const int gi = it >> (GS - 3);
              if (scope_ok && qt == (gi & 3)) publish(dst + gi, run * inv);
              run = -INFINITY;
            }
          }
        }
      }
    }
    if constexpr (GS == 3) {
#pragma unroll
      for (int h = 0; h < kTileRows / 32; ++h)
        if (scope_ok && (4 * h + qt) * 8 < rows) publish(dst + 4 * h + qt, mine[h] * inv);
    }
    __syncwarp();                                   // every lane has read the stage
    if (k + kDepth < my_tiles) fill(stage);
    if (++stage == kDepth) { stage = 0; phase ^= 1u; }
  }
  if (timed_out) {
    if (lane == 0 && a.err) atomicExch(a.err, kDevTimeoutFull);
    for (int s = 0; s < kDepth; ++s) {              // bounded chance for copies in flight to land
      mbar_wait(smem_addr(&sm->full[warp * kDepth + s]), 0);
      mbar_wait(smem_addr(&sm->full[warp * kDepth + s]), 1);
    }
  }

  // ---- the CTA's counts join the global histograms --------------------------------------------------------
  if (a.top_hist != nullptr) {
    __syncthreads();
    for (int i = threadIdx.x; i < kHistWords / 4; i += kThreads) {
      const uint4 v = reinterpret_cast<const uint4*>(sm->hist)[i];
      if ((v.x | v.y | v.z | v.w) == 0u) continue;
      const int col = (i * 8) / kKeyTopBins;                                      // 8 counters per vector
      const int rest = rest0 + col / ns_cols, in_set = col % ns_cols;
      if (rest >= a.n_rests) continue;
      const RowSet rs = row_set(p, rest, a.n_sub);
      const int s = (p.Hm == 1) ? rs.sub * kCols + in_set : rs.hm;
      if (s >= p.S) continue;
      unsigned long long* H = reinterpret_cast<unsigned long long*>(
          a.top_hist + (int64_t(rs.b) * p.S + s) * (kKeyTopBins / 2) + ((i * 4) % (kKeyTopBins / 2)));
      const unsigned long long lo = (unsigned long long)v.x | ((unsigned long long)v.y << 32);
      const unsigned long long hi = (unsigned long long)v.z | ((unsigned long long)v.w << 32);
      if (lo != 0ull) atomicAdd(H, lo);
      if (hi != 0ull) atomicAdd(H + 1, hi);
    }
  }
}

struct Plan {
  int g_shift;
  int tiles_per_row, n_sub, n_rests;
  int ctas, vset_items, ctas_per_vset, base, rem;
  bool fused;
  bool counts;
  bool fp8;
};

// Launch geometry of the streaming scorer for `p`; false when the shape does not take it.
bool plan(const Problem& p, Plan* pl) {
  const bool fp8 = p.meta_dtype == KVSWAP_E4M3;
  if ((p.meta_dtype != KVSWAP_F16 && !fp8) || p.NG < 1) return false;
  int g_shift = -1;
  for (int s = 0; s <= 5; ++s) if ((1 << s) == p.G) g_shift = s;
  const bool one_term = (p.Hm == 1) || (p.scope == KVSWAP_SCOPE_KV_HEAD);
  const int row_bytes = fp8 ? 32 : 64, tile_rows = kTileBytes / row_bytes;
  if (!one_term || g_shift < 0 || p.r * (fp8 ? 1 : 2) != row_bytes || p.meta_sn != p.r) return false;
  const int64_t rows_total = int64_t(p.NG) * p.G;
  const int64_t tiles_per_row = (rows_total + tile_rows - 1) / tile_rows;
  const int n_sub = (p.Hm == 1) ? (p.S + kCols - 1) / kCols : 1;
  const int64_t n_rests = int64_t(p.B) * ((p.Hm == 1) ? 1 : p.Hkv) * n_sub;
  const int64_t items = n_rests * tiles_per_row;
  if (items >= (int64_t(1) << 30)) return false;
  pl->fp8 = fp8;
  pl->g_shift = g_shift;
  pl->tiles_per_row = int(tiles_per_row); pl->n_sub = n_sub; pl->n_rests = int(n_rests);
  // One CTA per SM.  When the row sets divide the SMs (almost) evenly every row set gets its own CTAs,
  // so that no CTA works for two of them; otherwise all CTAs share the items as one contiguous range.
  const int per_set = int(kNumSMs / std::max<int64_t>(1, n_rests));
  if (n_rests <= kNumSMs && n_rests * per_set * 20 >= int64_t(kNumSMs) * 19 && tiles_per_row >= int64_t(per_set) * kWarps) {
    pl->vset_items = int(tiles_per_row);
    pl->ctas_per_vset = per_set;
    pl->ctas = int(n_rests) * per_set;
  } else {
    pl->vset_items = int(items);
    pl->ctas_per_vset = int(std::max<int64_t>(1, std::min<int64_t>(kNumSMs, (items + kWarps - 1) / kWarps)));
    pl->ctas = pl->ctas_per_vset;
  }
  const int warps = pl->ctas_per_vset * kWarps;
  pl->base = pl->vset_items / warps;
  pl->rem = pl->vset_items % warps;
  // The CTA builds the low-rank queries itself when it touches few row sets and the adapter has the
  // layout build_queries() reads (r = 32 columns, d a multiple of 32 up to 128).
  const int64_t cta_items = int64_t(pl->base + 1) * kWarps;
  const int64_t sets_touched = (cta_items + tiles_per_row - 1) / tiles_per_row + 1;
  pl->fused = p.r == 32 && (p.d == 32 || p.d == 64 || p.d == 128) && sets_touched <= kMaxSets;
  pl->counts = (pl->base + 1) * kWarps <= kMaxTilesPerCta;   // a CTA's counts stay below 2^16 per counter
  return true;
}

}  // namespace

bool score_stream_supported(const Problem& p) { Plan pl; return plan(p, &pl); }
bool score_stream_fuses_query(const Problem& p) { Plan pl; return plan(p, &pl) && pl.fused; }
bool score_stream_counts_top_digit(const Problem& p) { Plan pl; return plan(p, &pl) && pl.counts; }
void score_stream_row_sets(const Problem& p, int* n_rests, int* n_sub) {
  Plan pl;
  const bool ok = plan(p, &pl);
  *n_rests = ok ? pl.n_rests : 0;
  *n_sub = ok ? pl.n_sub : 1;
}

cudaError_t launch_score_stream(const Problem& p, const void* q, const float* proj, const float* uq, const void* meta,
                                float* scores, uint32_t* top_hist, uint32_t* err, cudaStream_t st) {
  Plan pl;
  if (!plan(p, &pl)) return cudaErrorInvalidValue;
  if (top_hist != nullptr && !pl.counts) return cudaErrorInvalidValue;
  // With q == NULL the queries come from `uq` even where the kernel could build them.
  if (q == nullptr) pl.fused = false;
  if (pl.fused ? (proj == nullptr) : (uq == nullptr)) return cudaErrorInvalidValue;
  StreamArgs a;
  a.q = q; a.proj = proj; a.uq = uq; a.meta = static_cast<const unsigned char*>(meta); a.scores = scores;
  a.top_hist = top_hist;
  a.tiles_per_row = pl.tiles_per_row; a.n_sub = pl.n_sub; a.n_rests = pl.n_rests;
  a.vset_items = pl.vset_items; a.ctas_per_vset = pl.ctas_per_vset; a.base = pl.base; a.rem = pl.rem;
  a.meta_scale = exp2f(float(p.meta_exp));
  a.err = err;
  const size_t smem = sizeof(Smem) + 128;
  auto go = [&](auto kern) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
    return launch_pdl(kern, dim3(pl.ctas), dim3(kThreads), smem, st, p, a);
  };
  auto go_gs = [&](auto fused, auto fp8) -> cudaError_t {
    constexpr bool F = decltype(fused)::value, E = decltype(fp8)::value;
    switch (pl.g_shift) {
      case 0: return go(score_stream_kernel<0, F, E>);
      case 1: return go(score_stream_kernel<1, F, E>);
      case 2: return go(score_stream_kernel<2, F, E>);
      case 3: return go(score_stream_kernel<3, F, E>);
      case 4: return go(score_stream_kernel<4, F, E>);
      default: return go(score_stream_kernel<5, F, E>);
    }
  };
  using T = std::true_type;
  using N = std::false_type;
  if (pl.fused) return pl.fp8 ? go_gs(T(), T()) : go_gs(T(), N());
  return pl.fp8 ? go_gs(N(), T()) : go_gs(N(), N());
}

}  // namespace kvswap
