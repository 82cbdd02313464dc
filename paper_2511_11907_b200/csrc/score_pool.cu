// K2: low-rank query (Eq. 1), token scoring, head aggregation and group ReduceMax (Sec. 4.3).
//
// The per-head score (Q_h A_g(h)) K_lr^T is linear in the low-rank query, so the sum over the
// heads of a scope is taken on the low-rank queries first:
//     T[b,s,n] = sum_t  uq[b, row(s,t), :] . meta[b, head(t), n, :]
// with, per KV head g,  u_g = (sum_{h: g(h)=g} q_h) A_g  and
//   joint metadata   (H_m = 1):    one term, head 0, uq row s = sum of u_g over the scope;
//   per-head metadata, KV_HEAD:    one term, head g = s, uq row g = u_g;
//   per-head metadata, ALL_HEADS:  H_kv terms, term t reads head t with uq row t = u_t.
//
// The scorers of this file (fp16 metadata rows of 64 bytes take the tensor-core scorer of
// score_stream.cu, which also builds the low-rank queries itself):
//   score_pool_tiles_kernel  the streaming path for fp32 metadata rows of 64 bytes (r = 16) that
//                            are dense in memory, G a power of two <= 32 and one term per score.
//                            Warps pull 2 KB tiles of 32 rows into shared memory with bulk
//                            asynchronous copies, several tiles in flight per warp.
//   score_pool_kernel        every other shape (any r, G, stride; the H_kv-term case).
#include <algorithm>

#include "async_copy.cuh"
#include "common.cuh"

namespace kvswap {
namespace {

constexpr int kThreads = 256;
constexpr uint32_t kFull = 0xffffffffu;

// ------------------------------------------------------------------------------------------
// K2a: uq rows.  grid (B, rows): a CTA produces one uq row, looping over the KV heads that feed
// it (one, except for joint metadata under the all-heads scope).  256 threads = 8 slices of the
// contraction index x 32 output columns (r <= 32), or the generic loop for larger r.
// ------------------------------------------------------------------------------------------
template <typename Q_T>
__global__ void __launch_bounds__(4 * kThreads)
lowrank_query_kernel(Problem p, const Q_T* __restrict__ q, const float* __restrict__ proj,
                     float* __restrict__ uq) {
  // blockDim.x = kThreads * n_grp: thread group `grp` (256 threads) takes the KV heads
  // g0 + grp, g0 + grp + n_grp, ... of the row, so that up to four heads are in flight at once.
  __shared__ float qsum[4][128];
  __shared__ float red[4 * kThreads];
  // With the query settled (KVSWAP_INPUTS_SETTLED) only the write of the result has to wait for
  // the previous kernel of the stream, whose predecessors may still be reading the buffer.
  const bool settled = (p.flags & KVSWAP_INPUTS_SETTLED) != 0;
  if (!settled) pdl_wait();
  pdl_trigger();
  const int b = blockIdx.x, row = blockIdx.y;
  const int tid = threadIdx.x % kThreads, grp = threadIdx.x / kThreads, n_grp = blockDim.x / kThreads;
  // KV heads summed into this row
  const bool joint_all = (p.Hm == 1 && p.scope == KVSWAP_SCOPE_ALL_HEADS);
  const int g0 = joint_all ? 0 : row;
  const int g1 = joint_all ? p.Hkv : row + 1;
  const int parts = kThreads / p.r;               // r <= 256
  const int j = tid % p.r, part = tid / p.r;
  float acc = 0.f;
  for (int gb = g0; gb < g1; gb += n_grp) {       // every group runs every iteration (barriers inside)
    const int g = gb + grp;
    const bool on = g < g1;
    __syncthreads();
    if (on) {
      for (int c = tid; c < p.d; c += kThreads) {
        // the rho loads are independent: issue them four at a time (one memory round trip for rho <= 4)
        const Q_T* qc = q + (int64_t(b) * p.Hq + g * p.rho) * p.d + c;
        float s = 0.f;
        for (int h0 = 0; h0 < p.rho; h0 += 4) {
          float v[4];
#pragma unroll
          for (int hh = 0; hh < 4; ++hh) v[hh] = (h0 + hh < p.rho) ? float(qc[int64_t(h0 + hh) * p.d]) : 0.f;
          s += (v[0] + v[1]) + (v[2] + v[3]);
        }
        qsum[grp][c] = s;
      }
    }
    // The adapter rows do not depend on q: fetch this thread's share before the barrier.
    const float* Pg = proj + int64_t(on ? g : g0) * p.d * p.r;
    float pj[16];
    int n_c = 0;
    if (on && part < parts) {
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int c = part + i * parts;
        pj[i] = (c < p.d) ? Pg[int64_t(c) * p.r + j] : 0.f;
      }
      n_c = (p.d - part + parts - 1) / parts;
    }
    __syncthreads();
    if (on && part < parts) {
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int c = part + i * parts;
        if (c < p.d) acc = fmaf(qsum[grp][c], pj[i], acc);
      }
      for (int i = 16; i < n_c; ++i) {              // only when d / parts > 16 (large r)
        const int c = part + i * parts;
        acc = fmaf(qsum[grp][c], Pg[int64_t(c) * p.r + j], acc);
      }
    }
  }
  red[threadIdx.x] = (part < parts) ? acc : 0.f;
  __syncthreads();
  if (settled) pdl_wait();
  if (threadIdx.x < p.r) {
    float s = 0.f;
    for (int gq = 0; gq < n_grp; ++gq)
      for (int k = 0; k < parts; ++k) s += red[gq * kThreads + k * p.r + threadIdx.x];
    uq[(int64_t(b) * p.Su + row) * p.r + threadIdx.x] = s;
  }
}

// ------------------------------------------------------------------------------------------
// K2, streaming path.
//
// Work item = (sequence b, metadata head hm, block of NS scopes, tile of kTileRows rows); items
// are numbered with the tile index fastest and every warp of the grid takes an equal contiguous
// share.  A warp owns kDepth shared-memory stages of one tile each, guarded by an mbarrier, and
// refills a stage as soon as it has consumed it, so kDepth tiles per warp are in flight.
//
// Inside a tile a warp-wide 16-byte read covers 8 rows x 64 bytes: lane = 4 * (row in the 8) +
// (16-byte quarter of the row).  A lane keeps the NS x (quarter) slice of the summed low-rank
// queries in registers, forms its partial dot products, and the four lanes of a row exchange
// them in a reduce-scatter (each ends with NS/4 complete scores).  ReduceMax over a group is a
// butterfly over the row bits of the lane index (G <= 8) and a running maximum over successive
// reads (G > 8).  Group scores of a tile are collected in shared memory and written out in rows.
// ------------------------------------------------------------------------------------------
constexpr int kTileRows = 32;
constexpr int kRowBytes = 64;
constexpr int kTileBytes = kTileRows * kRowBytes;
constexpr int kWarps = 8;
constexpr int kDepth = 4;
constexpr int kOutStride = kTileRows + 1;   // padded row of the per-warp output tile (bank spread)

struct TileControl {
  unsigned long long full[kWarps * kDepth];
};

// 16 bytes of a metadata row as fp32 pairs.
template <typename META_T>
__device__ __forceinline__ void lds_quarter(uint32_t addr, float2 (&m)[8 / sizeof(META_T)]) {
  uint32_t w[4];
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr));
  if constexpr (sizeof(META_T) == 2) {
#pragma unroll
    for (int i = 0; i < 4; ++i) m[i] = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
  } else {
    m[0] = make_float2(__uint_as_float(w[0]), __uint_as_float(w[1]));
    m[1] = make_float2(__uint_as_float(w[2]), __uint_as_float(w[3]));
  }
}

template <typename META_T, int NS>
__global__ void __launch_bounds__(kWarps * 32, 2)
score_pool_tiles_kernel(Problem p, const float* __restrict__ uq, const META_T* __restrict__ meta,
                        float* __restrict__ scores, int tiles_per_row, int n_sub, int g_shift,
                        uint32_t* __restrict__ err) {
  constexpr int KP = 8 / sizeof(META_T);            // fp32 pairs in a 16-byte quarter
  constexpr int NV = (NS >= 4) ? NS / 4 : 1;        // complete scores a lane ends up with
  extern __shared__ __align__(128) unsigned char dyn[];
  unsigned char* tiles = dyn;                                                       // [kWarps][kDepth][kTileBytes]
  TileControl* ctl = reinterpret_cast<TileControl*>(dyn + kWarps * kDepth * kTileBytes);
  float* outbuf = reinterpret_cast<float*>(dyn + kWarps * kDepth * kTileBytes + sizeof(TileControl));  // [kWarps][NS][kOutStride]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rq = lane >> 2, qt = lane & 3;          // row within a read, quarter of the row
  if (lane == 0) {                                  // every warp sets up its own stages: no CTA-wide wait
    for (int s = 0; s < kDepth; ++s) mbar_init(smem_addr(&ctl->full[warp * kDepth + s]), 1);
    mbar_init_fence();
  }
  __syncwarp();

  // Equal contiguous share of the work items for every warp of the grid (fewer than 2^31 items).
  const int rows_total = p.NG * p.G;                // scored rows per (sequence, metadata head)
  const int hm_count = (p.Hm == 1) ? 1 : p.Hkv;
  const int64_t items = int64_t(p.B) * hm_count * n_sub * tiles_per_row;
  const int64_t gw = int64_t(blockIdx.x) * kWarps + warp, n_gw = int64_t(gridDim.x) * kWarps;
  const int first = int(items * gw / n_gw), last = int(items * (gw + 1) / n_gw);
  const int my_tiles = last - first;

  // Cursors over the warp's items: (tile within the row set, row set = (b * hm_count + hm) * n_sub + sub).
  int f_tile = first % tiles_per_row, f_rest = first / tiles_per_row;     // next item to request
  int c_tile = f_tile, c_rest = f_rest;                                   // next item to consume

  const uint32_t ring = smem_addr(tiles) + uint32_t(warp) * kDepth * kTileBytes;
  const META_T* f_base = nullptr;                   // metadata of the fill cursor's (sequence, head)
  int f_base_rest = -1;
  auto fill = [&](int stage) {                      // requests the item under the fill cursor
    if (lane == 0) {
      if (f_rest != f_base_rest) {
        f_base_rest = f_rest;
        const int bh = f_rest / n_sub;
        f_base = meta + int64_t(bh / hm_count) * p.meta_sb + int64_t(bh % hm_count) * p.meta_sh;
      }
      const int rows = min(kTileRows, rows_total - f_tile * kTileRows);
      const META_T* src = f_base + int64_t(f_tile) * kTileRows * p.meta_sn;
      const uint32_t bar = smem_addr(&ctl->full[warp * kDepth + stage]);
      mbar_arrive_expect_tx(bar, uint32_t(rows) * kRowBytes);
      bulk_g2s(ring + uint32_t(stage) * kTileBytes, src, uint32_t(rows) * kRowBytes, bar);
    }
    if (++f_tile == tiles_per_row) { f_tile = 0; ++f_rest; }
  };
  // The metadata is never written by the kernel that precedes this one in the same call (the
  // low-rank query kernel), so the first tiles may be requested before the dependency wait.
  for (int k = 0; k < kDepth && k < my_tiles; ++k) fill(k);
  pdl_wait();
  pdl_trigger();

  // Scope order of this lane's registers: register c holds scope c ^ perm, so that both
  // reduce-scatter steps pair a kept register with the partner's sent one without selects.
  const int perm = (NS >= 8) ? (((lane & 1) << 2) | (lane & 2)) : (NS == 4) ? (((lane & 1) << 1) | ((lane >> 1) & 1))
                 : (NS == 2) ? (lane & 1) : 0;
  float2 uu[NS][KP];
  int cur_rest = -1;
  int b = 0, sub = 0, hm = 0;
  float vmax[NV];                                   // running group maxima (G > 8)
#pragma unroll
  for (int i = 0; i < NV; ++i) vmax[i] = -INFINITY;
  const int gb = (g_shift < 3) ? g_shift : 3;       // butterfly levels over the row bits
  float* out = outbuf + warp * (NS * kOutStride);
  int stage = 0;
  uint32_t phase = 0;
  bool timed_out = false;
  for (int k = 0; k < my_tiles; ++k) {
    const int tile = c_tile;
    if (c_rest != cur_rest) {                       // new (sequence, head, scope block): reload u
      cur_rest = c_rest;
      sub = c_rest % n_sub;
      const int bh = c_rest / n_sub;
      hm = bh % hm_count; b = bh / hm_count;
      const int urow0 = (p.Hm == 1) ? sub * NS : hm;
#pragma unroll
      for (int c = 0; c < NS; ++c) {
        const int sc = c ^ perm;
        const bool have = (p.Hm != 1) || (sub * NS + sc < p.S);
        const float* ur = uq + (int64_t(b) * p.Su + urow0 + ((p.Hm == 1 && have) ? sc : 0)) * p.r + qt * (2 * KP);
#pragma unroll
        for (int i = 0; i < KP; ++i)
          uu[c][i] = have ? *reinterpret_cast<const float2*>(ur + 2 * i) : make_float2(0.f, 0.f);
      }
    }
    if (++c_tile == tiles_per_row) { c_tile = 0; ++c_rest; }
    if (!__all_sync(kFull, mbar_wait(smem_addr(&ctl->full[warp * kDepth + stage]), phase))) { timed_out = true; break; }
    const int rows = min(kTileRows, rows_total - tile * kTileRows);
    const uint32_t base = ring + uint32_t(stage) * kTileBytes + uint32_t(lane) * 16u;
    for (int it = 0; it * 8 < rows; ++it) {
      float2 m[KP];
      lds_quarter<META_T>(base + uint32_t(it) * 8u * kRowBytes, m);
      float v[NS];
#pragma unroll
      for (int c = 0; c < NS; ++c) {
        float a = uu[c][0].x * m[0].x;
        a = fmaf(uu[c][0].y, m[0].y, a);
#pragma unroll
        for (int i = 1; i < KP; ++i) { a = fmaf(uu[c][i].x, m[i].x, a); a = fmaf(uu[c][i].y, m[i].y, a); }
        v[c] = a;
      }
      // ---- the four lanes of a row: reduce-scatter of the NS partial scores -----------------
      if constexpr (NS >= 8) {
#pragma unroll
        for (int c = 0; c < 4; ++c) v[c] += __shfl_xor_sync(kFull, v[c + 4], 1);
#pragma unroll
        for (int c = 0; c < 2; ++c) v[c] += __shfl_xor_sync(kFull, v[c + 2], 2);
      } else if constexpr (NS == 4) {
#pragma unroll
        for (int c = 0; c < 2; ++c) v[c] += __shfl_xor_sync(kFull, v[c + 2], 1);
        v[0] += __shfl_xor_sync(kFull, v[1], 2);
      } else if constexpr (NS == 2) {
        v[0] += __shfl_xor_sync(kFull, v[1], 1);
        v[0] += __shfl_xor_sync(kFull, v[0], 2);
      } else {
        v[0] += __shfl_xor_sync(kFull, v[0], 1);
        v[0] += __shfl_xor_sync(kFull, v[0], 2);
      }
      // ---- ReduceMax over the rows of a group --------------------------------------------------
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        float x = v[i];
        if (gb >= 1) x = fmaxf(x, __shfl_xor_sync(kFull, x, 4));
        if (gb >= 2) x = fmaxf(x, __shfl_xor_sync(kFull, x, 8));
        if (gb >= 3) x = fmaxf(x, __shfl_xor_sync(kFull, x, 16));
        vmax[i] = fmaxf(vmax[i], x);
      }
      const int row_end = it * 8 + 8;               // rows of the tile seen so far
      if (g_shift <= 3 || (row_end & (p.G - 1)) == 0) {
        // a group (or 8 >> g_shift groups) ends with this read: its first row's lanes publish it
        const int gi = (it * 8 + rq) >> g_shift;    // group within the tile
        if ((rq & ((1 << gb) - 1)) == 0) {
#pragma unroll
          for (int i = 0; i < NV; ++i) out[((i ^ perm) & (NS - 1)) * kOutStride + gi] = vmax[i];
        }
#pragma unroll
        for (int i = 0; i < NV; ++i) vmax[i] = -INFINITY;
      }
    }
    __syncwarp();
    // ---- write the tile's group scores, scope by scope ------------------------------------------
    {
      const int ngt = rows >> g_shift;              // groups in this tile
      const int g0 = (tile * kTileRows) >> g_shift;
      const int s0 = (p.Hm == 1) ? sub * NS : hm;
      const int ns = (p.Hm == 1) ? min(NS, p.S - s0) : 1;
      for (int i = lane; i < ns * ngt; i += 32) {
        const int s = i / ngt, gi = i - s * ngt;
        scores[(int64_t(b) * p.S + s0 + s) * p.score_pitch + g0 + gi] = out[s * kOutStride + gi];
      }
    }
    __syncwarp();                                   // stage and outbuf are free again
    if (k + kDepth < my_tiles) fill(stage);
    if (++stage == kDepth) { stage = 0; phase ^= 1u; }
  }
  if (timed_out) {
    if (lane == 0 && err) atomicExch(err, kDevTimeoutFull);
    for (int s = 0; s < kDepth; ++s) {              // bounded chance for copies in flight to land
      mbar_wait(smem_addr(&ctl->full[warp * kDepth + s]), 0);
      mbar_wait(smem_addr(&ctl->full[warp * kDepth + s]), 1);
    }
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
  pdl_wait();
  pdl_trigger();
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
    scores[(int64_t(b) * p.S + out0 + k) * p.score_pitch + grp0 + gi] = m;
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
  return launch_pdl(kern, grid, dim3(kThreads), smem, st, p, uq, static_cast<const META_T*>(meta), scores, gpt, lpr);
}

template <typename META_T, int NS>
cudaError_t launch_tiles(const Problem& p, const float* uq, const void* meta, float* scores, int g_shift,
                         uint32_t* err, cudaStream_t st) {
  const int rows_total = p.NG * p.G;
  const int tiles_per_row = (rows_total + kTileRows - 1) / kTileRows;
  const int n_sub = (p.Hm == 1) ? (p.S + NS - 1) / NS : 1;
  const int hm_count = (p.Hm == 1) ? 1 : p.Hkv;
  const int64_t items = int64_t(p.B) * hm_count * n_sub * tiles_per_row;
  // One wave of two CTAs per SM; fewer CTAs when there is not at least one tile per warp.
  const int64_t want = (items + kWarps - 1) / kWarps;
  const int ctas = int(std::max<int64_t>(1, std::min<int64_t>(2 * kNumSMs, want)));
  const size_t smem = size_t(kWarps) * kDepth * kTileBytes + sizeof(TileControl) + sizeof(float) * kWarps * NS * kOutStride;
  auto kern = score_pool_tiles_kernel<META_T, NS>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
  if (e != cudaSuccess) return e;
  return launch_pdl(kern, dim3(ctas), dim3(kWarps * 32), smem, st, p, uq, static_cast<const META_T*>(meta), scores,
                    tiles_per_row, n_sub, g_shift, err);
}

template <typename META_T>
cudaError_t launch_meta(const Problem& p, const float* uq, const void* meta, float* scores, uint32_t* err,
                        cudaStream_t st) {
  int g_shift = -1;
  for (int s = 0; s <= 5; ++s) if ((1 << s) == p.G) g_shift = s;
  const bool one_term = (p.Hm == 1) || (p.scope == KVSWAP_SCOPE_KV_HEAD);
  const int64_t tile_items = int64_t(p.B) * p.Hkv * ((int64_t(p.NG) * p.G + kTileRows - 1) / kTileRows);
  // fp16 rows of this kind are served by the tensor-core scorer (score_stream.cu)
  const bool streaming = one_term && g_shift >= 0 && p.r * int(sizeof(META_T)) == kRowBytes && p.meta_sn == p.r &&
                         tile_items < (int64_t(1) << 30);
  if constexpr (!std::is_same<META_T, __half>::value) {
    if (streaming) {
      const int ns = (p.Hm == 1) ? p.S : 1;
      if (ns == 1) return launch_tiles<META_T, 1>(p, uq, meta, scores, g_shift, err, st);
      if (ns == 2) return launch_tiles<META_T, 2>(p, uq, meta, scores, g_shift, err, st);
      if (ns <= 4) return launch_tiles<META_T, 4>(p, uq, meta, scores, g_shift, err, st);
      return launch_tiles<META_T, 8>(p, uq, meta, scores, g_shift, err, st);
    }
  }
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
  // One 256-thread group per KV head in flight: one group per row, up to four when a row sums
  // all KV heads (joint metadata under the all-heads scope).
  const bool joint_all = (p.Hm == 1 && p.scope == KVSWAP_SCOPE_ALL_HEADS);
  const dim3 block(kThreads * (joint_all ? std::min(4, p.Hkv) : 1));
  switch (p.q_dtype) {
    case KVSWAP_F32:
      return launch_pdl(lowrank_query_kernel<float>, grid, block, 0, st, p, static_cast<const float*>(q), proj, uq);
    case KVSWAP_BF16:
      return launch_pdl(lowrank_query_kernel<__nv_bfloat16>, grid, block, 0, st, p,
                        static_cast<const __nv_bfloat16*>(q), proj, uq);
    default:
      return launch_pdl(lowrank_query_kernel<__half>, grid, block, 0, st, p, static_cast<const __half*>(q), proj, uq);
  }
}

cudaError_t launch_score_pool(const Problem& p, const float* uq, const void* meta, float* scores, uint32_t* err,
                              cudaStream_t st) {
  if (p.meta_dtype == KVSWAP_F16) return launch_meta<__half>(p, uq, meta, scores, err, st);
  return launch_meta<float>(p, uq, meta, scores, err, st);
}

}  // namespace kvswap
