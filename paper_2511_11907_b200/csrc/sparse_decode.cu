// K4 + K5: exact decode attention over the selected groups and the rolling-buffer tail
// (Sec. 4.4, 4.4.1, 4.4.4): gather + split-K flash-decode with an fp32 online softmax, then a
// log-sum-exp merge of the split partials.
//
// The attended tokens of one (sequence, selection row) form a virtual list
//     v in [0, n_sel*G):  token  group_idx[v / G] * G + v % G
//     v in [n_sel*G, n_sel*G + tail):  token  NG*G + (v - n_sel*G)
// which is cut into `splits` contiguous ranges, one CTA each, and every range into chunks of
// kTok tokens.  A CTA serves RH query heads that share the KV head, so each K/V row is read once.
//
// Every warp of the CTA works alone on the chunks c = warp, warp + kWarps, ...: it owns `depth`
// shared-memory stages, each guarded by an mbarrier, and keeps them filled itself.  Lanes 0..7
// resolve the kTok token rows of a chunk and bring their K and V rows in with bulk asynchronous
// copies (one copy per run of consecutive rows: a whole group when rows are dense); the copy for
// chunk k + depth is issued the moment chunk k has been consumed, so `depth` chunks per warp are
// in flight while it computes and no warp ever waits for another.
//
// A warp owns D/32 channels per lane.  For a chunk it forms the kTok x RH partial dot products
// of its channel slice, then transposes-and-sums them across the warp (a reduce-scatter by
// shuffles) so that lane L ends up with the complete logit of (token L/4, head L%4): the softmax
// bookkeeping then runs once per chunk with all 32 lanes busy.  Probabilities go through a small
// shared-memory tile back to all lanes for the P.V update of their channel slice.
#include <algorithm>

#include "async_copy.cuh"
#include "common.cuh"

namespace kvswap {
namespace {

constexpr int kTok = 8;                         // tokens per stage
constexpr int kWarps = 8;                       // warps per CTA
constexpr int kThreads = kWarps * 32;
constexpr int kMaxDepth = 4;                    // stages per warp, at most
constexpr int kMaxStages = kWarps * kMaxDepth;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Control block at the start of dynamic shared memory.
struct Control {
  unsigned long long full[kMaxStages];          // data of the stage has landed
  uint32_t mask[kMaxStages];                    // bit t: token slot t of the stage holds a row
  float2 prob[kWarps][kTok * 4];                // softmax weights of the chunk, [token][head], each twice
  float2 corr[kWarps][4];                       // rescale of the running accumulator, [head], each twice
  uint32_t abort;                               // a wait timed out somewhere in the CTA
};
constexpr int kControlBytes = (sizeof(Control) + 255) & ~255;

template <typename Q_T>
__device__ __forceinline__ float q_to_float(Q_T v) { return float(v); }

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// DPL consecutive channels of one staged row, widened to fp32.
template <typename KV_T, int DPL>
__device__ __forceinline__ void lds_row(uint32_t addr, float (&f)[DPL]) {
  if constexpr (sizeof(KV_T) == 4) {
    if constexpr (DPL == 4) {
      asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(f[0]), "=f"(f[1]), "=f"(f[2]), "=f"(f[3]) : "r"(addr));
    } else {
      asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(f[0]), "=f"(f[1]) : "r"(addr));
    }
  } else {
    uint32_t w[DPL / 2];
    if constexpr (DPL == 4) {
      asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(w[0]), "=r"(w[1]) : "r"(addr));
    } else {
      asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w[0]) : "r"(addr));
    }
#pragma unroll
    for (int i = 0; i < DPL / 2; ++i) {
      if constexpr (std::is_same<KV_T, __nv_bfloat16>::value) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
      } else {
        const float2 t = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
        f[2 * i] = t.x; f[2 * i + 1] = t.y;
      }
    }
  }
}

// Where the attended tokens of one CTA come from.
struct TokenSource {
  const int32_t* idx;      // selection row
  int NG, G, g_shift;      // g_shift = log2(G) when G is a power of two, else -1
  int sel_tokens, tail0;   // n_sel * G, NG * G
  int v_begin, v_end;      // this CTA's range of the virtual token list

  // Group ordinal of virtual token v (v < sel_tokens).
  __device__ __forceinline__ int group_of(int v) const { return g_shift >= 0 ? (v >> g_shift) : (v / G); }
};

template <typename KV_T, typename Q_T, int D, int RH>
__global__ void __launch_bounds__(kThreads, 2)
sparse_decode_splitk_kernel(Problem p, const Q_T* __restrict__ q, const KV_T* __restrict__ K,
                            const KV_T* __restrict__ V, const int32_t* __restrict__ group_idx,
                            const int32_t* __restrict__ n_selected, float* __restrict__ partial,
                            int splits, int depth, int g_shift, uint32_t* __restrict__ err) {
  constexpr int DPL = D / 32;                                  // channels per lane
  constexpr uint32_t ROWB = D * sizeof(KV_T);                  // bytes of one K or V row
  constexpr uint32_t HALFB = kTok * ROWB;                      // K (or V) part of a stage
  constexpr uint32_t STAGEB = 2 * HALFB;
  constexpr uint32_t kFull = 0xffffffffu;

  extern __shared__ unsigned char smem_raw[];
  Control* ctl = reinterpret_cast<Control*>(smem_raw);
  // Stage ring, aligned to HALFB so that a row index can be xor-ed into an address.
  const uint32_t ring = (smem_addr(smem_raw) + kControlBytes + HALFB - 1) & ~(HALFB - 1);
  unsigned char* ring_ptr = smem_raw + (ring - smem_addr(smem_raw));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x;
  const int chunks = p.rho / RH;
  const int g = blockIdx.y / chunks, hc = blockIdx.y % chunks;
  const int b = blockIdx.z;
  const int h0 = g * p.rho + hc * RH;                          // first query head of this CTA
  const int srow = (p.scope == KVSWAP_SCOPE_KV_HEAD) ? g : 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kWarps * depth; ++s) mbar_init(smem_addr(&ctl->full[s]), 1);
    ctl->abort = 0;
    mbar_init_fence();
  }
  __syncthreads();

  // Nothing above touches global memory; everything below may depend on the previous kernel.
  pdl_wait();
  pdl_trigger();

  TokenSource src;
  src.idx = group_idx + (int64_t(b) * p.S + srow) * p.M;
  src.NG = p.NG; src.G = p.G; src.g_shift = g_shift;
  {
    int n_sel = n_selected[int64_t(b) * p.S + srow];
    n_sel = max(0, min(n_sel, p.M));
    src.tail0 = p.NG * p.G;
    src.sel_tokens = n_sel * p.G;
    const int total = src.sel_tokens + (p.N - src.tail0);
    int per_split = (total + splits - 1) / splits;
    per_split = (per_split + kTok - 1) / kTok * kTok;
    src.v_begin = min(total, per_split * split);
    src.v_end = min(total, src.v_begin + per_split);
  }
  const int n_chunks = (src.v_end - src.v_begin + kTok - 1) / kTok;
  const int my_chunks = (n_chunks > warp) ? (n_chunks - warp + kWarps - 1) / kWarps : 0;   // of this warp

  const KV_T* Kg = K + int64_t(b) * p.kv_sb + int64_t(g) * p.kv_sh;
  const KV_T* Vg = V + int64_t(b) * p.kv_sb + int64_t(g) * p.kv_sh;
  const bool dense = (p.kv_sn == D);

  // When rows are dense and G is a multiple of kTok, a chunk is kTok consecutive rows of one
  // group (or of the tail): lane 0 alone resolves it and issues one copy each for K and V.
  const bool whole = dense && (p.G % kTok == 0);

  // Group index (or -1) behind token slot `lane` of this warp's k-th chunk: the one global read
  // of the fill path, issued early so that its latency hides behind the compute of a chunk.
  auto fetch_group = [&](int k) -> int {
    const int v = src.v_begin + (warp + k * kWarps) * kTok + lane;
    if (lane < (whole ? 1 : kTok) && k < my_chunks && v < src.v_end && v < src.sel_tokens)
      return src.idx[src.group_of(v)];
    return -1;
  };
  // Fill: bring chunk k into `stage`.  `j` is fetch_group(k).  All 32 lanes call.
  auto fill = [&](int k, int j, int stage) {
    const int v = src.v_begin + (warp + k * kWarps) * kTok + lane;
    const uint32_t bar = smem_addr(&ctl->full[stage]);
    if (whole) {
      if (lane == 0) {
        const int rows = min(kTok, src.v_end - v);
        int n = -1;
        if (v < src.sel_tokens) {
          if (j >= 0 && j < src.NG) n = j * src.G + (v - src.group_of(v) * src.G);
        } else {
          n = src.tail0 + (v - src.sel_tokens);
        }
        ctl->mask[stage] = (n >= 0) ? ((1u << rows) - 1u) : 0u;
        mbar_arrive_expect_tx(bar, (n >= 0) ? uint32_t(rows) * 2u * ROWB : 0u);
        if (n >= 0) {
          const uint32_t dst = ring + uint32_t(stage) * STAGEB;
          bulk_g2s(dst, Kg + int64_t(n) * D, uint32_t(rows) * ROWB, bar);
          bulk_g2s(dst + HALFB, Vg + int64_t(n) * D, uint32_t(rows) * ROWB, bar);
        }
      }
      return;
    }
    int n = -1;
    if (lane < kTok && v < src.v_end) {
      if (v < src.sel_tokens) {
        if (j >= 0 && j < src.NG) n = j * src.G + (v - src.group_of(v) * src.G);
      } else {
        n = src.tail0 + (v - src.sel_tokens);
      }
    }
    const bool valid = n >= 0;
    const uint32_t vmask = __ballot_sync(kFull, valid);
    const int n_prev = __shfl_up_sync(kFull, n, 1);
    const bool head = valid && (!dense || lane == 0 || !((vmask >> (lane - 1)) & 1u) || n != n_prev + 1);
    const uint32_t heads = __ballot_sync(kFull, head);
    if (lane == 0) {
      ctl->mask[stage] = vmask;
      mbar_arrive_expect_tx(bar, uint32_t(__popc(vmask)) * 2u * ROWB);
    }
    if (head) {
      const uint32_t stop = (heads | ~vmask | (1u << kTok)) & ~((2u << lane) - 1u);
      const uint32_t run = uint32_t(__ffs(int(stop)) - 1 - lane);
      const uint32_t dst = ring + uint32_t(stage) * STAGEB + uint32_t(lane) * ROWB;
      bulk_g2s(dst, Kg + int64_t(n) * p.kv_sn, run * ROWB, bar);
      bulk_g2s(dst + HALFB, Vg + int64_t(n) * p.kv_sn, run * ROWB, bar);
    }
  };

  // ---- prologue: fill the first `depth` stages ---------------------------------------------------
  {
    int j0[kMaxDepth];
#pragma unroll
    for (int k = 0; k < kMaxDepth; ++k) j0[k] = (k < depth) ? fetch_group(k) : -1;
#pragma unroll
    for (int k = 0; k < kMaxDepth; ++k)
      if (k < depth && k < my_chunks) fill(k, j0[k], warp + kWarps * k);
  }

  // q slice of this lane, pre-scaled by log2(e)/sqrt(d) (logits live in the log2 domain), each
  // value twice: the packed FMA below works on two tokens at a time.
  const float scale = kLog2e * rsqrtf(float(D));
  float2 qq[RH][DPL];
#pragma unroll
  for (int hh = 0; hh < RH; ++hh)
#pragma unroll
    for (int j = 0; j < DPL; ++j) {
      const float x = q_to_float(q[(int64_t(b) * p.Hq + h0 + hh) * D + lane * DPL + j]) * scale;
      qq[hh][j] = make_float2(x, x);
    }

  float m_run = -INFINITY, l_run = 0.f;           // of head lane % 4 (replicated over the tokens)
  float2 acc[RH][DPL / 2];                         // channel pairs
#pragma unroll
  for (int hh = 0; hh < RH; ++hh)
#pragma unroll
    for (int j = 0; j < DPL / 2; ++j) acc[hh][j] = make_float2(0.f, 0.f);

  const int tok = lane >> 2, hd = lane & 3;        // the (token, head) this lane finishes
  const uint32_t lane_off = uint32_t(lane) * DPL * sizeof(KV_T);
  const uint32_t xperm = uint32_t(tok) * ROWB;     // slot s of this lane holds token s ^ tok
  float2* prob = ctl->prob[warp];
  float2* corr = ctl->corr[warp];
  int slot = 0;
  uint32_t phase = 0;
  bool timed_out = false;
  for (int k = 0; k < my_chunks; ++k) {
    const int stage = warp + kWarps * slot;
    const int j_next = fetch_group(k + depth);     // consumed by the refill at the end of the iteration
    if (!__all_sync(kFull, mbar_wait(smem_addr(&ctl->full[stage]), phase))) { timed_out = true; break; }
    const uint32_t mask = ctl->mask[stage];
    if (mask != 0u) {
      const uint32_t kbase = (ring + uint32_t(stage) * STAGEB + lane_off) ^ xperm;
      const uint32_t vbase = ring + uint32_t(stage) * STAGEB + HALFB + lane_off;

      // ---- partial q.k of this lane's channels; slot s <-> token s ^ tok, slots s and s + 4 share
      // a packed accumulator (.x, .y) ------------------------------------------------------------
      float2 part[4][4];
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        float ka[DPL], kb[DPL];
        lds_row<KV_T, DPL>(kbase ^ (uint32_t(s) * ROWB), ka);
        lds_row<KV_T, DPL>(kbase ^ (uint32_t(s + 4) * ROWB), kb);
#pragma unroll
        for (int hh = 0; hh < 4; ++hh) {
          float2 a = make_float2(0.f, 0.f);
          if (hh < RH) {
            a = __fmul2_rn(qq[hh][0], make_float2(ka[0], kb[0]));
#pragma unroll
            for (int j = 1; j < DPL; ++j) a = __ffma2_rn(qq[hh][j], make_float2(ka[j], kb[j]), a);
          }
          part[s][hh] = a;
        }
      }
      // ---- reduce-scatter over the warp: tokens over lane bits 4..2, heads over bits 1..0 ------
      float red[4][4];
#pragma unroll
      for (int s = 0; s < 4; ++s)
#pragma unroll
        for (int hh = 0; hh < 4; ++hh)
          red[s][hh] = (hh < RH) ? part[s][hh].x + __shfl_xor_sync(kFull, part[s][hh].y, 16) : 0.f;
#pragma unroll
      for (int s = 0; s < 2; ++s)
#pragma unroll
        for (int hh = 0; hh < RH; ++hh) red[s][hh] += __shfl_xor_sync(kFull, red[s + 2][hh], 8);
#pragma unroll
      for (int hh = 0; hh < RH; ++hh) red[0][hh] += __shfl_xor_sync(kFull, red[1][hh], 4);
      const bool b1 = lane & 2, b0 = lane & 1;
      const float keep0 = b1 ? red[0][2] : red[0][0], keep1 = b1 ? red[0][3] : red[0][1];
      const float send0 = b1 ? red[0][0] : red[0][2], send1 = b1 ? red[0][1] : red[0][3];
      const float r0 = keep0 + __shfl_xor_sync(kFull, send0, 2);
      const float r1 = keep1 + __shfl_xor_sync(kFull, send1, 2);
      float s_log = (b0 ? r1 : r0) + __shfl_xor_sync(kFull, b0 ? r0 : r1, 1);

      // ---- online softmax for (token tok, head hd) ----------------------------------------------
      const bool live = ((mask >> tok) & 1u) && hd < RH;
      s_log = live ? s_log : -INFINITY;
      float cmax = s_log;
      cmax = fmaxf(cmax, __shfl_xor_sync(kFull, cmax, 4));
      cmax = fmaxf(cmax, __shfl_xor_sync(kFull, cmax, 8));
      cmax = fmaxf(cmax, __shfl_xor_sync(kFull, cmax, 16));
      const float m_new = fmaxf(m_run, cmax);
      const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
      const float pw = ex2(s_log - m_safe);          // 0 for dead (token, head) pairs
      const float cr = ex2(m_run - m_safe);          // 0 while nothing has been seen yet
      float psum = pw;
      psum += __shfl_xor_sync(kFull, psum, 4);
      psum += __shfl_xor_sync(kFull, psum, 8);
      psum += __shfl_xor_sync(kFull, psum, 16);
      l_run = fmaf(l_run, cr, psum);
      m_run = m_new;
      prob[lane] = make_float2(pw, pw);
      const bool rescale = __any_sync(kFull, cr != 1.f);   // the running maximum moved for some head
      if (rescale && tok == 0) corr[hd] = make_float2(cr, cr);
      __syncwarp();

      // ---- P.V on this lane's channels -----------------------------------------------------------
      if (rescale) {
        const float4 c01 = *reinterpret_cast<const float4*>(corr);
        const float4 c23 = *reinterpret_cast<const float4*>(corr + 2);
        const float2 cv[4] = {make_float2(c01.x, c01.y), make_float2(c01.z, c01.w), make_float2(c23.x, c23.y),
                              make_float2(c23.z, c23.w)};
#pragma unroll
        for (int hh = 0; hh < RH; ++hh)
#pragma unroll
          for (int j = 0; j < DPL / 2; ++j) acc[hh][j] = __fmul2_rn(acc[hh][j], cv[hh]);
      }
      auto pv_token = [&](int t) {
        float vf[DPL];
        lds_row<KV_T, DPL>(vbase + uint32_t(t) * ROWB, vf);
        const float4 p01 = *reinterpret_cast<const float4*>(prob + 4 * t);
        const float4 p23 = *reinterpret_cast<const float4*>(prob + 4 * t + 2);
        const float2 pv[4] = {make_float2(p01.x, p01.y), make_float2(p01.z, p01.w), make_float2(p23.x, p23.y),
                              make_float2(p23.z, p23.w)};
#pragma unroll
        for (int hh = 0; hh < RH; ++hh)
#pragma unroll
          for (int j = 0; j < DPL / 2; ++j)
            acc[hh][j] = __ffma2_rn(pv[hh], make_float2(vf[2 * j], vf[2 * j + 1]), acc[hh][j]);
      };
      if (mask == (1u << kTok) - 1u) {
#pragma unroll
        for (int t = 0; t < kTok; ++t) pv_token(t);
      } else {
#pragma unroll
        for (int t = 0; t < kTok; ++t)
          if ((mask >> t) & 1u) pv_token(t);          // warp-uniform; stale rows are never read
      }
    }
    __syncwarp();                                   // all lanes are done with the stage and prob[]
    if (k + depth < my_chunks) fill(k + depth, j_next, stage);
    if (++slot == depth) { slot = 0; phase ^= 1u; }
  }
  if (timed_out) {
    // The wait gave up: record it, and before the CTA's shared memory is released give this
    // warp's copies that may still be in flight a bounded chance to land.  The partial written
    // below is then meaningless; the status word tells the host.
    if (lane == 0) { ctl->abort = 1; if (err) atomicExch(err, kDevTimeoutFull); }
    for (int s = 0; s < depth; ++s) {
      mbar_wait(smem_addr(&ctl->full[warp + kWarps * s]), 0);
      mbar_wait(smem_addr(&ctl->full[warp + kWarps * s]), 1);
    }
  }

  // ---- merge the warps of the CTA ------------------------------------------------------------------
  __syncthreads();               // every loop above is bounded, so every warp arrives here
  // The ring is idle now (every issued copy was waited for); reuse it for the merge.
  float* sm_m = reinterpret_cast<float*>(ring_ptr);                 // [kWarps][4]
  float* sm_l = sm_m + kWarps * 4;                                  // [kWarps][4]
  float* sm_acc = sm_l + kWarps * 4;                                // [kWarps][RH][D]
  if (lane < 4) { sm_m[warp * 4 + lane] = m_run; sm_l[warp * 4 + lane] = l_run; }
#pragma unroll
  for (int hh = 0; hh < RH; ++hh)
#pragma unroll
    for (int j = 0; j < DPL / 2; ++j)
      *reinterpret_cast<float2*>(&sm_acc[(warp * RH + hh) * D + lane * DPL + 2 * j]) = acc[hh][j];
  __syncthreads();
  for (int i = threadIdx.x; i < RH * D; i += kThreads) {
    const int hh = i / D, c = i % D;
    float mx = -INFINITY;
#pragma unroll
    for (int k = 0; k < kWarps; ++k) mx = fmaxf(mx, sm_m[k * 4 + hh]);
    float lsum = 0.f, a = 0.f;
    if (mx > -INFINITY) {
#pragma unroll
      for (int k = 0; k < kWarps; ++k) {
        const float w = ex2(sm_m[k * 4 + hh] - mx);
        lsum = fmaf(sm_l[k * 4 + hh], w, lsum);
        a = fmaf(sm_acc[(k * RH + hh) * D + c], w, a);
      }
    }
    float* dst = partial + ((int64_t(b) * p.Hq + h0 + hh) * splits + split) * (D + 2);
    if (c == 0) { dst[0] = mx; dst[1] = lsum; }
    dst[2 + c] = a;
  }
}

// K5: merge the split partials of one (sequence, head).  One CTA of D threads per row; every
// load of the row is issued before anything is computed (one memory round trip), the split
// weights are formed once by the first warp and shared.
constexpr int kMaxSplits = 256;

template <int D>
__global__ void __launch_bounds__(D)
combine_kernel(const float* __restrict__ partial, float* __restrict__ out, float* __restrict__ lse, int splits) {
  __shared__ float w_s[kMaxSplits];
  __shared__ float norm_s[2];                  // 1 / sum of weights (or 0), lse
  pdl_wait();
  pdl_trigger();
  const int64_t bh = blockIdx.x;
  const float* src = partial + bh * splits * (D + 2);
  const int c = threadIdx.x;
  constexpr int kUnroll = 16;
  float a_first[kUnroll];
#pragma unroll
  for (int s = 0; s < kUnroll; ++s) a_first[s] = (s < splits) ? src[s * (D + 2) + 2 + c] : 0.f;
  if (c < 32) {
    // weights: lane s handles splits s, s + 32, ...
    float mx = -INFINITY;
    for (int s = c; s < splits; s += 32) mx = fmaxf(mx, src[s * (D + 2)]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    float lsum = 0.f;
    for (int s = c; s < splits; s += 32) {
      const float w = (mx > -INFINITY) ? exp2f(src[s * (D + 2)] - mx) : 0.f;
      w_s[s] = w;
      lsum = fmaf(src[s * (D + 2) + 1], w, lsum);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, off);
    if (c == 0) {
      norm_s[0] = (lsum > 0.f) ? 1.f / lsum : 0.f;
      norm_s[1] = (lsum > 0.f) ? (mx + log2f(lsum)) * kLn2 : -INFINITY;
    }
  }
  __syncthreads();
  float a = 0.f;
#pragma unroll
  for (int s = 0; s < kUnroll; ++s) if (s < splits) a = fmaf(a_first[s], w_s[s], a);
  for (int s = kUnroll; s < splits; ++s) a = fmaf(src[s * (D + 2) + 2 + c], w_s[s], a);
  out[bh * D + c] = a * norm_s[0];
  if (lse != nullptr && c == 0) lse[bh] = norm_s[1];
}

template <typename KV_T, int D>
size_t stage_bytes() { return size_t(2) * kTok * D * sizeof(KV_T); }

template <typename KV_T, typename Q_T, int D, int RH>
cudaError_t launch_one(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                       const int32_t* group_idx, const int32_t* n_selected, float* partial, float* out, float* lse,
                       uint32_t* err, cudaStream_t st) {
  const int depth = w.depth;
  const size_t smem = kControlBytes + stage_bytes<KV_T, D>() / 2 + size_t(kWarps) * depth * stage_bytes<KV_T, D>();
  int g_shift = -1;
  for (int sft = 0; sft < 31; ++sft) if ((1 << sft) == p.G) g_shift = sft;
  auto kern = sparse_decode_splitk_kernel<KV_T, Q_T, D, RH>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
  if (e != cudaSuccess) return e;
  e = launch_pdl(kern, dim3(w.splits, p.Hkv * (p.rho / RH), p.B), dim3(kThreads), smem, st, p,
                 static_cast<const Q_T*>(q), static_cast<const KV_T*>(K), static_cast<const KV_T*>(V), group_idx,
                 n_selected, partial, w.splits, depth, g_shift, err);
  if (e != cudaSuccess) return e;
  return launch_pdl(combine_kernel<D>, dim3(p.B * p.Hq), dim3(D), 0, st, static_cast<const float*>(partial), out,
                    lse, w.splits);
}

template <typename KV_T, typename Q_T, int D>
cudaError_t launch_rh(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                      const int32_t* gi, const int32_t* ns, float* partial, float* out, float* lse, uint32_t* err,
                      cudaStream_t st) {
  switch (w.heads_per_cta) {
    case 4: return launch_one<KV_T, Q_T, D, 4>(p, w, q, K, V, gi, ns, partial, out, lse, err, st);
    case 3: return launch_one<KV_T, Q_T, D, 3>(p, w, q, K, V, gi, ns, partial, out, lse, err, st);
    case 2: return launch_one<KV_T, Q_T, D, 2>(p, w, q, K, V, gi, ns, partial, out, lse, err, st);
    default: return launch_one<KV_T, Q_T, D, 1>(p, w, q, K, V, gi, ns, partial, out, lse, err, st);
  }
}

template <typename KV_T, typename Q_T>
cudaError_t launch_d(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                     const int32_t* gi, const int32_t* ns, float* partial, float* out, float* lse, uint32_t* err,
                     cudaStream_t st) {
  if (p.d == 128) return launch_rh<KV_T, Q_T, 128>(p, w, q, K, V, gi, ns, partial, out, lse, err, st);
  return launch_rh<KV_T, Q_T, 64>(p, w, q, K, V, gi, ns, partial, out, lse, err, st);
}

template <typename KV_T>
cudaError_t launch_q(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                     const int32_t* gi, const int32_t* ns, float* partial, float* out, float* lse, uint32_t* err,
                     cudaStream_t st) {
  // q is stored as fp32 or in the K/V type (checked at validation).
  if (p.q_dtype == KVSWAP_F32) return launch_d<KV_T, float>(p, w, q, K, V, gi, ns, partial, out, lse, err, st);
  return launch_d<KV_T, KV_T>(p, w, q, K, V, gi, ns, partial, out, lse, err, st);
}

}  // namespace

// Split-K factor and ring depth of sparse_decode for a problem (host side).
void plan_sparse_decode(const Problem& p, Workspace* w) {
  // rho query heads share each K/V row; a CTA serves up to 4 of them per pass.
  int rh = 1;
  for (int c = 4; c >= 1; --c) if (p.rho % c == 0) { rh = c; break; }
  w->heads_per_cta = rh;
  const int64_t problems = int64_t(p.B) * p.Hkv * (p.rho / rh);
  const int64_t tokens = int64_t(p.Mp) * p.G + (p.N - int64_t(p.NG) * p.G);
  const int64_t n_chunks = std::max<int64_t>(1, (tokens + kTok - 1) / kTok);
  // One wave of 2 CTAs per SM when the problems are few; otherwise the split that fills whole
  // waves best, keeping at least two chunks per compute warp and split.
  const int64_t slots = int64_t(kNumSMs) * 2;
  const int64_t max_splits = std::min<int64_t>(256, std::max<int64_t>(1, n_chunks / (2 * kWarps)));
  int64_t best = 1;
  double best_eff = 0.0;
  for (int64_t s = 1; s <= max_splits; ++s) {
    const int64_t ctas = problems * s;
    const int64_t waves = (ctas + slots - 1) / slots;
    if (waves > 2 && s > 1) break;
    const int64_t per = (n_chunks + s - 1) / s;               // chunks of the largest split
    const double eff = double(n_chunks) * problems / (double(waves) * slots * per);
    if (eff > best_eff * 1.02) { best_eff = eff; best = s; }
  }
  w->splits = int(best);
  const size_t row = size_t(p.d) * (p.kv_dtype == KVSWAP_F32 ? 4 : 2);
  const size_t stage = 2 * kTok * row;
  w->depth = int(std::max<size_t>(2, std::min<size_t>(kMaxDepth, (100u << 10) / (kWarps * stage))));
}

cudaError_t launch_sparse_decode(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                                 const int32_t* group_idx, const int32_t* n_selected, float* partial, float* out,
                                 float* lse, uint32_t* err, cudaStream_t st) {
  switch (p.kv_dtype) {
    case KVSWAP_F32: return launch_q<float>(p, w, q, K, V, group_idx, n_selected, partial, out, lse, err, st);
    case KVSWAP_BF16: return launch_q<__nv_bfloat16>(p, w, q, K, V, group_idx, n_selected, partial, out, lse, err, st);
    default: return launch_q<__half>(p, w, q, K, V, group_idx, n_selected, partial, out, lse, err, st);
  }
}

}  // namespace kvswap
