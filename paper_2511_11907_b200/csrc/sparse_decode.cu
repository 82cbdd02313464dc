// K4 + K5: exact decode attention over the selected groups and the rolling-buffer tail
// (Sec. 4.4, 4.4.1, 4.4.4): gather + split-K flash-decode with an fp32 online softmax, then a
// log-sum-exp merge of the split partials.
//
// The attended tokens of one (sequence, selection row) form a virtual list
//     v in [0, M*G):  token  group_idx[v / G] * G + v % G   (absent when v / G >= n_sel or the index is invalid)
//     v in [M*G, M*G + tail):  token  NG*G + (v - M*G)
// which is cut into `splits` contiguous ranges, one CTA each, and every range into chunks of
// kTok tokens.  A CTA serves RH query heads that share the KV head, so each K/V row is read once.
//
// Every warp of the CTA works alone on the chunks c = warp, warp + kWarps, ...: it owns `depth`
// shared-memory stages and keeps them filled itself with 16-byte asynchronous copies (cp.async,
// one commit group per chunk), all 32 lanes copying: lanes 0..7 resolve the kTok token rows of a
// chunk, every lane then moves 16-byte pieces of those rows.  The copy for chunk k + depth is
// issued the moment chunk k has been consumed, so `depth` chunks per warp are in flight while it
// computes, no warp ever waits for another, and the only wait is cp.async.wait_group on the
// warp's own copies.  Rows of absent tokens (invalid group index, ragged end) are zero-filled.
//
// Staged rows are swizzled: 16-byte piece c of row r sits at piece c ^ (r % 8).  Eight rows read
// at the same logical piece (ldmatrix, or the row-parallel reads of the fp32 engine) then fall
// into eight different bank groups although the row pitch is a multiple of 128 bytes.
//
// What a warp does with a chunk is the business of its compute engine (below): fp32 pipes for
// fp32 K/V, tensor cores for 16-bit K/V.
#include <algorithm>
#include <cstdint>

#include "async_copy.cuh"
#include "combine.cuh"
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
  uint32_t mask[kMaxStages];                    // bit t: token slot t of the stage holds a row
  float2 prob[kWarps][kTok * 4];                // softmax weights of the chunk, [token][head], each twice
  float2 corr[kWarps][4];                       // rescale of the running accumulator, [head], each twice
};
constexpr int kControlBytes = (sizeof(Control) + 255) & ~255;

// Byte offset inside a stage half of byte `col` of row `r` (rows of ROWB bytes, pieces of 16).
template <uint32_t ROWB>
__device__ __forceinline__ uint32_t swz(uint32_t r, uint32_t col) {
  return r * ROWB + ((((col >> 4) ^ (r & 7u)) << 4) | (col & 15u));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  // src_bytes = 16 copies, 0 writes zeros without touching global memory
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

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

// ------------------------------------------------------------------------------------------
// Per-warp compute engines.  Both keep the online-softmax state of RH heads over the chunks a
// warp consumes and share one interface:
//   init(q of head 0 of the CTA, lane)        load the query slice
//   chunk(stage K address, stage V address, mask, probability tile, correction tile)
//   store(sm_m, sm_l, sm_acc)                  state -> shared memory for the CTA merge
//
// AluEngine: fp32 pipes.  A lane owns D/32 channels.  For a chunk it forms the kTok x RH partial
// dot products of its channel slice, then transposes-and-sums them across the warp (a
// reduce-scatter by shuffles) so that lane L ends up with the complete logit of (token L/4, head
// L%4): the softmax bookkeeping then runs once per chunk with all 32 lanes busy.  Probabilities
// go through a small shared-memory tile back to all lanes for the P.V update of their channels.
// ------------------------------------------------------------------------------------------
template <typename KV_T, typename Q_T, int D, int RH>
struct AluEngine {
  static constexpr int DPL = D / 32;                           // channels per lane
  static constexpr uint32_t ROWB = D * sizeof(KV_T);
  static constexpr uint32_t kFull = 0xffffffffu;
  float2 qq[RH][DPL];              // q slice, pre-scaled, each value twice (two tokens per packed FMA)
  float2 acc[RH][DPL / 2];         // channel pairs
  float m_run, l_run;              // of head lane % 4 (replicated over the tokens)
  int lane, tok, hd;
  uint32_t lane_col;               // first byte of this lane's channels within a row

  __device__ __forceinline__ void init(const Q_T* q0, int lane_) {
    lane = lane_; tok = lane >> 2; hd = lane & 3;
    lane_col = uint32_t(lane) * DPL * sizeof(KV_T);
    const float scale = kLog2e * rsqrtf(float(D));             // logits live in the log2 domain
#pragma unroll
    for (int hh = 0; hh < RH; ++hh)
#pragma unroll
      for (int j = 0; j < DPL; ++j) {
        const float x = q_to_float(q0[hh * D + lane * DPL + j]) * scale;
        qq[hh][j] = make_float2(x, x);
      }
    m_run = -INFINITY; l_run = 0.f;
#pragma unroll
    for (int hh = 0; hh < RH; ++hh)
#pragma unroll
      for (int j = 0; j < DPL / 2; ++j) acc[hh][j] = make_float2(0.f, 0.f);
  }

  __device__ __forceinline__ void chunk(uint32_t kstage, uint32_t vstage, uint32_t mask, float2* prob, float2* corr) {
    // ---- partial q.k of this lane's channels; register slot s holds token s ^ tok (so that the
    // reduce-scatter below needs no selects), slots s and s + 4 share a packed accumulator -------
    float2 part[4][4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      float ka[DPL], kb[DPL];
      lds_row<KV_T, DPL>(kstage + swz<ROWB>(uint32_t(s ^ tok), lane_col), ka);
      lds_row<KV_T, DPL>(kstage + swz<ROWB>(uint32_t((s + 4) ^ tok), lane_col), kb);
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
    // ---- reduce-scatter over the warp: tokens over lane bits 4..2, heads over bits 1..0 --------
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

    // ---- online softmax for (token tok, head hd) ------------------------------------------------
    const bool live = ((mask >> tok) & 1u) && hd < RH;
    s_log = live ? s_log : -INFINITY;
    float cmax = s_log;
    cmax = fmaxf(cmax, __shfl_xor_sync(kFull, cmax, 4));
    cmax = fmaxf(cmax, __shfl_xor_sync(kFull, cmax, 8));
    cmax = fmaxf(cmax, __shfl_xor_sync(kFull, cmax, 16));
    const float m_new = fmaxf(m_run, cmax);
    const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
    const float pw = ex2(s_log - m_safe);            // 0 for dead (token, head) pairs
    const float cr = ex2(m_run - m_safe);            // 0 while nothing has been seen yet
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

    // ---- P.V on this lane's channels -------------------------------------------------------------
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
      lds_row<KV_T, DPL>(vstage + swz<ROWB>(uint32_t(t), lane_col), vf);
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
        if ((mask >> t) & 1u) pv_token(t);            // warp-uniform
    }
  }

  // sm_m, sm_l: [8] per warp;  sm_acc: [RH][D] per warp
  __device__ __forceinline__ void store(float* sm_m, float* sm_l, float* sm_acc) const {
    if (lane < 4) { sm_m[lane] = m_run; sm_l[lane] = l_run; }
#pragma unroll
    for (int hh = 0; hh < RH; ++hh)
#pragma unroll
      for (int j = 0; j < DPL / 2; ++j)
        *reinterpret_cast<float2*>(&sm_acc[hh * D + lane * DPL + 2 * j]) = acc[hh][j];
  }
};

// ------------------------------------------------------------------------------------------
// MmaEngine: 16-bit K/V and q of the same type.  With rho heads sharing every K/V row the two
// products of a chunk are small dense contractions -- logits[heads x tokens] = Q[heads x d] K^T
// and out^T[d x heads] += V^T[d x tokens] P[tokens x heads] -- and at ~60 fp32 instructions per
// token the fp32 pipes, not HBM, bound the gather.  They run on the tensor cores instead
// (mma.sync, fp32 accumulation), operands fetched from the staged rows with ldmatrix:
//   logits: m16n8k16, A = Q (rows = heads, rows >= RH zero; kept in registers), B = K^T, so
//           lane (g = lane/4, t = lane%4) with g < RH receives head g's logits of tokens 2t, 2t+1;
//   P.V:    m16n8k8 per 16 channels, A = V^T (ldmatrix.trans), B = P -- whose fragment layout is
//           exactly the one the logits arrive in.  P is split into a 16-bit head and a 16-bit
//           remainder (two products) so that the weights stay fp32-accurate.
// Q, K and V enter unrounded (they are stored in the operand type); the scale 1/sqrt(d) is
// applied to the fp32 logits.
// ------------------------------------------------------------------------------------------
template <typename KV_T>
__device__ __forceinline__ void mma_k16(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  // rows 8..15 of A (a1, a3) are zero
  if constexpr (std::is_same<KV_T, __nv_bfloat16>::value) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
  } else {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
  }
}
template <typename KV_T>
__device__ __forceinline__ void mma_k8(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  if constexpr (std::is_same<KV_T, __nv_bfloat16>::value) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(b0));
  } else {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(b0));
  }
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// Two fp32 values -> packed 16-bit pair (x in the low half) and the packed remainders.
template <typename KV_T>
__device__ __forceinline__ void split_pair(float x, float y, uint32_t& hi, uint32_t& lo) {
  if constexpr (std::is_same<KV_T, __nv_bfloat16>::value) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
    const float2 hf = __bfloat1622float2(h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(x - hf.x, y - hf.y);
    hi = *reinterpret_cast<const uint32_t*>(&h); lo = *reinterpret_cast<const uint32_t*>(&l);
  } else {
    const __half2 h = __floats2half2_rn(x, y);
    const float2 hf = __half22float2(h);
    const __half2 l = __floats2half2_rn(x - hf.x, y - hf.y);
    hi = *reinterpret_cast<const uint32_t*>(&h); lo = *reinterpret_cast<const uint32_t*>(&l);
  }
}

template <typename KV_T, typename Q_T, int D, int RH>
struct MmaEngine {
  static_assert(sizeof(KV_T) == 2 && std::is_same<KV_T, Q_T>::value, "16-bit K/V and q of one type");
  static constexpr uint32_t ROWB = D * sizeof(KV_T);
  static constexpr uint32_t kFull = 0xffffffffu;
  static constexpr int KS = D / 16;          // k-steps of the logits = 16-channel blocks of the output
  uint32_t qa[KS][2];                        // A fragments of Q (rows 0..7 of each k-step)
  float oacc[KS][4];                         // out^T: [block][0,1] channel 16*blk+g, heads 2t,2t+1; [2,3] channel +8
  float m_run, l_run;                        // of head g = lane / 4 (replicated over t)
  float scale;
  int lane, g, t;
  uint32_t ld_row, ld_piece;                 // ldmatrix: row this lane addresses, piece within a 64-byte span

  __device__ __forceinline__ void init(const Q_T* q0, int lane_) {
    lane = lane_; g = lane >> 2; t = lane & 3;
    scale = kLog2e * rsqrtf(float(D));
    ld_row = uint32_t(lane & 7); ld_piece = uint32_t(lane >> 3);
    const uint32_t* qrow = reinterpret_cast<const uint32_t*>(q0 + (g < RH ? g : 0) * D);   // 2 channels per word
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qa[ks][0] = (g < RH) ? qrow[8 * ks + t] : 0u;            // channels 16ks + 2t, +1
      qa[ks][1] = (g < RH) ? qrow[8 * ks + 4 + t] : 0u;        // channels 16ks + 8 + 2t, +1
    }
#pragma unroll
    for (int i = 0; i < KS; ++i) { oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f; }
    m_run = -INFINITY; l_run = 0.f;
  }

  __device__ __forceinline__ void chunk(uint32_t kstage, uint32_t vstage, uint32_t mask, float2*, float2*) {
    // ---- logits of head g for tokens 2t, 2t+1 -----------------------------------------------------
    float sacc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int kk = 0; kk < D / 32; ++kk) {
      uint32_t r[4];
      ldsm_x4(kstage + swz<ROWB>(ld_row, (uint32_t(4 * kk) + ld_piece) << 4), r);   // channels 32kk .. 32kk+31
      mma_k16<KV_T>(sacc, qa[2 * kk][0], qa[2 * kk][1], r[0], r[1]);
      mma_k16<KV_T>(sacc, qa[2 * kk + 1][0], qa[2 * kk + 1][1], r[2], r[3]);
    }
    const bool head_ok = g < RH;
    float s0 = (head_ok && ((mask >> (2 * t)) & 1u)) ? sacc[0] * scale : -INFINITY;
    float s1 = (head_ok && ((mask >> (2 * t + 1)) & 1u)) ? sacc[1] * scale : -INFINITY;
    // ---- online softmax of head g over the four lanes that share it ----------------------------------
    float cmax = fmaxf(s0, s1);
    cmax = fmaxf(cmax, __shfl_xor_sync(kFull, cmax, 1));
    cmax = fmaxf(cmax, __shfl_xor_sync(kFull, cmax, 2));
    const float m_new = fmaxf(m_run, cmax);
    const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
    const float p0 = ex2(s0 - m_safe), p1 = ex2(s1 - m_safe);  // 0 for absent tokens / heads
    const float cr = ex2(m_run - m_safe);                      // 0 while nothing has been seen yet
    float psum = p0 + p1;
    psum += __shfl_xor_sync(kFull, psum, 1);
    psum += __shfl_xor_sync(kFull, psum, 2);
    l_run = fmaf(l_run, cr, psum);
    m_run = m_new;
    if (__any_sync(kFull, head_ok && cr != 1.f)) {
      // accumulator columns of this lane are heads 2t and 2t+1: their factors live in lanes 8t, 8t+4
      const float c0 = __shfl_sync(kFull, cr, (8 * t) & 31), c1 = __shfl_sync(kFull, cr, (8 * t + 4) & 31);
#pragma unroll
      for (int i = 0; i < KS; ++i) { oacc[i][0] *= c0; oacc[i][1] *= c1; oacc[i][2] *= c0; oacc[i][3] *= c1; }
    }
    // ---- out^T += V^T P, P = head + remainder -----------------------------------------------------------
    uint32_t phi, plo;
    split_pair<KV_T>(p0, p1, phi, plo);
#pragma unroll
    for (int kk = 0; kk < D / 32; ++kk) {
      uint32_t r[4];
      ldsm_x4_trans(vstage + swz<ROWB>(ld_row, (uint32_t(4 * kk) + ld_piece) << 4), r);   // V^T, channels 32kk .. 32kk+31
      mma_k8<KV_T>(oacc[2 * kk], r[0], r[1], phi);
      mma_k8<KV_T>(oacc[2 * kk], r[0], r[1], plo);
      mma_k8<KV_T>(oacc[2 * kk + 1], r[2], r[3], phi);
      mma_k8<KV_T>(oacc[2 * kk + 1], r[2], r[3], plo);
    }
  }

  __device__ __forceinline__ void store(float* sm_m, float* sm_l, float* sm_acc) const {
    if (t == 0) { sm_m[g] = m_run; sm_l[g] = l_run; }        // g = 0..7: one slot per possible head
#pragma unroll
    for (int i = 0; i < KS; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int head = 2 * t + (e & 1), ch = 16 * i + g + ((e & 2) ? 8 : 0);
        if (head < RH) sm_acc[head * D + ch] = oacc[i][e];
      }
  }
};

// Where the attended tokens of one CTA come from.
struct TokenSource {
  const int32_t* idx;      // selection row
  int NG, G, g_shift;      // g_shift = log2(G) when G is a power of two, else -1
  int sel_tokens, tail0;   // n_sel * G, NG * G
  int v_begin, v_end;      // this CTA's range of the virtual token list

  // Group ordinal of virtual token v (v < sel_tokens).
  __device__ __forceinline__ int group_of(int v) const { return g_shift >= 0 ? (v >> g_shift) : (v / G); }
};

template <typename KV_T, typename Q_T, int D, int RH, typename Engine>
__global__ void __launch_bounds__(kThreads, 2)
sparse_decode_splitk_kernel(Problem p, const Q_T* __restrict__ q, const KV_T* __restrict__ K,
                            const KV_T* __restrict__ V, const int32_t* __restrict__ group_idx,
                            const int32_t* __restrict__ n_selected, float* __restrict__ partial,
                            int splits, int depth, int g_shift, uint32_t* __restrict__ err) {
  constexpr uint32_t ROWB = D * sizeof(KV_T);                  // bytes of one K or V row
  constexpr uint32_t HALFB = kTok * ROWB;                      // K (or V) part of a stage
  constexpr uint32_t STAGEB = 2 * HALFB;
  constexpr uint32_t kFull = 0xffffffffu;

  extern __shared__ unsigned char smem_raw[];
  Control* ctl = reinterpret_cast<Control*>(smem_raw);
  // Stage ring, aligned to 128 bytes (the swizzle works on row-relative offsets).
  const uint32_t ring = (smem_addr(smem_raw) + kControlBytes + 127u) & ~127u;
  unsigned char* ring_ptr = smem_raw + (ring - smem_addr(smem_raw));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x;
  const int chunks = p.rho / RH;
  const int g = blockIdx.y / chunks, hc = blockIdx.y % chunks;
  const int b = blockIdx.z;
  const int h0 = g * p.rho + hc * RH;                          // first query head of this CTA
  const int srow = (p.scope == KVSWAP_SCOPE_KV_HEAD) ? g : 0;

  // Everything below may depend on the previous kernel in the stream -- unless the caller has
  // promised that q and the selection are settled: then only this kernel's writes (the partials,
  // which the previous launch's combine may still be reading) have to wait for it.
  const bool settled = (p.flags & KVSWAP_INPUTS_SETTLED) != 0;
  const bool wait_early = settled && (p.flags & kFlagWaitEarly) != 0;
  if (!settled) pdl_wait();
  if (!wait_early) pdl_trigger();

  // The virtual token list is laid out for M selected groups, whatever n_selected says (slots of
  // groups beyond n_selected are simply absent), so that the split of the list does not wait for a
  // global read: n_selected is fetched together with the first group indices.
  TokenSource src;
  src.idx = group_idx + (int64_t(b) * p.S + srow) * p.M;
  src.NG = p.NG; src.G = p.G; src.g_shift = g_shift;
  src.tail0 = p.NG * p.G;
  src.sel_tokens = p.M * p.G;
  {
    const int total = src.sel_tokens + (p.N - src.tail0);
    int per_split = (total + splits - 1) / splits;
    per_split = (per_split + kTok - 1) / kTok * kTok;
    src.v_begin = min(total, per_split * split);
    src.v_end = min(total, src.v_begin + per_split);
  }
  const int n_sel_given = n_selected[int64_t(b) * p.S + srow];
  const int n_sel = max(0, min(n_sel_given, p.M));
  // KVSWAP_CHECK_INDICES: the first split of each list looks it over once, ahead of the loop (which skips what
  // is out of range either way), and records what it finds.  (No wait in this kernel can run out: err serves this only.)
  if ((p.flags & KVSWAP_CHECK_INDICES) != 0 && err != nullptr && split == 0) {
    bool bad = n_sel != n_sel_given;
    for (int i = threadIdx.x; i < n_sel; i += kThreads) {
      const int j = src.idx[i];
      bad = bad || (j != -1 && (j < 0 || j >= p.NG));
    }
    if (bad) atomicExch(err, kDevBadIndex);
  }
  const int n_chunks = (src.v_end - src.v_begin + kTok - 1) / kTok;
  const int my_chunks = (n_chunks > warp) ? (n_chunks - warp + kWarps - 1) / kWarps : 0;   // of this warp

  const unsigned char* Kg = reinterpret_cast<const unsigned char*>(K + int64_t(b) * p.kv_sb + int64_t(g) * p.kv_sh);
  const unsigned char* Vg = reinterpret_cast<const unsigned char*>(V + int64_t(b) * p.kv_sb + int64_t(g) * p.kv_sh);
  const int64_t row_pitch = p.kv_sn * int64_t(sizeof(KV_T));   // bytes between token rows in global memory

  // Group index (or -1) behind token slot `lane` of this warp's k-th chunk: the one dependent
  // global read of the fill path, issued early so that its latency hides behind a chunk's compute.
  auto fetch_group = [&](int k) -> int {
    const int v = src.v_begin + (warp + k * kWarps) * kTok + lane;
    if (lane < kTok && k < my_chunks && v < src.v_end && v < src.sel_tokens) {
      const int go = src.group_of(v);
      if (go < n_sel) return src.idx[go];
    }
    return -1;
  };
  // Fill: bring chunk k into `stage` (one commit group).  `j` is fetch_group(k).  All lanes call.
  constexpr uint32_t kPieces = ROWB / 16;                      // 16-byte pieces per row
  auto fill = [&](int k, int j, int stage) {
    if (k < my_chunks) {
      const int v = src.v_begin + (warp + k * kWarps) * kTok + lane;
      int n = -1;                                              // token row behind slot `lane`
      if (lane < kTok && v < src.v_end) {
        if (v < src.sel_tokens) {
          if (j >= 0 && j < src.NG) n = j * src.G + (v - src.group_of(v) * src.G);
        } else {
          n = src.tail0 + (v - src.sel_tokens);
        }
      }
      const uint32_t vmask = __ballot_sync(kFull, n >= 0);
      if (lane == 0) ctl->mask[stage] = vmask;
      const uint32_t kdst = ring + uint32_t(stage) * STAGEB;
#pragma unroll
      for (uint32_t i = 0; i < kTok * kPieces / 32; ++i) {
        const uint32_t e = i * 32 + uint32_t(lane);
        const uint32_t r = e / kPieces, c = e % kPieces;
        const int n_r = __shfl_sync(kFull, n, int(r));
        const int64_t off = int64_t(n_r < 0 ? 0 : n_r) * row_pitch + int64_t(c) * 16;
        const uint32_t bytes = n_r < 0 ? 0u : 16u;
        const uint32_t d = kdst + swz<ROWB>(r, c << 4);
        cp_async16(d, Kg + off, bytes);
        cp_async16(d + HALFB, Vg + off, bytes);
      }
    }
    cp_async_commit();                                         // an empty group keeps the count uniform
  };

  // ---- prologue: fill the first `depth` stages ---------------------------------------------------
  {
    int j0[kMaxDepth];
#pragma unroll
    for (int k = 0; k < kMaxDepth; ++k) j0[k] = (k < depth) ? fetch_group(k) : -1;
#pragma unroll
    for (int k = 0; k < kMaxDepth; ++k)
      if (k < depth) fill(k, j0[k], warp + kWarps * k);
  }
  if (wait_early) {                                // the first fills are in flight
    pdl_wait();
    pdl_trigger();
  }

  Engine eng;
  eng.init(q + (int64_t(b) * p.Hq + h0) * D, lane);
  float2* prob = ctl->prob[warp];
  float2* corr = ctl->corr[warp];
  int slot = 0;
  for (int k = 0; k < my_chunks; ++k) {
    const int stage = warp + kWarps * slot;
    const int j_next = fetch_group(k + depth);     // consumed by the refill at the end of the iteration
    // `depth` groups are in flight and the oldest is chunk k's: wait until depth - 1 remain.
    if (depth == 2) cp_async_wait<1>(); else if (depth == 3) cp_async_wait<2>(); else cp_async_wait<3>();
    __syncwarp();                                  // every lane's pieces of the chunk have landed
    const uint32_t mask = ctl->mask[stage];
    if (mask != 0u) {
      const uint32_t kstage = ring + uint32_t(stage) * STAGEB;
      eng.chunk(kstage, kstage + HALFB, mask, prob, corr);
    }
    __syncwarp();                                  // all lanes are done with the stage and prob[]
    fill(k + depth, j_next, stage);
    if (++slot == depth) slot = 0;
  }
  cp_async_wait<0>();

  // ---- merge the warps of the CTA ------------------------------------------------------------------
  __syncthreads();
  // The ring is idle now (every copy was waited for); reuse it for the merge.
  float* sm_m = reinterpret_cast<float*>(ring_ptr);                 // [kWarps][8]
  float* sm_l = sm_m + kWarps * 8;                                  // [kWarps][8]
  float* sm_acc = sm_l + kWarps * 8;                                // [kWarps][RH][D]
  eng.store(sm_m + warp * 8, sm_l + warp * 8, sm_acc + warp * RH * D);
  __syncthreads();
  if (settled && !wait_early) pdl_wait();
  for (int i = threadIdx.x; i < RH * D; i += kThreads) {
    const int hh = i / D, c = i % D;
    float mx = -INFINITY;
#pragma unroll
    for (int k = 0; k < kWarps; ++k) mx = fmaxf(mx, sm_m[k * 8 + hh]);
    float lsum = 0.f, a = 0.f;
    if (mx > -INFINITY) {
#pragma unroll
      for (int k = 0; k < kWarps; ++k) {
        const float w = ex2(sm_m[k * 8 + hh] - mx);
        lsum = fmaf(sm_l[k * 8 + hh], w, lsum);
        a = fmaf(sm_acc[(k * RH + hh) * D + c], w, a);
      }
    }
    float* dst = partial + ((int64_t(b) * p.Hq + h0 + hh) * splits + split) * (D + 2);
    if (c == 0) { dst[0] = mx; dst[1] = lsum; }
    dst[2 + c] = a;
  }
}

// K5: merge the split partials of one (sequence, head): one CTA of D threads per row (combine.cuh).
template <int D>
__global__ void __launch_bounds__(D)
combine_kernel(const float* __restrict__ partial, float* __restrict__ out, float* __restrict__ lse, int splits) {
  __shared__ float w_s[kMaxSplits];
  __shared__ float norm_s[2];                  // 1 / sum of weights (or 0), lse
  // The next kernel of the stream may start its own prologue at once; this one needs the
  // partials of the gather kernel before it.
  pdl_trigger();
  pdl_wait();
  combine_row<D>(partial, out, lse, splits, blockIdx.x, true, threadIdx.x, w_s, norm_s, 0);
}

template <typename KV_T, int D>
size_t stage_bytes() { return size_t(2) * kTok * D * sizeof(KV_T); }

template <typename KV_T, typename Q_T, int D, int RH>
cudaError_t launch_one(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                       const int32_t* group_idx, const int32_t* n_selected, float* partial, float* out, float* lse,
                       uint32_t* err, bool combine, cudaStream_t st) {
  const int depth = w.depth;
  const size_t smem = kControlBytes + 128 + size_t(kWarps) * depth * stage_bytes<KV_T, D>();
  int g_shift = -1;
  for (int sft = 0; sft < 31; ++sft) if ((1 << sft) == p.G) g_shift = sft;
  // Tensor-core engine for 16-bit K/V with q of the same type (up to 8 heads per K/V row); the
  // fp32-pipe engine otherwise (up to 4).
  constexpr bool kMma = sizeof(KV_T) == 2 && std::is_same<KV_T, Q_T>::value;
  using Engine = typename std::conditional<kMma, MmaEngine<KV_T, KV_T, D, RH>, AluEngine<KV_T, Q_T, D, (RH <= 4 ? RH : 4)>>::type;
  if (!kMma && RH > 4) return cudaErrorInvalidValue;             // never planned: see plan_sparse_decode
  auto kern = sparse_decode_splitk_kernel<KV_T, Q_T, D, RH, Engine>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
  if (e != cudaSuccess) return e;
  e = launch_pdl(kern, dim3(w.splits, p.Hkv * (p.rho / RH), p.B), dim3(kThreads), smem, st, p,
                 static_cast<const Q_T*>(q), static_cast<const KV_T*>(K), static_cast<const KV_T*>(V), group_idx,
                 n_selected, partial, w.splits, depth, g_shift, err);
  if (e != cudaSuccess || !combine) return e;
  return launch_pdl(combine_kernel<D>, dim3(p.B * p.Hq), dim3(D), 0, st, static_cast<const float*>(partial), out,
                    lse, w.splits);
}

template <typename KV_T, typename Q_T, int D>
cudaError_t launch_rh(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                      const int32_t* gi, const int32_t* ns, float* partial, float* out, float* lse, uint32_t* err,
                      bool combine, cudaStream_t st) {
  switch (w.heads_per_cta) {
    case 8: return launch_one<KV_T, Q_T, D, 8>(p, w, q, K, V, gi, ns, partial, out, lse, err, combine, st);
    case 7: return launch_one<KV_T, Q_T, D, 7>(p, w, q, K, V, gi, ns, partial, out, lse, err, combine, st);
    case 6: return launch_one<KV_T, Q_T, D, 6>(p, w, q, K, V, gi, ns, partial, out, lse, err, combine, st);
    case 5: return launch_one<KV_T, Q_T, D, 5>(p, w, q, K, V, gi, ns, partial, out, lse, err, combine, st);
    case 4: return launch_one<KV_T, Q_T, D, 4>(p, w, q, K, V, gi, ns, partial, out, lse, err, combine, st);
    case 3: return launch_one<KV_T, Q_T, D, 3>(p, w, q, K, V, gi, ns, partial, out, lse, err, combine, st);
    case 2: return launch_one<KV_T, Q_T, D, 2>(p, w, q, K, V, gi, ns, partial, out, lse, err, combine, st);
    default: return launch_one<KV_T, Q_T, D, 1>(p, w, q, K, V, gi, ns, partial, out, lse, err, combine, st);
  }
}

template <typename KV_T, typename Q_T>
cudaError_t launch_d(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                     const int32_t* gi, const int32_t* ns, float* partial, float* out, float* lse, uint32_t* err,
                     bool combine, cudaStream_t st) {
  if (p.d == 128) return launch_rh<KV_T, Q_T, 128>(p, w, q, K, V, gi, ns, partial, out, lse, err, combine, st);
  return launch_rh<KV_T, Q_T, 64>(p, w, q, K, V, gi, ns, partial, out, lse, err, combine, st);
}

template <typename KV_T>
cudaError_t launch_q(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                     const int32_t* gi, const int32_t* ns, float* partial, float* out, float* lse, uint32_t* err,
                     bool combine, cudaStream_t st) {
  // q is stored as fp32 or in the K/V type (checked at validation).
  if (p.q_dtype == KVSWAP_F32) return launch_d<KV_T, float>(p, w, q, K, V, gi, ns, partial, out, lse, err, combine, st);
  return launch_d<KV_T, KV_T>(p, w, q, K, V, gi, ns, partial, out, lse, err, combine, st);
}

}  // namespace

// Split-K factor and ring depth of sparse_decode for a problem (host side).
void plan_sparse_decode(const Problem& p, Workspace* w) {
  // rho query heads share each K/V row; a CTA serves up to 4 of them per pass.
  int rh = 1;
  // the tensor-core engine (16-bit K/V, q of the same type) takes up to 8, the fp32-pipe engine up to 4
  const int rh_max = (p.kv_dtype != KVSWAP_F32 && p.q_dtype == p.kv_dtype) ? 8 : 4;
  for (int c = rh_max; c >= 1; --c) if (p.rho % c == 0) { rh = c; break; }
  w->heads_per_cta = rh;
  const int64_t problems = int64_t(p.B) * p.Hkv * (p.rho / rh);
  const int64_t tokens = int64_t(p.M) * p.G + (p.N - int64_t(p.NG) * p.G);
  const int64_t n_chunks = std::max<int64_t>(1, (tokens + kTok - 1) / kTok);
  // Cost of a split factor s, in chunk times of the slowest CTA: waves * (chunks per CTA + the
  // fixed part of a CTA -- first index fetch, first rows, merge -- worth about 14 chunks), with
  // 2 CTAs per SM resident; at least two chunks per warp and split.
  const int64_t slots = int64_t(kNumSMs) * 2;
  const int64_t max_splits = std::min<int64_t>(256, std::max<int64_t>(1, n_chunks / (2 * kWarps)));
  int64_t best = 1, best_cost = INT64_MAX;
  for (int64_t s = 1; s <= max_splits; ++s) {
    const int64_t waves = (problems * s + slots - 1) / slots;
    if (waves > 2 && s > 1) break;
    const int64_t cost = waves * ((n_chunks + s - 1) / s + 14);
    if (cost < best_cost) { best_cost = cost; best = s; }
  }
  w->splits = int(best);
  const size_t row = size_t(p.d) * (p.kv_dtype == KVSWAP_F32 ? 4 : 2);
  const size_t stage = 2 * kTok * row;
  w->depth = int(std::max<size_t>(2, std::min<size_t>(kMaxDepth, (100u << 10) / (kWarps * stage))));
}

// The combine pass alone, for a gather that was enqueued with combine = false.
cudaError_t launch_combine_only(const Problem& p, const Workspace& w, const float* partial, float* out, float* lse,
                                cudaStream_t st) {
  if (p.d == 128)
    return launch_pdl(combine_kernel<128>, dim3(p.B * p.Hq), dim3(128), 0, st, partial, out, lse, w.splits);
  return launch_pdl(combine_kernel<64>, dim3(p.B * p.Hq), dim3(64), 0, st, partial, out, lse, w.splits);
}

cudaError_t launch_sparse_decode(const Problem& p, const Workspace& w, const void* q, const void* K, const void* V,
                                 const int32_t* group_idx, const int32_t* n_selected, float* partial, float* out,
                                 float* lse, uint32_t* err, cudaStream_t st, bool combine) {
  switch (p.kv_dtype) {
    case KVSWAP_F32: return launch_q<float>(p, w, q, K, V, group_idx, n_selected, partial, out, lse, err, combine, st);
    case KVSWAP_BF16: return launch_q<__nv_bfloat16>(p, w, q, K, V, group_idx, n_selected, partial, out, lse, err, combine, st);
    default: return launch_q<__half>(p, w, q, K, V, group_idx, n_selected, partial, out, lse, err, combine, st);
  }
}

}  // namespace kvswap
