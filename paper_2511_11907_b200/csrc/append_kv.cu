// New KV entries (Sec. 4.4.1): the token generated in a decode step joins the rolling buffer.
//
// In this layout the rolling buffer is not a separate allocation: it is the rows of the K/V store
// past the last complete group, which the attention kernel always covers.  Appending is therefore
// one row copy per (sequence, KV head) for K and for V; the "flush" of a completed group leaves the
// rows where they are and only builds the group's rows of the compact cache (project_keys over
// the group's token range).
#include <algorithm>

#include "common.cuh"

namespace kvswap {
namespace {

constexpr int kMaxAppendLayers = 32;

// Stores of the layers one launch serves (blockIdx.y = layer).
struct StoreTable {
  unsigned char* K[kMaxAppendLayers];
  unsigned char* V[kMaxAppendLayers];
};

// One CTA per (sequence, KV head, layer): the first half of the threads copies the K row, the
// second half the V row, 16 bytes per thread.  k_new, v_new: [layers, B, H_kv, d].
__global__ void append_rows_kernel(const unsigned char* __restrict__ k_new, const unsigned char* __restrict__ v_new,
                                   const StoreTable stores, int Hkv, int row_bytes, int64_t sb_bytes, int64_t sh_bytes,
                                   int64_t row_offset_bytes) {
  const int bg = blockIdx.x, b = bg / Hkv, g = bg % Hkv, layer = blockIdx.y;
  const int pieces = row_bytes / 16;
  const int t = threadIdx.x;
  const bool is_v = t >= pieces;
  const int piece = is_v ? t - pieces : t;
  if (piece >= pieces) return;
  const int64_t src_off = (int64_t(layer) * gridDim.x + bg) * row_bytes + piece * 16;
  const unsigned char* src = (is_v ? v_new : k_new) + src_off;
  unsigned char* dst = (is_v ? stores.V[layer] : stores.K[layer]) + int64_t(b) * sb_bytes + int64_t(g) * sh_bytes +
                       row_offset_bytes + piece * 16;
  *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
}

// Flush of a completed group in a tiered cache: the G rows that accumulated in the rolling-buffer
// area of each layer's reuse store are written to the slow tier.  One CTA per (sequence, KV head,
// layer), 16 bytes per thread and step.
struct FlushTable {
  const unsigned char* K_fast[kMaxAppendLayers];
  const unsigned char* V_fast[kMaxAppendLayers];
  unsigned char* K_slow[kMaxAppendLayers];
  unsigned char* V_slow[kMaxAppendLayers];
};

__global__ void flush_rows_kernel(const FlushTable tab, int Hkv, int G, int row_bytes, int64_t fast_sb, int64_t fast_sh,
                                  int64_t fast_row0, int64_t slow_sb, int64_t slow_sh, int64_t slow_sn,
                                  int64_t slow_row0) {
  const int bg = blockIdx.x, b = bg / Hkv, g = bg % Hkv, layer = blockIdx.y;
  const int pieces = row_bytes / 16;
  for (int t = threadIdx.x; t < 2 * G * pieces; t += blockDim.x) {
    const int piece = t % pieces, row = (t / pieces) % G;
    const bool is_v = t >= G * pieces;
    const unsigned char* src = (is_v ? tab.V_fast[layer] : tab.K_fast[layer]) + int64_t(b) * fast_sb +
                               int64_t(g) * fast_sh + (fast_row0 + row) * row_bytes + piece * 16;
    unsigned char* dst = (is_v ? tab.V_slow[layer] : tab.K_slow[layer]) + int64_t(b) * slow_sb + int64_t(g) * slow_sh +
                         (slow_row0 + row) * slow_sn + piece * 16;
    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
  }
}

}  // namespace

// Copies rows [fast_row0, fast_row0 + G) of each layer's dense reuse store ([B, H_kv, fast_rows, d])
// to rows [slow_row0, slow_row0 + G) of the slow-tier store (strides of `p`).
cudaError_t launch_flush_rows(const Problem& p, const void* const* K_fast, const void* const* V_fast, void* const* K_slow,
                              void* const* V_slow, int n_layers, int64_t fast_rows, int64_t fast_row0, int64_t slow_row0,
                              cudaStream_t st) {
  const int e = (p.kv_dtype == KVSWAP_F32) ? 4 : 2;
  const int row_bytes = p.d * e;
  for (int l0 = 0; l0 < n_layers; l0 += kMaxAppendLayers) {
    const int count = std::min(kMaxAppendLayers, n_layers - l0);
    FlushTable tab = {};
    for (int l = 0; l < count; ++l) {
      tab.K_fast[l] = static_cast<const unsigned char*>(K_fast[l0 + l]);
      tab.V_fast[l] = static_cast<const unsigned char*>(V_fast[l0 + l]);
      tab.K_slow[l] = static_cast<unsigned char*>(K_slow[l0 + l]);
      tab.V_slow[l] = static_cast<unsigned char*>(V_slow[l0 + l]);
    }
    flush_rows_kernel<<<dim3(p.B * p.Hkv, count), 256, 0, st>>>(
        tab, p.Hkv, p.G, row_bytes, int64_t(p.Hkv) * fast_rows * row_bytes, fast_rows * row_bytes, fast_row0,
        p.kv_sb * e, p.kv_sh * e, p.kv_sn * e, slow_row0);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
  }
  return cudaSuccess;
}

// Writes k_new, v_new [n_layers, B, H_kv, d] to token row `n` of each layer's K and V (strides of
// `p`), kMaxAppendLayers layers per launch.
cudaError_t launch_append_rows(const Problem& p, const void* k_new, const void* v_new, void* const* K, void* const* V,
                               int n_layers, int n, cudaStream_t st) {
  const int e = (p.kv_dtype == KVSWAP_F32) ? 4 : 2;
  const int row_bytes = p.d * e;                     // 128 .. 512, a multiple of 16
  const int threads = 2 * (row_bytes / 16);
  const int64_t layer_bytes = int64_t(p.B) * p.Hkv * row_bytes;
  for (int l0 = 0; l0 < n_layers; l0 += kMaxAppendLayers) {
    const int count = std::min(kMaxAppendLayers, n_layers - l0);
    StoreTable stores = {};
    for (int l = 0; l < count; ++l) {
      stores.K[l] = static_cast<unsigned char*>(K[l0 + l]);
      stores.V[l] = static_cast<unsigned char*>(V[l0 + l]);
    }
    append_rows_kernel<<<dim3(p.B * p.Hkv, count), threads, 0, st>>>(
        static_cast<const unsigned char*>(k_new) + l0 * layer_bytes,
        static_cast<const unsigned char*>(v_new) + l0 * layer_bytes, stores, p.Hkv, row_bytes, p.kv_sb * e,
        p.kv_sh * e, int64_t(n) * p.kv_sn * e);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
  }
  return cudaSuccess;
}

}  // namespace kvswap
