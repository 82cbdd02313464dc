// New KV entries (Sec. 4.4.1): the token generated in a decode step joins the rolling buffer.
//
// In this layout the rolling buffer is not a separate allocation: it is the rows of the K/V store
// past the last complete group, which the attention kernel always covers.  Appending is therefore
// one row copy per (sequence, KV head) for K and for V; the "flush" of a completed group leaves the
// rows where they are and only builds the group's rows of the compact cache (project_keys over
// the group's token range).
#include "common.cuh"

namespace kvswap {
namespace {

// One CTA per (sequence, KV head): the first half of the threads copies the K row, the second half
// the V row, 16 bytes per thread.
__global__ void append_rows_kernel(const unsigned char* __restrict__ k_new, const unsigned char* __restrict__ v_new,
                                   unsigned char* __restrict__ K, unsigned char* __restrict__ V, int Hkv, int row_bytes,
                                   int64_t sb_bytes, int64_t sh_bytes, int64_t row_offset_bytes) {
  const int bg = blockIdx.x, b = bg / Hkv, g = bg % Hkv;
  const int pieces = row_bytes / 16;
  const int t = threadIdx.x;
  const bool is_v = t >= pieces;
  const int piece = is_v ? t - pieces : t;
  if (piece >= pieces) return;
  const unsigned char* src = (is_v ? v_new : k_new) + int64_t(bg) * row_bytes + piece * 16;
  unsigned char* dst = (is_v ? V : K) + int64_t(b) * sb_bytes + int64_t(g) * sh_bytes + row_offset_bytes + piece * 16;
  *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
}

}  // namespace

// Writes k_new, v_new [B, H_kv, d] to token row `n` of K and V (strides of `p`).
cudaError_t launch_append_rows(const Problem& p, const void* k_new, const void* v_new, void* K, void* V, int n,
                               cudaStream_t st) {
  const int e = (p.kv_dtype == KVSWAP_F32) ? 4 : 2;
  const int row_bytes = p.d * e;                     // 128 .. 512, a multiple of 16
  const int threads = 2 * (row_bytes / 16);
  append_rows_kernel<<<p.B * p.Hkv, threads, 0, st>>>(
      static_cast<const unsigned char*>(k_new), static_cast<const unsigned char*>(v_new),
      static_cast<unsigned char*>(K), static_cast<unsigned char*>(V), p.Hkv, row_bytes, p.kv_sb * e, p.kv_sh * e,
      int64_t(n) * p.kv_sn * e);
  return cudaGetLastError();
}

}  // namespace kvswap
